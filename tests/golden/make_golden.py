"""Writes tests/golden/oracle_tiny_slab.json: the oracle's outputs for one small seeded slab.

The file pins the oracle against accidental change (a deliberate change of its arithmetic regenerates the
file in the same commit and says which passage of the paper justifies it).  Only the oracle and the seeded
input generator are used; nothing here touches the CUDA library.

    python tests/golden/make_golden.py
"""
import json
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import oracle                                             # noqa: E402
from paper_2512_07993_b200 import workloads as W         # noqa: E402


def compute():
    cfg = W.config(0, batch=1, ctx_lo=160, ctx_hi=160, budget=64, seed=4242)
    L = W.make_layer(cfg)
    b, h, g = 0, 1, cfg.group
    rows = W.slab_rows(L, b, h)
    N, S = int(L["kv_len"][b, h]), int(L["n_sent"][b, h])
    K, V = W.bf16_bits(L["K"])[rows][:N], W.bf16_bits(L["V"])[rows][:N]
    Q = W.bf16_bits(L["q_win"])[b, h * g:(h + 1) * g]
    off, sid = L["sent_off"][b, h, :S + 1], L["sent_id"][b, h, :S]
    tok = oracle.token_importance(K, Q)
    imp, vbar = oracle.pool(K, off, tok, 1e-6)
    _, red, lam = oracle.gram_terms(vbar, 0.95)
    score = oracle.final_score(imp, red, lam, 0.1)
    keep, kept, new_len = oracle.select(score, off, cfg.budget, cfg.window)
    keep_f, tok_keep, new_len_f = oracle.select_fill(score, off, tok.astype(np.float32), cfg.budget, cfg.window)
    Ko, _, im, nso, nsid = oracle.compact(K, V, keep, off, sid)
    out_bits, _ = oracle.decode_attn(W.bf16_bits(L["q"])[b, h * g:(h + 1) * g], Ko, oracle.compact(K, V, keep, off, sid)[1], len(im))
    red_tok = oracle.token_redundancy(K[:48])
    r = lambda a: [float(f"{x:.12e}") for x in np.asarray(a, np.float64)]
    return {
        "input": "workloads.config(0, batch=1, ctx_lo=160, ctx_hi=160, budget=64, seed=4242), slab (0, 1)",
        "sent_off": [int(x) for x in off],
        "tok_imp_first8": r(tok[:8]), "tok_imp_sum": float(f"{tok.sum():.12e}"),
        "imp": r(imp), "red": r(red), "lam": r(lam), "score_f32": r(score),
        "keep": [int(x) for x in keep], "new_len": int(new_len),
        "keep_fill": [int(x) for x in keep_f], "tok_keep_fill": [int(x) for x in np.nonzero(tok_keep)[0]],
        "new_len_fill": int(new_len_f),
        "index_map": [int(x) for x in im], "new_sent_off": [int(x) for x in nso], "new_sent_id": [int(x) for x in nsid],
        "decode_out_bits_head0_first8": [int(x) for x in out_bits[0, :8]],
        "token_redundancy_first48_rows": r(red_tok),
    }


if __name__ == "__main__":
    with open(os.path.join(HERE, "oracle_tiny_slab.json"), "w") as f:
        json.dump(compute(), f, separators=(",", ":"))
        f.write("\n")
    print("written")
