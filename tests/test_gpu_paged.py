"""GPU parity of decode attention over a paged cache (skipkv_decode_attn_paged): the same rows scattered over
a shuffled page pool must give the bits the contiguous entry point gives, and match the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2512_07993_b200 import workloads as W

pytestmark = pytest.mark.gpu

PAGE = 128


def paged_copy(L, D, seed):
    """Scatter every slab's rows over a shuffled pool; unused rows and pages hold NaN bit patterns."""
    cfg = L["cfg"]
    bt, Hk = cfg.batch, cfg.n_kv_heads
    pages_of = lambda b: (int(L["cap"][b]) + PAGE - 1) // PAGE
    max_pages = max(pages_of(b) for b in range(bt))
    n_used = sum(pages_of(b) for b in range(bt)) * Hk
    n_pool = n_used + 7
    r = np.random.Generator(np.random.Philox(seed))
    ids = r.permutation(n_pool)[:n_used]
    nan = torch.full((n_pool * PAGE, 128), float("nan"), dtype=torch.bfloat16)
    Kp, Vp = nan.clone(), nan.clone()
    table = np.full((bt, Hk, max_pages), -1, np.int32)
    k = 0
    for b in range(bt):
        for h in range(Hk):
            rows = W.slab_rows(L, b, h)
            n = int(L["kv_len"][b, h])
            for j in range(pages_of(b)):
                pg = int(ids[k]); k += 1
                table[b, h, j] = pg
                lo, hi = j * PAGE, min((j + 1) * PAGE, n)
                if hi > lo:
                    Kp[pg * PAGE:pg * PAGE + hi - lo] = L["K"][rows.start + lo:rows.start + hi]
                    Vp[pg * PAGE:pg * PAGE + hi - lo] = L["V"][rows.start + lo:rows.start + hi]
    return Kp.cuda(), Vp.cuda(), torch.as_tensor(table).cuda(), max_pages


@pytest.mark.parametrize("case", ["smoke", "ragged", "group5", "one-row"])
def test_paged_decode_matches_contiguous_and_oracle(case):
    from paper_2512_07993_b200 import build, binding as B
    build.build()
    cfg = {"smoke": W.config(0),
           "ragged": W.config(0, batch=3, ctx_lo=100, ctx_hi=1500, seed=77),
           "group5": W.config(0, n_q_heads=10, n_kv_heads=2, ctx_lo=500, ctx_hi=900, seed=78),
           "one-row": W.config(0, batch=2, ctx_lo=1, ctx_hi=1, seed=83)}[case]
    L = W.make_layer(cfg)
    D = B.DeviceLayer(L)
    hidden0 = D.hidden.clone()
    D.decode_attn(steer=True)
    torch.cuda.synchronize()
    out_ref, hidden_ref = D.out.clone(), D.hidden.clone()
    Kp, Vp, table, max_pages = paged_copy(L, D, 5)
    D.hidden.copy_(hidden0); D.out.zero_()
    B.skipkv_decode_attn_paged(D.shape, D.q, Kp, Vp, table, max_pages, D.kv_len, D.out, D.hidden, D.steer_vec, D.alpha,
                               D.flag, D.ws)
    torch.cuda.synchronize()
    assert D.status() == 0
    assert torch.equal(D.out.view(torch.int16), out_ref.view(torch.int16))
    assert torch.equal(D.hidden.view(torch.int16), hidden_ref.view(torch.int16))
    sh = dict(batch=cfg.batch, Hq=cfg.n_q_heads, Hk=cfg.n_kv_heads, d=cfg.head_dim, alpha=cfg.window,
              max_sent=L["max_sent"], slab_off=L["slab_off"], cap=L["cap"])
    _, o64 = oracle.decode_attn_batch(sh, W.bf16_bits(L["q"]), W.bf16_bits(L["K"]), W.bf16_bits(L["V"]), L["kv_len"])
    got = D.out.float().cpu().numpy().astype(np.float64)
    scale = np.abs(o64).max(axis=-1, keepdims=True); scale[scale == 0] = 1.0
    assert (np.abs(got - o64) / scale).max() <= 2e-2


def test_paged_decode_rejects_missing_table():
    from paper_2512_07993_b200 import build, binding as B
    build.build()
    D = B.DeviceLayer(W.make_layer(W.config(0)))
    with pytest.raises(B.SkipKVError) as e:
        B.skipkv_decode_attn_paged(D.shape, D.q, D.K, D.V, None, 4, D.kv_len, D.out, None, None, None, None, D.ws)
    assert e.value.code == -1
    with pytest.raises(B.SkipKVError) as e:
        B.skipkv_decode_attn_paged(D.shape, D.q, D.K, D.V, D.kv_len, 0, D.kv_len, D.out, None, None, None, None, D.ws)
    assert e.value.code == -1
