"""GPU parity of the token-level redundancy term (skipkv_token_redundancy) against the CPU oracle:
every live row of every slab, rtol 1e-3 (fp32 dot products of exact bf16 products, one approximate
exponential per matrix element), plus the invariant that a slab's values sum to 1."""
import numpy as np
import pytest
import torch

import oracle
from paper_2512_07993_b200 import workloads as W

pytestmark = pytest.mark.gpu

CASES = {
    "smoke": lambda: W.config(0),
    "ragged": lambda: W.config(0, batch=3, ctx_lo=100, ctx_hi=1500, budget=256, seed=77),
    "one-tile": lambda: W.config(0, batch=2, ctx_lo=1, ctx_hi=128, seed=80),
    "steady-state": lambda: W.config(0, batch=1, ctx_lo=4224, ctx_hi=4224, sent_lo=8, sent_hi=96, seed=81),
    "spare-rows": lambda: W.config(0, batch=2, ctx_lo=700, ctx_hi=900, cap_extra=77, seed=82),
}


def run(cfg, kv_len_override=None):
    from paper_2512_07993_b200 import build, binding as B
    build.build()
    L = W.make_layer(cfg)
    if kv_len_override is not None:
        L["kv_len"] = kv_len_override(L["kv_len"].copy())
    D = B.DeviceLayer(L)
    red = torch.full((D.K.shape[0],), float("nan"), dtype=torch.float32, device="cuda")
    B.skipkv_token_redundancy(D.shape, D.params, D.K, D.kv_len, red, D.ws)
    torch.cuda.synchronize()
    assert D.status() == 0
    return L, red.cpu().numpy()


@pytest.mark.parametrize("case", list(CASES))
def test_token_redundancy_parity(case):
    cfg = CASES[case]()
    L, red = run(cfg)
    Kb = W.bf16_bits(L["K"])
    for b in range(cfg.batch):
        for h in range(cfg.n_kv_heads):
            rows = W.slab_rows(L, b, h)
            N = int(L["kv_len"][b, h])
            ref = oracle.token_redundancy(Kb[rows][:N], 1e-6)
            got = red[rows][:N].astype(np.float64)
            err = np.abs(got - ref) - 1e-3 * np.abs(ref)
            assert (err <= 0).all(), f"slab ({b},{h}): worst excess {err.max():.3e} at {int(err.argmax())} of {N}"
            if N > 1:
                assert abs(got.sum() - 1.0) < 1e-3
            assert np.isnan(red[rows][N:]).all()            # rows beyond the live ones are not written


def test_token_redundancy_empty_and_single_row_slabs():
    cfg = CASES["smoke"]()
    def override(kv):
        kv[0, 0] = 0; kv[0, 1] = 1; kv[1, 0] = 129
        return kv
    L, red = run(cfg, override)
    Kb = W.bf16_bits(L["K"])
    for b in range(cfg.batch):
        for h in range(cfg.n_kv_heads):
            rows = W.slab_rows(L, b, h)
            N = int(L["kv_len"][b, h])
            got = red[rows]
            assert np.isnan(got[N:]).all()
            if N == 1:
                assert got[0] == 0.0
            elif N > 1:
                ref = oracle.token_redundancy(Kb[rows][:N], 1e-6)
                assert (np.abs(got[:N] - ref) <= 1e-3 * np.abs(ref)).all()
