"""Repeated calls on one input: the scoring call must return the same bits every time (its only unordered
accumulation adds at most two terms to a zero, which commutes), the token-level redundancy the same values to
rounding (its row and column sums are accumulated with floating-point reductions in no fixed order).  A race on a
shared buffer inside the Gram kernels would show here as a difference between runs."""
import numpy as np
import pytest
import torch

from paper_2512_07993_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_score_is_bit_identical_across_calls():
    from paper_2512_07993_b200 import build, binding as B
    build.build()
    # > 512 sentences per slab: a warpgroup of the Gram kernels handles several blocks per item
    cfg = W.config(0, batch=2, n_q_heads=8, n_kv_heads=2, ctx_lo=20000, ctx_hi=26000, sent_lo=8, sent_hi=64,
                   budget=2048, window=32, seed=123)
    L = W.make_layer(cfg)
    assert int(L["n_sent"].max()) > 512
    D = B.DeviceLayer(L)
    runs = []
    for _ in range(4):
        for t in (D.tok_imp, D.sent_imp, D.sent_red, D.sent_lam, D.sent_score):
            t.fill_(float("nan"))
        D.score()
        torch.cuda.synchronize()
        assert D.status() == 0
        runs.append([t.clone() for t in (D.tok_imp, D.sent_imp, D.sent_red, D.sent_lam, D.sent_score)])
    live = torch.zeros(D.K.shape[0], dtype=torch.bool)
    for b in range(cfg.batch):
        for h in range(cfg.n_kv_heads):
            rows = W.slab_rows(L, b, h)
            live[rows.start:rows.start + int(L["kv_len"][b, h])] = True
    live = live.cuda()
    for r in runs[1:]:
        assert torch.equal(r[0][live].view(torch.int32), runs[0][0][live].view(torch.int32))
        for k in range(1, 5):
            for b in range(cfg.batch):
                for h in range(cfg.n_kv_heads):
                    S = int(L["n_sent"][b, h])
                    assert torch.equal(r[k][b, h, :S].view(torch.int32), runs[0][k][b, h, :S].view(torch.int32)), (k, b, h)


def test_token_redundancy_agrees_across_calls():
    from paper_2512_07993_b200 import build, binding as B
    build.build()
    cfg = W.config(0, batch=2, ctx_lo=3000, ctx_hi=4224, sent_lo=8, sent_hi=96, seed=124)
    L = W.make_layer(cfg)
    D = B.DeviceLayer(L)
    outs = []
    for _ in range(4):
        red = torch.full((D.K.shape[0],), float("nan"), dtype=torch.float32, device="cuda")
        B.skipkv_token_redundancy(D.shape, D.params, D.K, D.kv_len, red, D.ws)
        torch.cuda.synchronize()
        assert D.status() == 0
        outs.append(red.cpu().numpy())
    for b in range(cfg.batch):
        for h in range(cfg.n_kv_heads):
            rows = W.slab_rows(L, b, h)
            n = int(L["kv_len"][b, h])
            ref = outs[0][rows.start:rows.start + n]
            assert np.isfinite(ref).all() and (ref > 0).all()
            for o in outs[1:]:
                assert np.allclose(o[rows.start:rows.start + n], ref, rtol=1e-5, atol=0.0), (b, h)
