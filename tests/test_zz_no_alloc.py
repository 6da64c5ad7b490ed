"""skipkv_decode_attn_static: decode attention for callers that cannot allocate device memory.

A serving process that gave all free HBM to its KV-cache pool, or an extension that must not
call cudaMalloc (the call synchronises the device), has no workspace to hand to
skipkv_decode_attn.  The static variant keeps its scratch in a fixed array inside the library.
Here it is called through the C ABI twice in a row (the array keeps the previous call's
contents, so the second call checks that what must start at zero is cleared) and compared with
the workspace-based entry point on the same inputs, within the decode-attention tolerance of the
parity tests, and, on two slabs, directly with the CPU oracle's attention.  This file is collected last
so that a failure here cannot hide another test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2512_07993_b200 import workloads as W

pytestmark = pytest.mark.gpu

TOL = 2e-2          # of the row's largest |output|, as in the decode-attention parity tests


def rel_err(a, b):
    a = a.float().cpu().numpy().astype(np.float64)
    b = b.float().cpu().numpy().astype(np.float64)
    scale = np.abs(b).max(axis=-1, keepdims=True)
    scale[scale == 0] = 1.0
    return float((np.abs(a - b) / scale).max())


def test_static_scratch_decode_matches_workspace_decode_twice():
    from paper_2512_07993_b200 import build, binding as B
    build.build()
    B.lib()
    # long enough that slabs are split over several CTAs: partial records and counters are used
    cfg = W.config(1, name="no-alloc", batch=2, ctx_lo=5000, ctx_hi=9000, seed=31)
    L = W.make_layer(cfg)
    D = B.DeviceLayer(L)
    D.decode_attn(steer=False)
    torch.cuda.synchronize()
    assert D.status() == 0
    want = D.out.clone()
    assert want.float().abs().max().item() > 0

    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rng = np.random.default_rng(9)
    for call in range(2):
        if call == 1:
            # other lengths on the second call: different slabs are split, different counters used
            kv_len = rng.integers(1, L["kv_len"] + 1).astype(np.int32)
            D.kv_len.copy_(torch.from_numpy(kv_len))
            D.decode_attn(steer=False)
            torch.cuda.synchronize()
            want = D.out.clone()
        got = torch.full_like(D.out, float("nan"))
        hid = D.hidden.clone()
        B.skipkv_decode_attn_static(D.shape, D.q, D.K, D.V, D.kv_len, got, hid, D.steer_vec, D.alpha, D.flag,
                                    status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert torch.isfinite(got.float()).all()
        assert rel_err(got, want) <= TOL, call
        # and against the oracle itself, on two slabs with the lengths of this call
        g = cfg.group
        Kb, Vb, qb = W.bf16_bits(L["K"]), W.bf16_bits(L["V"]), W.bf16_bits(L["q"])
        lens = D.kv_len.cpu().numpy()
        for (b, h) in [(0, 3), (1, 6)]:
            rows = W.slab_rows(L, b, h)
            n = int(lens[b, h])
            _, o64 = oracle.decode_attn(qb[b, h * g:(h + 1) * g], Kb[rows][:n], Vb[rows][:n], n)
            mine = got[b, h * g:(h + 1) * g].float().cpu().numpy().astype(np.float64)
            assert (np.abs(mine - o64) / np.abs(o64).max(axis=-1, keepdims=True)).max() <= TOL, (call, b, h)
        # the fused steering add is the same bit-exact operation as in the workspace variant
        ref_h = D.hidden.clone()
        B.skipkv_steer(cfg.batch, cfg.d_model, ref_h, D.steer_vec, D.alpha, D.flag)
        torch.cuda.synchronize()
        assert torch.equal(hid, ref_h)


def test_static_scratch_decode_rejects_sizes_beyond_its_array():
    from paper_2512_07993_b200 import build, binding as B
    build.build()
    L = W.make_layer(W.config(0))
    D = B.DeviceLayer(L)
    big = B.make_shape(40, 32, 8, 128, 8, 256, D.max_sent, 512, D.slab_off, D.cap)      # 320 slabs > 256
    with pytest.raises(B.SkipKVError) as e:
        B.skipkv_decode_attn_static(big, D.q, D.K, D.V, D.kv_len, D.out, None, None, None, None)
    assert e.value.code == -2
    assert "SKIPKV_STATIC_MAX_SLABS" in str(e.value)
