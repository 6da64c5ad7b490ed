"""The bounded device waits running out, without anything hanging or faulting.

Every spin inside the kernels (on a copy's completion barrier, on the hand-off counter of the in-place compaction)
gives up after a number of polls that the workspace carries (skipkv_set_wait_limit).  skipkv_wait_probe waits for an
event that never happens, so its wait always runs out: it pins the path limit -> give up -> status bit.  With the limit
at a couple of polls a copy of tens of kilobytes normally cannot land in time either, so the waits of the real kernels
run out in the ordinary course of a call: the kernels must return whatever happens, a wait that ran out must show in
the status word (a call whose waits all happened to succeed must be correct instead), and after
skipkv_workspace_init (which also restores the default limit) the same call must give the oracle's result.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2512_07993_b200 import workloads as W

pytestmark = pytest.mark.gpu

COMPACT_TIMEOUT, COPY_TIMEOUT = 0x1, 0x2


def layer(cfg):
    from paper_2512_07993_b200 import build, binding as B
    build.build()
    L = W.make_layer(cfg)
    return L, B.DeviceLayer(L), B


def test_wait_probe_reports_the_timeout_and_the_workspace_recovers():
    L, D, B = layer(W.config(0))
    B.skipkv_set_wait_limit(D.ws, 200)
    B.skipkv_wait_probe(D.ws)
    torch.cuda.synchronize()
    assert B.skipkv_status(D.ws, raise_on_error=False) == COPY_TIMEOUT
    with pytest.raises(B.SkipKVError):                      # the same through the raising form
        B.skipkv_wait_probe(D.ws); D.status()
    B.skipkv_workspace_init(D.shape, D.ws)
    D.decode_attn(steer=False)
    torch.cuda.synchronize()
    assert D.status() == 0


def test_decode_wait_runs_out_and_recovers():
    cfg = W.config(1, name="timeout-decode", batch=2, ctx_lo=6000, ctx_hi=9000, seed=41)
    L, D, B = layer(cfg)
    B.skipkv_set_wait_limit(D.ws, 2)
    D.decode_attn(steer=False)
    torch.cuda.synchronize()                                # the kernel came back
    bits = B.skipkv_status(D.ws, raise_on_error=False)
    assert bits in (0, COPY_TIMEOUT), hex(bits)
    timed_out = bits != 0
    if not timed_out:                                       # every copy landed within two polls: then the result stands
        first = D.out.clone()
    with_default = lambda: (B.skipkv_workspace_init(D.shape, D.ws), D.decode_attn(steer=False), torch.cuda.synchronize())
    with_default()
    assert D.status() == 0
    if not timed_out:
        assert torch.equal(first, D.out)
    g = cfg.group
    Kb, Vb, q = W.bf16_bits(L["K"]), W.bf16_bits(L["V"]), W.bf16_bits(L["q"])
    out = W.bf16_bits(D.out.cpu())
    for (b, h) in [(0, 0), (1, 7)]:
        rows = W.slab_rows(L, b, h)
        n = int(L["kv_len"][b, h])
        _, o64 = oracle.decode_attn(q[b, h * g:(h + 1) * g], Kb[rows][:n], Vb[rows][:n], n)
        got = W.bits_to_bf16(out[b, h * g:(h + 1) * g]).float().numpy().astype(np.float64)
        assert (np.abs(got - o64) / np.abs(o64).max(axis=-1, keepdims=True)).max() <= 2e-2


def test_compaction_wait_runs_out_and_recovers():
    """Several 256-row segments per stream, so that stores wait for the loads of the segments before them."""
    cfg = W.config(1, name="timeout-compact", batch=2, ctx_lo=6000, ctx_hi=9000, budget=3000, seed=42)
    L, D, B = layer(cfg)
    D.score(); D.select()
    torch.cuda.synchronize()
    keep = D.keep.clone()
    pristine = {k: getattr(D, k).clone() for k in ("K", "V", "sent_off", "sent_id", "n_sent", "kv_len")}
    B.skipkv_set_wait_limit(D.ws, 2)
    D.compact()
    torch.cuda.synchronize()                                # the kernels came back
    bits = B.skipkv_status(D.ws, raise_on_error=False)
    assert bits & ~(COPY_TIMEOUT | COMPACT_TIMEOUT) == 0, hex(bits)
    timed_out = bits != 0
    if not timed_out:
        first_K, first_len = D.K.clone(), D.kv_len.clone()
    # start again from the untouched cache with the default limit
    for k, v in pristine.items():
        getattr(D, k).copy_(v)
    B.skipkv_workspace_init(D.shape, D.ws)
    D.keep.copy_(keep)
    D.compact()
    torch.cuda.synchronize()
    assert D.status() == 0
    if not timed_out:
        assert torch.equal(first_len, D.kv_len) and torch.equal(first_K, D.K)
    sh = dict(batch=cfg.batch, Hq=cfg.n_q_heads, Hk=cfg.n_kv_heads, d=cfg.head_dim, alpha=cfg.window,
              max_sent=L["max_sent"], slab_off=L["slab_off"], cap=L["cap"])
    cp = oracle.compact_batch(sh, W.bf16_bits(L["K"]), W.bf16_bits(L["V"]), keep.cpu().numpy(), L["sent_off"], L["sent_id"],
                              L["n_sent"], L["kv_len"])
    assert np.array_equal(D.kv_len.cpu().numpy(), cp["kv_len"])
    Kg, Vg = W.bf16_bits(D.K.cpu()), W.bf16_bits(D.V.cpu())
    for b in range(cfg.batch):
        for h in range(cfg.n_kv_heads):
            rows = W.slab_rows(L, b, h)
            n = int(cp["kv_len"][b, h])
            assert np.array_equal(Kg[rows][:n], cp["K"][rows][:n]) and np.array_equal(Vg[rows][:n], cp["V"][rows][:n])
