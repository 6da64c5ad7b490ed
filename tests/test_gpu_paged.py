"""GPU parity of the path over a paged cache (skipkv_score_paged, skipkv_compact_paged, skipkv_decode_attn_paged,
skipkv_decode_step_paged): the same rows scattered over a shuffled page pool must give the bits the contiguous
entry points give (which the other parity tests compare with the CPU oracle), and match the oracle directly."""
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


def paged_shape(B, D, Kp):
    """The layer's shape with the pool's row count (bounds the tiled copies); slab offsets are not used."""
    cfg = D.cfg
    return B.make_shape(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.window, cfg.d_model, D.max_sent,
                        int(D.cap.max()), D.slab_off, D.cap, int(Kp.shape[0]))


def gather_slab(pool, table, b, h, n):
    """Rows 0..n of slab (b, h) read through its block table."""
    t = torch.arange(n, device=pool.device)
    pages = table[b, h][t // PAGE].long()
    return pool[pages * PAGE + t % PAGE]


PAGED_CASES = {"smoke": dict(),
               "ragged": dict(batch=3, ctx_lo=100, ctx_hi=1500, seed=77),
               "group5": dict(n_q_heads=10, n_kv_heads=2, ctx_lo=500, ctx_hi=900, seed=78),
               "long": dict(batch=2, ctx_lo=3000, ctx_hi=6000, seed=79)}


@pytest.mark.parametrize("case", list(PAGED_CASES))
def test_paged_score_and_compact_match_contiguous(case):
    from paper_2512_07993_b200 import build, binding as B
    build.build()
    cfg = W.config(0, **PAGED_CASES[case])
    L = W.make_layer(cfg)
    D = B.DeviceLayer(L)
    Kp, Vp, table, max_pages = paged_copy(L, D, 11)
    shp = paged_shape(B, D, Kp)
    bt, Hk = cfg.batch, cfg.n_kv_heads

    # scoring: every output the same bits
    D.score()
    torch.cuda.synchronize()
    assert D.status() == 0
    ref = {k: getattr(D, k).clone() for k in ("tok_imp", "sent_imp", "sent_red", "sent_lam", "sent_score")}
    f32 = dict(dtype=torch.float32, device="cuda")
    tok_p = torch.full((bt, Hk, max_pages * PAGE), float("nan"), **f32)
    outs = {k: torch.full_like(ref[k], float("nan")) for k in ("sent_imp", "sent_red", "sent_lam", "sent_score")}
    B.skipkv_score_paged(shp, D.params, Kp, table, max_pages, D.q_win, D.kv_len, D.sent_off, D.n_sent, tok_p,
                         outs["sent_imp"], outs["sent_red"], outs["sent_lam"], outs["sent_score"], D.ws)
    torch.cuda.synchronize()
    assert D.status() == 0
    ns = L["n_sent"]
    for b in range(bt):
        for h in range(Hk):
            n, S = int(L["kv_len"][b, h]), int(ns[b, h])
            rows = W.slab_rows(L, b, h)
            assert torch.equal(tok_p[b, h, :n].view(torch.int32), ref["tok_imp"][rows.start:rows.start + n].view(torch.int32)), (b, h)
            for k in outs:
                assert torch.equal(outs[k][b, h, :S].view(torch.int32), ref[k][b, h, :S].view(torch.int32)), (k, b, h)

    # selection is layout-free; compaction: same rows, tables, lengths and index map
    D.select()
    tabs = {k: getattr(D, k).clone() for k in ("sent_off", "sent_id", "n_sent", "kv_len")}
    D.compact()
    torch.cuda.synchronize()
    assert D.status() == 0
    im_p = torch.full((bt, Hk, max_pages * PAGE), -7, dtype=torch.int32, device="cuda")
    B.skipkv_compact_paged(shp, Kp, Vp, table, max_pages, D.keep, tabs["sent_off"], tabs["sent_id"], tabs["n_sent"],
                           tabs["kv_len"], im_p, D.ws)
    torch.cuda.synchronize()
    assert D.status() == 0
    for k in tabs:
        assert torch.equal(tabs[k], getattr(D, k)), k
    assert int((tabs["kv_len"].cpu() < torch.as_tensor(L["kv_len"])).sum()) > 0       # something was evicted
    for b in range(bt):
        for h in range(Hk):
            n_old, n_new = int(L["kv_len"][b, h]), int(tabs["kv_len"][b, h])
            rows = W.slab_rows(L, b, h)
            for pool, flat in ((Kp, D.K), (Vp, D.V)):
                got = gather_slab(pool, table, b, h, n_new)
                assert torch.equal(got.view(torch.int16), flat[rows.start:rows.start + n_new].view(torch.int16)), (b, h)
            assert torch.equal(im_p[b, h, :n_new], D.index_map[rows.start:rows.start + n_new]), (b, h)
            assert int((im_p[b, h, n_new:] != -7).sum()) == 0, (b, h)            # entries behind the new length untouched

    # and the attention over the compacted pages
    D.decode_attn(steer=False)
    torch.cuda.synchronize()
    want = D.out.clone()
    D.out.zero_()
    B.skipkv_decode_attn_paged(shp, D.q, Kp, Vp, table, max_pages, tabs["kv_len"], D.out, None, None, None, None, D.ws)
    torch.cuda.synchronize()
    assert D.status() == 0
    assert torch.equal(D.out.view(torch.int16), want.view(torch.int16))


def test_paged_decode_step_matches_contiguous():
    """Three fused decode steps (append + range list + window + attention) on the paged cache and on the
    contiguous one: same outputs, tables and rows; lengths chosen so that appends cross into a fresh page."""
    from paper_2512_07993_b200 import build, binding as B
    build.build()
    cfg = W.config(0, batch=3, ctx_lo=254, ctx_hi=258, cap_extra=8, seed=91)
    L = W.make_layer(cfg)
    ms = int(L["max_sent"]) + 4                            # room for the sentences the steps open
    for key in ("sent_off", "sent_id"):
        old = L[key]
        new = np.zeros(old.shape[:2] + (ms + (1 if key == "sent_off" else 0),), np.int32)
        new[..., :old.shape[2]] = old
        new[..., old.shape[2]:] = old[..., -1:] if key == "sent_off" else -1
        L[key] = new
    L["max_sent"] = ms
    D = B.DeviceLayer(L)
    Kp, Vp, table, max_pages = paged_copy(L, D, 13)
    shp = paged_shape(B, D, Kp)
    P = B.DeviceLayer(L)                       # tables, window and buffers of the paged run
    bt, Hk = cfg.batch, cfg.n_kv_heads
    gen_ = torch.Generator().manual_seed(17)
    for step in range(3):
        k_new = torch.randn(bt, Hk, 128, generator=gen_).to(torch.bfloat16).cuda()
        v_new = torch.randn(bt, Hk, 128, generator=gen_).to(torch.bfloat16).cuda()
        q = torch.randn(bt, cfg.n_q_heads, 128, generator=gen_).to(torch.bfloat16).cuda()
        new_sent = torch.as_tensor([(step + b) % 2 for b in range(bt)], dtype=torch.uint8).cuda()
        gid = torch.full((bt,), 50 + step, dtype=torch.int32, device="cuda")
        slot = step % cfg.window
        kv_c, kv_p = torch.full_like(D.kv_len, -3), torch.full_like(D.kv_len, -3)
        B.skipkv_decode_step(D.shape, q, k_new, v_new, D.K, D.V, D.kv_len, kv_c, D.sent_off, D.sent_id, D.n_sent,
                             new_sent, gid, D.q_win, slot, D.out, D.hidden, D.steer_vec, D.alpha, D.flag, D.ws)
        B.skipkv_decode_step_paged(shp, q, k_new, v_new, Kp, Vp, table, max_pages, P.kv_len, kv_p, P.sent_off,
                                   P.sent_id, P.n_sent, new_sent, gid, P.q_win, slot, P.out, P.hidden, P.steer_vec,
                                   P.alpha, P.flag, P.ws)
        torch.cuda.synchronize()
        assert D.status() == 0 and P.status() == 0
        assert torch.equal(kv_c, kv_p) and torch.equal(kv_c, D.kv_len + 1)
        D.kv_len, P.kv_len = kv_c, kv_p
        for k in ("sent_off", "sent_id", "n_sent", "q_win"):
            assert torch.equal(getattr(D, k), getattr(P, k)), (step, k)
        assert torch.equal(D.out.view(torch.int16), P.out.view(torch.int16)), step
        assert torch.equal(D.hidden.view(torch.int16), P.hidden.view(torch.int16)), step
    for b in range(bt):
        for h in range(Hk):
            n = int(D.kv_len[b, h]); rows = W.slab_rows(L, b, h)
            assert torch.equal(gather_slab(Kp, table, b, h, n).view(torch.int16), D.K[rows.start:rows.start + n].view(torch.int16))
            assert torch.equal(gather_slab(Vp, table, b, h, n).view(torch.int16), D.V[rows.start:rows.start + n].view(torch.int16))


def test_paged_score_and_compact_reject_bad_arguments():
    from paper_2512_07993_b200 import build, binding as B
    build.build()
    D = B.DeviceLayer(W.make_layer(W.config(0)))
    args = (D.q_win, D.kv_len, D.sent_off, D.n_sent, None, D.sent_imp, D.sent_red, D.sent_lam, D.sent_score, D.ws)
    with pytest.raises(B.SkipKVError) as e:
        B.skipkv_score_paged(D.shape, D.params, D.K, None, 4, *args)
    assert e.value.code == -1
    too_many = (int(D.cap.max()) + 127) // PAGE + 1                  # beyond what the workspace was sized for
    with pytest.raises(B.SkipKVError) as e:
        B.skipkv_score_paged(D.shape, D.params, D.K, D.kv_len, too_many, *args)
    assert e.value.code == -1
    with pytest.raises(B.SkipKVError) as e:
        B.skipkv_compact_paged(D.shape, D.K, D.V, None, 4, D.keep, D.sent_off, D.sent_id, D.n_sent, D.kv_len, None, D.ws)
    assert e.value.code == -1
