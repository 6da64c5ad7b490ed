"""The decode loop of the method on the GPU, step by step against the CPU oracle (Algorithm 2 driven
synthetically: random keys, values and queries stand in for the model; delimiters arrive at seeded sentence
ends).  Every step appends a token (K/V row, range list, observation window), runs decode attention with the
steering add on delimiter steps, and every `interval` steps evicts down to the budget.  The oracle mirrors the
state on the host with its own functions.  After every step the attention output and the steered hidden state
are compared; after every eviction the whole cache (rows, lengths, range tables) is compared bit for bit.  The
eviction follows the usual contract: the GPU's keep flags equal the oracle's selection rule applied to the GPU's
scores, the GPU's scores are within rtol 1e-3 of the oracle's, and the host state then follows those flags.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2512_07993_b200 import workloads as W

pytestmark = pytest.mark.gpu

SIGMA, TAU, EPS = float(np.float32(0.1)), float(np.float32(0.95)), float(np.float32(1e-6))


def close(name, got, ref, rtol=1e-3, atol=0.0):
    got = np.asarray(got, np.float64); ref = np.asarray(ref, np.float64)
    err = np.abs(got - ref) - (atol + rtol * np.abs(ref))
    assert (err <= 0).all(), f"{name}: worst excess {err.max():.3e} at {int(err.argmax())}"


@pytest.mark.parametrize("fill,fused", [(False, False), (True, False), (False, True), (True, True)])
def test_decode_loop_with_periodic_eviction(fill, fused):
    """Small shape, every slab mirrored, every step checked; with the two launches per step (append_step, then
    decode attention) and with the single fused launch (decode_step)."""
    cfg = W.config(0, cap_extra=48, budget=200, ctx_lo=300, ctx_hi=420, seed=91)
    run_loop(cfg, steps=150, interval=32, fill=fill, sampled=None, decode_every=1, fused=fused)


def test_decode_loop_llama8b_shape_first_two_evictions():
    """The decode-loop workload's shape (10 sequences, 8 KV heads x 4, 8192 cached tokens, budget 2048, eviction
    every 128 steps, 32-query window ring, 256 spare rows per slab) through its first two evictions; three
    slabs are mirrored by the oracle, decode attention is checked on them every 16th step and after each
    eviction, invariants on every slab."""
    run_loop(W.config(4), steps=260, interval=128, fill=False, sampled=[(0, 0), (4, 5), (9, 7)], decode_every=16)


def test_decode_loop_llama8b_shape_fused_step():
    """The same workload shape with the fused step launch, through the first eviction."""
    run_loop(W.config(4), steps=140, interval=128, fill=False, sampled=[(1, 2), (8, 0)], decode_every=16, fused=True)


def run_loop(cfg, steps, interval, fill, sampled, decode_every, fused=False):
    from paper_2512_07993_b200 import build, binding as B
    build.build()
    L = W.make_layer(cfg)
    ms = int(L["max_sent"]) + steps                       # room for the sentences that will be appended
    for key, fillv in (("sent_off", None), ("sent_id", -1)):
        old = L[key]
        new = np.zeros(old.shape[:2] + (ms + (1 if key == "sent_off" else 0),), np.int32)
        new[..., :old.shape[2]] = old
        new[..., old.shape[2]:] = old[..., -1:] if key == "sent_off" else -1
        L[key] = new
    L["max_sent"] = ms
    D = B.DeviceLayer(L)
    tok_keep = torch.zeros(D.K.shape[0], dtype=torch.uint8, device="cuda")
    kv_len_other = torch.full_like(D.kv_len, -5)
    g, Hk, Hq, bt = cfg.group, cfg.n_kv_heads, cfg.n_q_heads, cfg.batch
    slabs = sampled if sampled is not None else [(b, h) for b in range(bt) for h in range(Hk)]
    r = np.random.Generator(np.random.Philox(2024))
    # host mirror
    Kh, Vh = W.bf16_bits(L["K"]).copy(), W.bf16_bits(L["V"]).copy()
    kv = L["kv_len"].copy()
    offs = {(b, h): L["sent_off"][b, h, :L["n_sent"][b, h] + 1].copy() for (b, h) in slabs}
    ids = {(b, h): L["sent_id"][b, h, :L["n_sent"][b, h]].copy() for (b, h) in slabs}
    qwin = W.bf16_bits(L["q_win"]).copy()
    hidden = W.bf16_bits(L["hidden"]).copy()
    steer_bits = W.bf16_bits(L["steer_vec"])
    next_gen = np.array([int(L["n_sent"][b, 0]) for b in range(bt)], np.int32)
    new_sent = np.zeros(bt, np.uint8)                      # the cached context ends inside an open sentence
    draw_len = lambda: r.integers(max(2, cfg.sent_lo // 2), cfg.sent_hi // 2 + 1, size=bt)
    left = draw_len()                                      # tokens until each sequence's next delimiter
    evictions = 0
    for t in range(steps):
        k_new = W.to_bf16(r.standard_normal((bt, Hk, 128), dtype=np.float32))
        v_new = W.to_bf16(r.standard_normal((bt, Hk, 128), dtype=np.float32))
        q = W.to_bf16(r.standard_normal((bt, Hq, 128), dtype=np.float32))
        left -= 1
        delim = (left == 0).astype(np.uint8)
        left = np.where(left == 0, draw_len(), left)
        slot = t % cfg.window
        gen_id = next_gen.copy()
        # ---- GPU step
        D.flag.copy_(torch.as_tensor(delim)); D.q.copy_(q)
        if fused:
            B.skipkv_decode_step(D.shape, D.q, k_new.cuda(), v_new.cuda(), D.K, D.V, D.kv_len, kv_len_other, D.sent_off,
                                 D.sent_id, D.n_sent, torch.as_tensor(new_sent).cuda(), torch.as_tensor(gen_id).cuda(),
                                 D.q_win, slot, D.out, D.hidden, D.steer_vec, D.alpha, D.flag, D.ws)
            D.kv_len, kv_len_other = kv_len_other, D.kv_len        # the new lengths are the current ones
        else:
            B.skipkv_append_step(D.shape, D.K, D.V, k_new.cuda(), v_new.cuda(), D.kv_len, D.sent_off, D.sent_id,
                                 D.n_sent, torch.as_tensor(new_sent).cuda(), torch.as_tensor(gen_id).cuda(), D.q_win,
                                 D.q, slot, D.ws)
            D.decode_attn(steer=True)
        # ---- host mirror
        kb, vb, qb = W.bf16_bits(k_new), W.bf16_bits(v_new), W.bf16_bits(q)
        for (b, h) in slabs:
            row = W.slab_rows(L, b, h).start + int(kv[b, h])
            Kh[row], Vh[row] = kb[b, h], vb[b, h]
            offs[(b, h)], ids[(b, h)] = oracle.append_token(offs[(b, h)], ids[(b, h)], bool(new_sent[b]), gen_id[b])
        kv += 1
        qwin[:, :, slot] = qb
        next_gen += new_sent
        hidden = oracle.steer(hidden, steer_bits, L["alpha"], delim)
        torch.cuda.synchronize()
        assert D.status() == 0
        assert np.array_equal(D.kv_len.cpu().numpy(), kv)
        if t % decode_every == 0 or t % interval == 0:      # the step after an eviction is always checked
            out = W.bf16_bits(D.out.cpu())
            for (b, h) in slabs:
                rows = W.slab_rows(L, b, h)
                n = int(kv[b, h])
                _, o64 = oracle.decode_attn(qb[b, h * g:(h + 1) * g], Kh[rows][:n], Vh[rows][:n], n)
                got = W.bits_to_bf16(out[b, h * g:(h + 1) * g]).float().numpy().astype(np.float64)
                assert (np.abs(got - o64) / np.abs(o64).max(axis=-1, keepdims=True)).max() <= 2e-2, f"step {t} slab ({b},{h})"
        assert np.array_equal(W.bf16_bits(D.hidden.cpu()), hidden), f"hidden at step {t}"
        new_sent = delim.copy()                            # the token after a delimiter starts a sentence
        if t % 37 == 5:                                    # range tables, now and then
            so, sid, ns = D.sent_off.cpu().numpy(), D.sent_id.cpu().numpy(), D.n_sent.cpu().numpy()
            for (b, h), off in offs.items():
                S = len(ids[(b, h)])
                assert ns[b, h] == S and np.array_equal(so[b, h, :S + 1], off) and (so[b, h, S + 1:] == off[-1]).all()
                assert np.array_equal(sid[b, h, :S], ids[(b, h)])
            assert np.array_equal(W.bf16_bits(D.q_win.cpu()), qwin)
        # ---- eviction
        if (t + 1) % interval == 0:
            evictions += 1
            D.score()
            if fill:
                B.skipkv_select_fill(D.shape, D.params, D.sent_score, D.tok_imp, D.sent_off, D.n_sent, D.keep, tok_keep,
                                     D.kept_idx, D.n_kept, D.new_len, D.ws)
            else:
                D.select()
            torch.cuda.synchronize()
            sc, tok = D.sent_score.cpu().numpy(), D.tok_imp.cpu().numpy()
            keep, tk = D.keep.cpu().numpy(), tok_keep.cpu().numpy()
            if fill:
                B.skipkv_compact_fill(D.shape, D.K, D.V, D.keep, tok_keep, D.sent_off, D.sent_id, D.n_sent, D.kv_len,
                                      D.index_map, D.ws)
            else:
                D.compact()
            torch.cuda.synchronize()
            assert D.status() == 0
            Kg, Vg = W.bf16_bits(D.K.cpu()), W.bf16_bits(D.V.cpu())
            so, sid, ns, kvg = (x.cpu().numpy() for x in (D.sent_off, D.sent_id, D.n_sent, D.kv_len))
            assert (kvg <= cfg.budget).all()
            assert np.array_equal(D.new_len.cpu().numpy(), kvg)
            for b in range(bt):
                for h in range(Hk):
                    if (b, h) not in offs:
                        assert kvg[b, h] <= cfg.budget and so[b, h, ns[b, h]] == kvg[b, h]
                        kv[b, h] = kvg[b, h]
                        continue
                    rows = W.slab_rows(L, b, h)
                    n, off = int(kv[b, h]), offs[(b, h)]
                    S = len(off) - 1
                    o_tok = oracle.token_importance(Kh[rows][:n], qwin[b, h * g:(h + 1) * g])
                    o_imp, vbar = oracle.pool(Kh[rows][:n], off, o_tok, EPS)
                    _, o_red, o_lam = oracle.gram_terms(vbar, TAU)
                    close(f"score step {t} ({b},{h})", sc[b, h, :S], oracle.final_score(o_imp, o_red, o_lam, SIGMA),
                          rtol=1e-3, atol=1e-6)
                    if fill:
                        k_ref, t_ref, nl = oracle.select_fill(sc[b, h, :S], off, tok[rows][:n], cfg.budget, cfg.window)
                        assert nl == min(n, cfg.budget)
                    else:
                        k_ref, _, nl = oracle.select(sc[b, h, :S], off, cfg.budget, cfg.window)
                        t_ref = np.repeat(k_ref, np.diff(off))
                    assert np.array_equal(keep[b, h, :S], k_ref), f"keep at step {t} ({b},{h})"
                    Ko, Vo, _, nso, nsid = oracle.compact_tokens(Kh[rows][:n], Vh[rows][:n], t_ref, off, ids[(b, h)])
                    m = Ko.shape[0]
                    assert m == nl == int(kvg[b, h])
                    assert np.array_equal(Kg[rows][:m], Ko) and np.array_equal(Vg[rows][:m], Vo)
                    assert ns[b, h] == len(nsid) and np.array_equal(so[b, h, :len(nso)], nso)
                    assert np.array_equal(sid[b, h, :len(nsid)], nsid)
                    Kh[rows.start:rows.start + m] = Ko; Vh[rows.start:rows.start + m] = Vo
                    kv[b, h] = m; offs[(b, h)] = nso; ids[(b, h)] = nsid
    assert evictions == steps // interval and (kv <= cfg.budget + interval).all()


def test_append_step_full_slab_and_full_range_list():
    from paper_2512_07993_b200 import build, binding as B
    build.build()
    cfg = W.config(0, cap_extra=1)
    L = W.make_layer(cfg)                                  # range tables exactly as long as the longest sequence needs
    D = B.DeviceLayer(L)
    bt, Hk = cfg.batch, cfg.n_kv_heads
    z = torch.zeros(bt, Hk, 128, dtype=torch.bfloat16, device="cuda")
    ones = torch.ones(bt, dtype=torch.uint8, device="cuda"); gen = torch.full((bt,), 999, dtype=torch.int32, device="cuda")
    ns0, kv0 = D.n_sent.cpu().numpy().copy(), D.kv_len.cpu().numpy().copy()
    so0 = D.sent_off.cpu().numpy().copy()
    full = ns0 == D.max_sent                               # slabs whose range list has no free entry
    assert full.any() and not full.all()
    B.skipkv_append_step(D.shape, D.K, D.V, z, z, D.kv_len, D.sent_off, D.sent_id, D.n_sent, ones, gen, None, None, 0, D.ws)
    torch.cuda.synchronize()
    assert B.skipkv_status(D.ws, raise_on_error=False) == 0x4          # the full lists were reported
    ns1, so1 = D.n_sent.cpu().numpy(), D.sent_off.cpu().numpy()
    assert np.array_equal(D.kv_len.cpu().numpy(), kv0 + 1)
    assert np.array_equal(ns1, np.where(full, ns0, ns0 + 1))           # full: the token joined the last sentence
    for b in range(bt):
        for h in range(Hk):
            assert so1[b, h, ns1[b, h]] == kv0[b, h] + 1 and (so1[b, h, ns1[b, h]:] == kv0[b, h] + 1).all()
            assert np.array_equal(so1[b, h, :ns0[b, h]], so0[b, h, :ns0[b, h]])
    # the single spare row is used up: one more append leaves every slab unchanged and reports it
    B.skipkv_append_step(D.shape, D.K, D.V, z, z, D.kv_len, D.sent_off, D.sent_id, D.n_sent, ones, gen, None, None, 0, D.ws)
    torch.cuda.synchronize()
    assert B.skipkv_status(D.ws, raise_on_error=False) == 0x4
    assert np.array_equal(D.kv_len.cpu().numpy(), kv0 + 1) and np.array_equal(D.n_sent.cpu().numpy(), ns1)
    B.skipkv_workspace_init(D.shape, D.ws)


def test_decode_step_full_slab_and_full_range_list():
    """The fused launch at its limits: a range list without a free entry lets the token join the last sentence;
    a slab without a free row is attended over as it is; both are reported."""
    from paper_2512_07993_b200 import build, binding as B
    build.build()
    cfg = W.config(0, cap_extra=1)
    L = W.make_layer(cfg)
    D = B.DeviceLayer(L)
    bt, Hk = cfg.batch, cfg.n_kv_heads
    g = torch.Generator().manual_seed(8)
    k_new = torch.randn(bt, Hk, 128, generator=g).to(torch.bfloat16).cuda()
    v_new = torch.randn(bt, Hk, 128, generator=g).to(torch.bfloat16).cuda()
    ones = torch.ones(bt, dtype=torch.uint8, device="cuda"); gen = torch.full((bt,), 999, dtype=torch.int32, device="cuda")
    ns0, kv0 = D.n_sent.cpu().numpy().copy(), D.kv_len.cpu().numpy().copy()
    full = ns0 == D.max_sent
    assert full.any() and not full.all()
    kv_out = torch.full_like(D.kv_len, -3)

    def step():
        B.skipkv_decode_step(D.shape, D.q, k_new, v_new, D.K, D.V, D.kv_len, kv_out, D.sent_off, D.sent_id, D.n_sent, ones,
                             gen, None, 0, D.out, None, None, None, None, D.ws)
        torch.cuda.synchronize()

    step()
    assert B.skipkv_status(D.ws, raise_on_error=False) == 0x4
    assert np.array_equal(kv_out.cpu().numpy(), kv0 + 1)
    ns1, so1 = D.n_sent.cpu().numpy(), D.sent_off.cpu().numpy()
    assert np.array_equal(ns1, np.where(full, ns0, ns0 + 1))
    for b in range(bt):
        for h in range(Hk):
            assert (so1[b, h, ns1[b, h]:] == kv0[b, h] + 1).all()
    out1 = D.out.clone()
    # the same attention from the unfused entry point over the cache the step left behind
    D.kv_len.copy_(kv_out)
    D.decode_attn(steer=False)
    torch.cuda.synchronize()
    assert torch.equal(D.out.view(torch.int16), out1.view(torch.int16))
    # no spare row left: the step changes nothing and attends over the rows that are there
    kv_out.fill_(-3)
    step()
    assert B.skipkv_status(D.ws, raise_on_error=False) == 0x4
    assert np.array_equal(kv_out.cpu().numpy(), kv0 + 1) and np.array_equal(D.n_sent.cpu().numpy(), ns1)
    assert torch.equal(D.out.view(torch.int16), out1.view(torch.int16))
    B.skipkv_workspace_init(D.shape, D.ws)


def test_decode_step_on_an_empty_slab():
    """A slab with no cached row: the appended row is its only row, so the attention output is that value row."""
    from paper_2512_07993_b200 import build, binding as B
    build.build()
    cfg = W.config(0, cap_extra=4)
    L = W.make_layer(cfg)
    L["kv_len"][0, 1] = 0; L["n_sent"][0, 1] = 0; L["sent_off"][0, 1, :] = 0; L["sent_id"][0, 1, :] = -1
    D = B.DeviceLayer(L)
    bt, Hk, g = cfg.batch, cfg.n_kv_heads, cfg.group
    gen_ = torch.Generator().manual_seed(9)
    k_new = torch.randn(bt, Hk, 128, generator=gen_).to(torch.bfloat16); v_new = torch.randn(bt, Hk, 128, generator=gen_).to(torch.bfloat16)
    zeros = torch.zeros(bt, dtype=torch.uint8, device="cuda"); gid = torch.full((bt,), 41, dtype=torch.int32, device="cuda")
    kv_out = torch.full_like(D.kv_len, -3)
    B.skipkv_decode_step(D.shape, D.q, k_new.cuda(), v_new.cuda(), D.K, D.V, D.kv_len, kv_out, D.sent_off, D.sent_id, D.n_sent,
                         zeros, gid, None, 0, D.out, None, None, None, None, D.ws)
    torch.cuda.synchronize()
    assert D.status() == 0
    assert np.array_equal(kv_out.cpu().numpy(), L["kv_len"] + 1)
    out = D.out.cpu()
    for q in range(g, 2 * g):                                        # the heads of KV head 1 of sequence 0
        assert torch.equal(out[0, q].view(torch.int16), v_new[0, 1].view(torch.int16))
    row = W.slab_rows(L, 0, 1).start
    assert torch.equal(D.K[row].cpu().view(torch.int16), k_new[0, 1].view(torch.int16))
    assert torch.equal(D.V[row].cpu().view(torch.int16), v_new[0, 1].view(torch.int16))
    assert int(D.n_sent[0, 1]) == 1 and int(D.sent_id[0, 1, 0]) == 41
    so = D.sent_off[0, 1].cpu().numpy()
    assert so[0] == 0 and (so[1:] == 1).all()
    # the other slabs: the same bits as the two-launch path on a fresh copy
    D2 = B.DeviceLayer(L)
    B.skipkv_append_step(D2.shape, D2.K, D2.V, k_new.cuda(), v_new.cuda(), D2.kv_len, D2.sent_off, D2.sent_id, D2.n_sent, zeros,
                         gid, None, None, 0, D2.ws)
    D2.decode_attn(steer=False)
    torch.cuda.synchronize()
    assert np.array_equal(D2.kv_len.cpu().numpy(), kv_out.cpu().numpy())
    assert torch.equal(D2.sent_off, D.sent_off) and torch.equal(D2.n_sent, D.n_sent) and torch.equal(D2.sent_id, D.sent_id)
    assert torch.equal(D2.K, D.K) and torch.equal(D2.V, D.V)
    err = (D2.out.float() - D.out.float()).abs().max().item()
    assert err <= 2e-2 * D2.out.float().abs().max().item()


def test_fused_steps_back_to_back_without_synchronisation():
    """Forty decode steps enqueued with no host synchronisation in between, once as two launches per step and once
    as the fused launch (length buffers swapped every step): same cache, tables, lengths and last output."""
    from paper_2512_07993_b200 import build, binding as B
    build.build()
    cfg = W.config(0, batch=3, cap_extra=64, ctx_lo=200, ctx_hi=500, seed=97)
    L = W.make_layer(cfg)
    ms = int(L["max_sent"]) + 48
    for key in ("sent_off", "sent_id"):
        old = L[key]
        new = np.zeros(old.shape[:2] + (ms + (1 if key == "sent_off" else 0),), np.int32)
        new[..., :old.shape[2]] = old
        new[..., old.shape[2]:] = old[..., -1:] if key == "sent_off" else -1
        L[key] = new
    L["max_sent"] = ms
    bt, Hk, Hq = cfg.batch, cfg.n_kv_heads, cfg.n_q_heads
    g = torch.Generator().manual_seed(3)
    steps = 40
    ks = torch.randn(steps, bt, Hk, 128, generator=g).to(torch.bfloat16).cuda()
    vs = torch.randn(steps, bt, Hk, 128, generator=g).to(torch.bfloat16).cuda()
    qs = torch.randn(steps, bt, Hq, 128, generator=g).to(torch.bfloat16).cuda()
    starts = (torch.rand(steps, bt, generator=g) < 0.2).to(torch.uint8).cuda()
    flags = (torch.rand(steps, bt, generator=g) < 0.3).to(torch.uint8).cuda()
    gids = (torch.arange(steps, dtype=torch.int32)[:, None] + 1000 * torch.arange(bt, dtype=torch.int32)[None, :]).cuda()

    def run(fused):
        D = B.DeviceLayer(L)
        other = torch.zeros_like(D.kv_len)
        for t in range(steps):
            slot = t % cfg.window
            if fused:
                B.skipkv_decode_step(D.shape, qs[t], ks[t], vs[t], D.K, D.V, D.kv_len, other, D.sent_off, D.sent_id, D.n_sent,
                                     starts[t], gids[t], D.q_win, slot, D.out, D.hidden, D.steer_vec, D.alpha, flags[t], D.ws)
                D.kv_len, other = other, D.kv_len
            else:
                B.skipkv_append_step(D.shape, D.K, D.V, ks[t], vs[t], D.kv_len, D.sent_off, D.sent_id, D.n_sent, starts[t],
                                     gids[t], D.q_win, qs[t], slot, D.ws)
                B.skipkv_decode_attn(D.shape, qs[t], D.K, D.V, D.kv_len, D.out, D.hidden, D.steer_vec, D.alpha, flags[t], D.ws)
        torch.cuda.synchronize()
        assert D.status() == 0
        return D

    A, F = run(False), run(True)
    assert torch.equal(A.kv_len, F.kv_len) and int(A.kv_len.min()) == int(L["kv_len"].min()) + steps
    for name in ("K", "V", "sent_off", "sent_id", "n_sent", "q_win", "hidden"):
        assert torch.equal(getattr(A, name), getattr(F, name)), name
    err = (A.out.float() - F.out.float()).abs().max().item()
    assert err <= 2e-2 * A.out.float().abs().max().item()
