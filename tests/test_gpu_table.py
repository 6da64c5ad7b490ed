"""GPU parity of the generation-space lookup table (skipkv_table_step) and of the score call that
reads it (skipkv_score_table) against the CPU oracle.

The table is built on the GPU one decode step at a time and compared with the oracle's one-shot
definition over the same hidden states; the penalty looked up through the cache-space sentence ids
must be the table entry bit for bit, and the final score within the fp32 tolerance of the other
score terms (rtol 1e-3).  A similarity within 1e-5 of the threshold may be flagged on one side only
(both sides take that decision in their own precision: fp32 dot products here, fp64 in the oracle);
such entries are counted and must be rare.
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


class DeviceTable:
    """Device state of skipkv_table_step for `batch` sequences (allocation and marshalling only)."""

    def __init__(self, batch, d_model, max_gen_sent):
        dev = torch.device("cuda")
        self.batch, self.d_model, self.max_gen_sent = batch, d_model, max_gen_sent
        self.acc = torch.zeros(batch, d_model, dtype=torch.float32, device=dev)
        self.acc_count = torch.zeros(batch, dtype=torch.int32, device=dev)
        self.emb = torch.full((batch, max_gen_sent, d_model), float("nan"), dtype=torch.float32, device=dev)
        self.n_gen_sent = torch.zeros(batch, dtype=torch.int32, device=dev)
        self.closed = torch.full((batch,), -7, dtype=torch.int32, device=dev)
        self.T = torch.full((batch, max_gen_sent), float("nan"), dtype=torch.float32, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)

    def step(self, hidden_last, flag, tau=TAU):
        from paper_2512_07993_b200 import binding as B
        B.skipkv_table_step(self.batch, self.d_model, self.max_gen_sent, hidden_last, flag, self.acc, self.acc_count,
                            self.emb, self.n_gen_sent, self.closed, self.T, tau, EPS, self.status)


def run_generation(cfg, steps, d_model, max_gen_sent, check_closed_every=37):
    from paper_2512_07993_b200 import build
    build.build()
    g = W.make_generation(cfg, steps, d_model)
    H = g["H"].cuda()
    flags = torch.as_tensor(g["flag"]).cuda()
    D = DeviceTable(cfg.batch, d_model, max_gen_sent)
    n_closed = np.zeros(cfg.batch, np.int64)
    for t in range(steps):
        D.step(H[:, t].contiguous(), flags[t].contiguous())
        n_closed += g["flag"][t]
        if t % check_closed_every == 0 or t == steps - 1:
            want = np.where(g["flag"][t] == 1, np.minimum(n_closed - 1, max_gen_sent), -1)
            want = np.where(want >= max_gen_sent, -1, want)
            assert np.array_equal(D.closed.cpu().numpy(), want), f"closed[] at step {t}"
    torch.cuda.synchronize()
    return g, D


@pytest.mark.parametrize("d_model,steps", [(512, 600), (4096, 700), (200, 150)])
def test_table_step_matches_definition(d_model, steps):
    cfg = W.config(0, batch=3)
    g, D = run_generation(cfg, steps, d_model, 64)
    assert int(D.status.item()) == 0
    n = D.n_gen_sent.cpu().numpy()
    T = D.T.cpu().numpy(); emb = D.emb.cpu().numpy()
    cnt = D.acc_count.cpu().numpy(); acc = D.acc.cpu().numpy()
    excused = 0
    for b in range(cfg.batch):
        off = g["gen_off"][b]
        S = len(off) - 1
        assert S > 32 or steps < 600                      # more than one block of earlier sentences
        assert n[b] == S
        Hb = W.bf16_bits(g["H"][b])
        T_ref, G = oracle.lookup_table(Hb, off, TAU, EPS)
        _, vbar = oracle.pool(Hb, off, np.zeros(Hb.shape[0]), EPS)
        close(f"emb[{b}]", emb[b, :S], vbar, rtol=1e-5, atol=1e-7)
        later_max = np.array([G[i, i + 1:].max() if i + 1 < S else -1.0 for i in range(S)])
        sure = np.abs(later_max - TAU) > 1e-5
        excused += int((~sure).sum())
        assert np.array_equal(T[b, :S][sure] > 0, T_ref[sure] > 0), f"flags differ in sequence {b}"
        close(f"T[{b}]", T[b, :S][sure], T_ref[sure], rtol=0.0, atol=1e-5)
        assert ((T_ref > 0).sum() >= 2 or steps < 600) and T[b, S - 1] == 0.0
        # the open sentence: running sum and count of the tokens after the last closed one
        open_rows = W.bits_to_bf16(Hb[off[-1]:]).double().numpy()
        assert cnt[b] == open_rows.shape[0]
        close(f"acc[{b}]", acc[b], open_rows.sum(axis=0) if len(open_rows) else np.zeros(d_model), rtol=1e-5, atol=1e-5)
    assert excused <= 1


def test_table_full_drops_sentences_and_reports():
    cfg = W.config(0, batch=2)
    g, D = run_generation(cfg, 200, 256, 5)
    assert int(D.status.item()) & 0x4                     # SKIPKV_STATUS_BAD_TABLE
    assert (D.n_gen_sent.cpu().numpy() == 5).all()
    T = D.T.cpu().numpy()
    for b in range(cfg.batch):
        off = g["gen_off"][b][:6]
        T_ref, G = oracle.lookup_table(W.bf16_bits(g["H"][b]), off, TAU, EPS)
        assert np.array_equal(T[b, :5] > 0, T_ref > 0)
        close(f"T[{b}]", T[b, :5], T_ref, rtol=0.0, atol=1e-5)


def test_table_step_rejects_bad_arguments():
    from paper_2512_07993_b200 import binding as B, build
    build.build()
    D = DeviceTable(2, 256, 8)
    h = torch.zeros(2, 256, dtype=torch.bfloat16, device="cuda"); f = torch.zeros(2, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.SkipKVError) as e:
        B.skipkv_table_step(2, 252, 8, h, f, D.acc, D.acc_count, D.emb, D.n_gen_sent, D.closed, D.T, TAU, EPS)
    assert e.value.code == -2
    with pytest.raises(B.SkipKVError) as e:
        B.skipkv_table_step(2, 256, 0, h, f, D.acc, D.acc_count, D.emb, D.n_gen_sent, D.closed, D.T, TAU, EPS)
    assert e.value.code == -1
    with pytest.raises(B.SkipKVError) as e:
        B.skipkv_table_step(2, 256, 8, h, None, D.acc, D.acc_count, D.emb, D.n_gen_sent, D.closed, D.T, TAU, EPS)
    assert e.value.code == -1
    torch.cuda.synchronize()


def random_table(batch, table_len, seed):
    r = np.random.Generator(np.random.Philox(seed))
    T = np.where(r.random((batch, table_len)) < 0.3, r.uniform(TAU, 1.0, (batch, table_len)), 0.0)
    return T.astype(np.float32)


@pytest.mark.parametrize("case", ["smoke", "ragged", "group5"])
def test_score_table_parity_and_eviction(case):
    from paper_2512_07993_b200 import build, binding as B
    build.build()
    cfg = {"smoke": W.config(0),
           "ragged": W.config(0, batch=3, ctx_lo=100, ctx_hi=1500, budget=256, seed=77),
           "group5": W.config(0, n_q_heads=10, n_kv_heads=2, ctx_lo=500, ctx_hi=900, budget=200, seed=78)}[case]
    L = W.make_layer(cfg)
    ms = int(L["max_sent"])
    # cache-space sentence i came from generation-space sentence 2*i+1; a few have no entry
    L["sent_id"] = np.where(L["sent_id"] >= 0, 2 * L["sent_id"] + 1, -1).astype(np.int32)
    table_len = 2 * ms - 3                                 # the last ids fall outside the table
    L["sent_id"][:, 0, 0] = -1
    T = random_table(cfg.batch, table_len, 5)
    D = B.DeviceLayer(L)
    Td = torch.as_tensor(T).cuda()

    def score_table():
        B.skipkv_score_table(D.shape, D.params, D.K, D.q_win, D.kv_len, D.sent_off, D.sent_id, D.n_sent, Td, table_len,
                             D.tok_imp, D.sent_imp, D.sent_red, D.sent_lam, D.sent_score, D.ws)

    score_table()
    torch.cuda.synchronize()
    assert D.status() == 0
    g = cfg.group
    Kb, Qw = W.bf16_bits(L["K"]), W.bf16_bits(L["q_win"])
    imp, red, lam, sc = (x.cpu().numpy() for x in (D.sent_imp, D.sent_red, D.sent_lam, D.sent_score))
    for b in range(cfg.batch):
        for h in range(cfg.n_kv_heads):
            rows = W.slab_rows(L, b, h)
            N, S = int(L["kv_len"][b, h]), int(L["n_sent"][b, h])
            off, sid = L["sent_off"][b, h, :S + 1], L["sent_id"][b, h, :S]
            o_imp, o_red, o_lam, o_sc = oracle.score_with_table(Kb[rows][:N], Qw[b, h * g:(h + 1) * g], off, sid, T[b],
                                                                SIGMA, TAU, EPS)
            assert np.array_equal(lam[b, h, :S], o_lam.astype(np.float32)), f"lam[{b},{h}]"
            close(f"imp[{b},{h}]", imp[b, h, :S], o_imp)
            close(f"red[{b},{h}]", red[b, h, :S], o_red)
            close(f"score[{b},{h}]", sc[b, h, :S], o_sc, rtol=1e-3, atol=1e-6)
    assert (lam > 0).any() and (lam[:, 0, 0] == 0).all()

    # evict with these scores, then score again: the survivors still find their own entries
    D.select(); D.compact(); score_table()
    torch.cuda.synchronize()
    assert D.status() == 0
    keep = D.keep.cpu().numpy()
    lam2, ns2, sid2 = D.sent_lam.cpu().numpy(), D.n_sent.cpu().numpy(), D.sent_id.cpu().numpy()
    for b in range(cfg.batch):
        for h in range(cfg.n_kv_heads):
            S = int(L["n_sent"][b, h])
            k_own, _, _ = oracle.select(sc[b, h, :S], L["sent_off"][b, h, :S + 1], cfg.budget, cfg.window)
            assert np.array_equal(keep[b, h, :S], k_own)
            n2 = int(ns2[b, h])
            assert n2 == int(k_own.sum())
            assert np.array_equal(sid2[b, h, :n2], L["sent_id"][b, h, :S][k_own == 1])
            assert np.array_equal(lam2[b, h, :n2], oracle.map_table(T[b], sid2[b, h, :n2]).astype(np.float32))
            assert np.array_equal(lam2[b, h, :n2], lam[b, h, :S][k_own == 1])


def test_table_feeds_score():
    """The table kept by skipkv_table_step used directly as the penalty source of skipkv_score_table."""
    from paper_2512_07993_b200 import build, binding as B
    build.build()
    cfg = W.config(0, batch=2, ctx_lo=600, ctx_hi=600, budget=200)
    L = W.make_layer(cfg)                                  # cache sentences = the first generation-space sentences
    g, Dt = run_generation(cfg, 600, 256, int(L["max_sent"]) + 8)
    D = B.DeviceLayer(L)
    B.skipkv_score_table(D.shape, D.params, D.K, D.q_win, D.kv_len, D.sent_off, D.sent_id, D.n_sent, Dt.T,
                         Dt.max_gen_sent, None, D.sent_imp, D.sent_red, D.sent_lam, D.sent_score, D.ws)
    torch.cuda.synchronize()
    assert D.status() == 0
    lam = D.sent_lam.cpu().numpy()
    T = Dt.T.cpu().numpy(); n = Dt.n_gen_sent.cpu().numpy()
    for b in range(cfg.batch):
        T_ref, _ = oracle.lookup_table(W.bf16_bits(g["H"][b]), g["gen_off"][b], TAU, EPS)
        for h in range(cfg.n_kv_heads):
            S = int(L["n_sent"][b, h])
            sid = L["sent_id"][b, h, :S]
            inside = sid < n[b]
            assert np.array_equal(lam[b, h, :S][inside], T[b][sid[inside]])
            assert np.array_equal(lam[b, h, :S][inside] > 0, T_ref[sid[inside]] > 0)
