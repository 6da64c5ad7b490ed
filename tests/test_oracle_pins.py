"""Pins for the CPU oracle: closed forms, invariants, library routines and brute force.

The paper prints no worked numeric example, so each oracle function is pinned against
what the mathematics fixes.  Every pin is chosen so that a plausible mistake (a dropped
term, a transposed operand, a wrong axis or index) fails at least one assertion.
"""
import itertools
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2512_07993_b200 import workloads as W


def bits(x):
    """float array (bf16-representable or not) -> bf16 bit patterns via torch RNE."""
    return W.bf16_bits(torch.as_tensor(np.asarray(x, np.float32)).to(torch.bfloat16))


def unbits(b):
    return W.bits_to_bf16(b).float().numpy().astype(np.float64)


def sigm(x):
    return 1.0 / (1.0 + math.exp(-x))


rng = np.random.default_rng(7)


# ------------------------------------------------------------------ O1 token importance
def test_o1_closed_form_two_tokens():
    # d=4 so the scale is 1/2; K = [(2,0,0,0), 0]; one head, one row with q=(c,0,0,0):
    # logits (c, 0) -> weights (sigmoid(c), sigmoid(-c)).
    K = bits([[2, 0, 0, 0], [0, 0, 0, 0]])
    for c in (1.0, -3.0, 0.5):
        Q = bits([[[c, 0, 0, 0]]])
        ti = oracle.token_importance(K, Q)
        assert np.allclose(ti, [sigm(c), sigm(-c)], rtol=0, atol=1e-15)


def test_o1_layout_max_over_heads_mean_over_window():
    # n=2 heads, alpha=2 rows, Q stored [head][row][d].  Row logits c(q,w):
    # c(0,0)=1, c(0,1)=3, c(1,0)=-1, c(1,1)=-2.
    K = bits([[2, 0, 0, 0], [0, 0, 0, 0]])
    Q = bits([[[1, 0, 0, 0], [3, 0, 0, 0]], [[-1, 0, 0, 0], [-2, 0, 0, 0]]])
    ti = oracle.token_importance(K, Q)
    t0 = 0.5 * (max(sigm(1), sigm(-1)) + max(sigm(3), sigm(-2)))
    t1 = 0.5 * (max(sigm(-1), sigm(1)) + max(sigm(-3), sigm(2)))
    assert np.allclose(ti, [t0, t1], atol=1e-15)
    # a [row][head] reading of Q, or max over rows / mean over heads, gives other numbers
    wrong_layout = 0.5 * (max(sigm(1), sigm(3)) + max(sigm(-1), sigm(-2)))
    wrong_axes = max(0.5 * (sigm(1) + sigm(-1)), 0.5 * (sigm(3) + sigm(-2)))
    assert abs(t0 - wrong_layout) > 1e-2 and abs(t0 - wrong_axes) > 1e-2


def test_o1_equal_keys_uniform():
    N, d = 37, 16
    K = np.tile(bits(rng.standard_normal((1, d))), (N, 1))
    Q = bits(rng.standard_normal((3, 5, d)))
    ti = oracle.token_importance(K, Q)
    assert np.allclose(ti, 1.0 / N, rtol=1e-14)


def test_o1_mass_bounds_and_single_head_sum():
    N, d = 200, 32
    K = bits(rng.standard_normal((N, d)))
    for n in (1, 4):
        Q = bits(rng.standard_normal((n, 6, d)))
        s = oracle.token_importance(K, Q).sum()
        if n == 1:
            assert abs(s - 1.0) < 1e-12
        else:
            assert 1.0 - 1e-12 <= s <= n + 1e-12 and s > 1.05


def test_o1_matches_library_softmax():
    # alpha=1, n=1 is textbook attention weights; general case against torch fp64 ops.
    N, d = 150, 64
    Kb = bits(rng.standard_normal((N, d)))
    Qb = bits(rng.standard_normal((4, 8, d)))
    K, Q = torch.from_numpy(unbits(Kb)), torch.from_numpy(unbits(Qb))
    one = oracle.token_importance(Kb, Qb[:1, :1])
    ref1 = torch.softmax(K @ Q[0, 0] / math.sqrt(d), dim=0).numpy()
    assert np.allclose(one, ref1, rtol=1e-12, atol=1e-16)
    A = torch.softmax(torch.einsum("qwd,td->qwt", Q, K) / math.sqrt(d), dim=-1)
    ref = A.amax(dim=0).mean(dim=0).numpy()
    assert np.allclose(oracle.token_importance(Kb, Qb), ref, rtol=1e-12, atol=1e-16)


def test_o1_key_shift_invariance():
    # adding one fixed vector to every key shifts each logit row by a constant
    N, d = 64, 16
    K = np.round(rng.standard_normal((N, d)) * 4) / 4          # exact in bf16 with the shift
    u = np.round(rng.standard_normal(d) * 4) / 4
    Q = rng.standard_normal((2, 3, d))
    a = oracle.token_importance(bits(K), bits(Q))
    b = oracle.token_importance(bits(K + u), bits(Q))
    assert np.array_equal(unbits(bits(K + u)), K + u)
    assert np.allclose(a, b, rtol=1e-11, atol=1e-16)


# ------------------------------------------------------------------ O2 pooling
def test_o2_closed_form():
    K = bits([[3, 4, 0, 0], [3, 4, 0, 0], [0, 0, 6, 8], [0, 0, 0, 0], [1, 0, 0, 0]])
    off = [0, 2, 3, 5]
    ti = np.array([0.1, 0.3, 0.2, 0.25, 0.15])
    imp, vbar = oracle.pool(K, off, ti, eps=1e-6)
    assert np.allclose(imp, [0.2, 0.2, 0.2], atol=1e-15)
    assert np.allclose(vbar[0], np.array([3, 4, 0, 0]) / (5 + 1e-6), atol=1e-15)
    assert np.allclose(vbar[1], np.array([0, 0, 6, 8]) / (10 + 1e-6), atol=1e-15)
    assert np.allclose(vbar[2], np.array([0.5, 0, 0, 0]) / (0.5 + 1e-6), atol=1e-15)


def test_o2_mass_permutation_scale():
    N, d = 90, 32
    lens = [10, 25, 5, 50]
    off = np.concatenate([[0], np.cumsum(lens)])
    K = np.round(rng.standard_normal((N, d)) * 8) / 8
    ti = rng.random(N)
    imp, vbar = oracle.pool(bits(K), off, ti)
    assert abs((imp * lens).sum() - ti.sum()) < 1e-12
    # permute tokens inside sentence 1
    perm = np.arange(N)
    perm[10:35] = 10 + rng.permutation(25)
    imp2, vbar2 = oracle.pool(bits(K[perm]), off, ti[perm])
    assert np.allclose(imp, imp2, atol=1e-14) and np.allclose(vbar, vbar2, atol=1e-14)
    # scale sentence 3's keys by 2 (exact in bf16): cosine geometry unchanged
    K2 = K.copy(); K2[40:] *= 2
    _, vbar3 = oracle.pool(bits(K2), off, ti, eps=0.0)
    _, vbar0 = oracle.pool(bits(K), off, ti, eps=0.0)
    assert np.allclose(vbar0, vbar3, atol=1e-14)
    assert np.allclose(np.linalg.norm(vbar0, axis=1), 1.0, atol=1e-14)


# ------------------------------------------------------------------ O3 Gram terms
def test_o3_closed_form_axis_and_diagonal():
    e = np.eye(4)
    vbar = np.stack([e[0], e[0], e[1]])
    G, red, lam = oracle.gram_terms(vbar, 0.95)
    assert np.array_equal(G, [[1, 1, 0], [1, 1, 0], [0, 0, 1]])
    E = math.e
    assert np.allclose(red, [(E / (E + 1) + 0.5) / 3, (E / (E + 1) + 0.5) / 3, (2 / (E + 1)) / 3], atol=1e-15)
    assert np.array_equal(lam, [1.0, 0.0, 0.0])


def test_o3_sum_orthogonal_identical():
    S, d = 9, 16
    v = rng.standard_normal((S, d)); v /= np.linalg.norm(v, axis=1, keepdims=True)
    _, red, _ = oracle.gram_terms(v, 0.95)
    assert abs(red.sum() - 1.0) < 1e-13
    _, red, lam = oracle.gram_terms(np.eye(d)[:S], 0.95)
    assert np.allclose(red, 1.0 / S, atol=1e-15) and not lam.any()
    G, red, lam = oracle.gram_terms(np.tile(v[:1], (S, 1)), 0.95)
    assert np.allclose(G, 1.0, atol=1e-15) and np.allclose(red, 1.0 / S, atol=1e-15)
    assert np.allclose(lam[:-1], 1.0, atol=1e-15) and lam[-1] == 0.0   # last copy is kept


def test_o3_duplicates_flag_earlier_keep_later():
    d = 8
    v = np.eye(d)[:6].copy()
    v[4] = v[1]                      # sentence 4 repeats sentence 1
    v[5] = v[1]                      # and so does 5: three copies
    _, _, lam = oracle.gram_terms(v, 0.95)
    assert np.array_equal(lam, [0, 1, 0, 0, 1, 0])
    # strictly-later only: tau below the self-similarity must not flag everything
    _, _, lam = oracle.gram_terms(np.eye(d)[:4], 0.5)
    assert not lam.any()
    # lam takes the largest later similarity
    c1, c2 = 0.96, 0.99
    v = np.zeros((3, 3)); v[0] = [1, 0, 0]
    v[1] = [c1, math.sqrt(1 - c1 * c1), 0]; v[2] = [c2, 0, math.sqrt(1 - c2 * c2)]
    _, _, lam = oracle.gram_terms(v, 0.95)
    assert abs(lam[0] - c2) < 1e-15 and lam[2] == 0.0
    assert abs(lam[1] - c1 * c2) < 1e-15          # 0.9504 > tau


def test_o3_matches_library_softmax():
    S, d = 23, 12
    v = rng.standard_normal((S, d)); v /= np.linalg.norm(v, axis=1, keepdims=True)
    G, red, _ = oracle.gram_terms(v, 0.95)
    Gt = torch.from_numpy(v) @ torch.from_numpy(v).T
    assert np.allclose(G, Gt.numpy(), atol=1e-15)
    Gt = Gt.masked_fill(torch.eye(S, dtype=torch.bool), float("-inf"))
    ref = torch.softmax(Gt, dim=1).sum(dim=0) / S
    assert np.allclose(red, ref.numpy(), rtol=1e-13)


def test_o1_to_o4_sentence_permutation_equivariance():
    d, lens = 16, [5, 9, 3, 7, 4]
    N = sum(lens)
    off = np.concatenate([[0], np.cumsum(lens)])
    K = bits(rng.standard_normal((N, d))); Q = bits(rng.standard_normal((2, 4, d)))
    def run(Kb, off):
        ti = oracle.token_importance(Kb, Q)
        imp, vbar = oracle.pool(Kb, off, ti)
        G, red, lam = oracle.gram_terms(vbar, 0.95)
        return imp, red, G
    imp, red, G = run(K, off)
    perm = [3, 0, 4, 2, 1]
    rows = np.concatenate([np.arange(off[i], off[i + 1]) for i in perm])
    off2 = np.concatenate([[0], np.cumsum([lens[i] for i in perm])])
    imp2, red2, G2 = run(K[rows], off2)
    assert np.allclose(imp2, imp[perm], rtol=1e-11)
    assert np.allclose(red2, red[perm], rtol=1e-11)
    assert np.allclose(G2, G[np.ix_(perm, perm)], atol=1e-13)


def test_o4_closed_form():
    s = oracle.final_score([0.5, 0.25], [0.125, 0.5], [0.0, 1.0], 0.25)
    assert np.array_equal(s, np.array([0.25 * 0.5 - 0.75 * 0.125, 0.25 * 0.25 - 0.75 * 0.5 - 1.0], np.float32))
    # rounded once from double
    x = oracle.final_score([1.0 / 3], [1.0 / 7], [0.0], 0.1)
    assert x[0] == np.float32(0.1 * (1.0 / 3) - 0.9 * (1.0 / 7))


# ------------------------------------------------------------------ O5 selection
def brute_select(score, lens, budget, protect_tail):
    S = len(lens)
    off = np.concatenate([[0], np.cumsum(lens)])
    total = off[-1]
    if total <= budget:
        return np.ones(S, np.uint8)
    forced = [i for i in range(S) if protect_tail > 0 and lens[i] > 0 and off[i + 1] > total - protect_tail]
    rest = [i for i in range(S) if i not in forced]
    # rank of i among the rest = number of j that beat it
    beaten_by = {i: sum(1 for j in rest if (score[j] > score[i]) or (score[j] == score[i] and j < i))
                 for i in rest}
    rest = sorted(rest, key=lambda i: beaten_by[i])
    order = forced + rest
    best = 0
    for m in range(S + 1):                       # largest prefix that fits
        if sum(lens[i] for i in order[:m]) <= budget:
            best = m
        else:
            break
    keep = np.zeros(S, np.uint8)
    keep[order[:best]] = 1
    return keep


def test_o5_bruteforce_small():
    r = np.random.default_rng(11)
    for trial in range(300):
        S = int(r.integers(1, 9))
        lens = r.integers(1, 9, size=S)
        score = np.round(r.standard_normal(S), 1).astype(np.float32)   # many exact ties
        budget = int(r.integers(0, lens.sum() + 3))
        pt = int(r.integers(0, 6))
        off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
        keep, kept, new_len = oracle.select(score, off, budget, pt)
        ref = brute_select(score, lens, budget, pt)
        assert np.array_equal(keep, ref), (trial, score, lens, budget, pt)
        assert new_len == int((lens * ref).sum()) <= max(budget, 0) or lens.sum() <= budget
        assert np.array_equal(kept, np.nonzero(ref)[0])


def test_o5_hand_examples():
    off = np.array([0, 4, 8, 12, 16], np.int32)
    # scores: best is 2, then 0, then 3, then 1.  Budget 9 -> keeps 2 and 0 (8 tokens), stops at 3.
    keep, kept, nl = oracle.select(np.array([0.5, -1.0, 0.9, 0.1], np.float32), off, 9, 0)
    assert keep.tolist() == [1, 0, 1, 0] and kept.tolist() == [0, 2] and nl == 8
    # no skipping ahead: the first sentence that does not fit ends the walk
    off2 = np.array([0, 4, 12, 14], np.int32)      # lengths 4, 8, 2
    keep, _, nl = oracle.select(np.array([0.9, 0.5, 0.1], np.float32), off2, 7, 0)
    assert keep.tolist() == [1, 0, 0] and nl == 4
    # ties: lower index wins
    keep, _, _ = oracle.select(np.array([0.3, 0.3, 0.3, 0.3], np.float32), off, 8, 0)
    assert keep.tolist() == [1, 1, 0, 0]
    # protected tail: last 5 tokens touch sentences 2 and 3, they go first whatever their score
    keep, _, nl = oracle.select(np.array([0.9, 0.8, -5.0, -6.0], np.float32), off, 12, 5)
    assert keep.tolist() == [1, 0, 1, 1] and nl == 12
    # fits already: identity
    keep, kept, nl = oracle.select(np.array([0.0, 0.0, 0.0, 0.0], np.float32), off, 16, 0)
    assert keep.all() and nl == 16 and kept.tolist() == [0, 1, 2, 3]


def test_o5_invariants_random():
    r = np.random.default_rng(5)
    for _ in range(50):
        S = int(r.integers(5, 200))
        lens = r.integers(1, 97, size=S)
        off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
        score = r.standard_normal(S).astype(np.float32)
        budget = int(lens.sum() // 3)
        keep, kept, nl = oracle.select(score, off, budget, 32)
        assert nl <= budget and nl == int(lens[keep.astype(bool)].sum())
        total = off[-1]
        forced = off[1:] > total - 32
        kept_un = keep.astype(bool) & ~forced
        drop_un = ~keep.astype(bool) & ~forced
        if kept_un.any() and drop_un.any():
            assert score[kept_un].min() >= score[drop_un].max()
        assert nl > budget - 96 - 1 or not drop_un.any()
        # idempotent: selecting again on the survivors keeps them all
        off2 = np.concatenate([[0], np.cumsum(lens[kept])]).astype(np.int32)
        keep2, _, nl2 = oracle.select(score[kept], off2, budget, 32)
        assert keep2.all() and nl2 == nl


def test_flagged_sentences_go_first():
    # lam ~ 1 dwarfs the token-level terms, so every flagged sentence is dropped before
    # any unflagged one
    cfg = W.config(0, dup_rate=0.4, ctx_lo=400, ctx_hi=400, batch=1)
    L = W.make_layer(cfg)
    sl = W.slab_rows(L, 0, 0)
    n = int(L["kv_len"][0, 0]); S = int(L["n_sent"][0, 0])
    Kb = W.bf16_bits(L["K"][sl][:n]); Qb = W.bf16_bits(L["q_win"][0, :cfg.group])
    off = L["sent_off"][0, 0, :S + 1]
    ti = oracle.token_importance(Kb, Qb)
    imp, vbar = oracle.pool(Kb, off, ti)
    _, red, lam = oracle.gram_terms(vbar, 0.95)
    score = oracle.final_score(imp, red, lam, 0.1)
    flagged = lam > 0
    # a family = a fresh sentence and every (transitive) noisy copy of it; all members are
    # mutually similar, so every member but the last one has a later twin
    src = L["dup_src"][0]
    root = np.arange(S)
    for i in range(S):
        if src[i] >= 0:
            root[i] = root[src[i]]
    has_later_twin = np.array([(root[i + 1:] == root[i]).any() for i in range(S)])
    assert flagged.sum() >= 3 and np.array_equal(flagged, has_later_twin)
    assert score[flagged].max() < score[~flagged].min()
    keep, _, _ = oracle.select(score, off, int(0.7 * n), 0)
    if (keep == 0).any() and (~flagged & (keep == 0)).any():
        assert not keep[flagged].any()


# ------------------------------------------------------------------ O6 compaction
def test_o6_rows_and_ranges():
    d = 8
    lens = [3, 2, 4, 1, 5]
    N = sum(lens)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    K = bits(rng.standard_normal((N, d))); V = bits(rng.standard_normal((N, d)))
    keep = np.array([0, 1, 0, 1, 1], np.uint8)
    sid = np.array([10, 11, 12, 13, 14], np.int32)
    Ko, Vo, im, nso, nsid = oracle.compact(K, V, keep, off, sid)
    assert im.tolist() == [3, 4, 9, 10, 11, 12, 13, 14]
    assert np.all(np.diff(im) > 0)
    assert np.array_equal(Ko, K[im]) and np.array_equal(Vo, V[im])
    assert nso.tolist() == [0, 2, 3, 8] and nsid.tolist() == [11, 13, 14]
    # keep none / keep all
    Ko, _, im, nso, nsid = oracle.compact(K, V, np.zeros(5, np.uint8), off, sid)
    assert len(Ko) == 0 and nso.tolist() == [0] and len(nsid) == 0
    Ko, Vo, im, nso, nsid = oracle.compact(K, V, np.ones(5, np.uint8), off, sid)
    assert np.array_equal(Ko, K) and im.tolist() == list(range(N)) and np.array_equal(nso, off)


def test_o6_random_against_numpy_gather():
    r = np.random.default_rng(3)
    for _ in range(20):
        S = int(r.integers(1, 40)); d = 4
        lens = r.integers(0, 12, size=S)             # empty sentences allowed
        off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
        N = int(off[-1])
        K = r.integers(0, 65535, size=(N, d)).astype(np.uint16)
        V = r.integers(0, 65535, size=(N, d)).astype(np.uint16)
        keep = (r.random(S) < 0.5).astype(np.uint8)
        Ko, Vo, im, nso, nsid = oracle.compact(K, V, keep, off, np.arange(S, dtype=np.int32))
        mask = np.repeat(keep.astype(bool), lens)
        assert np.array_equal(im, np.nonzero(mask)[0])
        assert np.array_equal(Ko, K[mask]) and np.array_equal(Vo, V[mask])
        alive = keep.astype(bool) & (lens > 0)
        assert np.array_equal(nsid, np.nonzero(alive)[0])
        assert np.array_equal(nso, np.concatenate([[0], np.cumsum(lens[alive])]))


# ------------------------------------------------------------------ O7 decode attention
def test_o7_special_cases():
    d = 16
    q = bits(rng.standard_normal((4, d)))
    K = bits(rng.standard_normal((1, d))); V = bits(rng.standard_normal((1, d)))
    out, _ = oracle.decode_attn(q, K, V, 1)
    assert np.array_equal(out, np.tile(V, (4, 1)))                 # single token: out = V[0]
    out, _ = oracle.decode_attn(q, K, V, 0)
    assert not out.any()                                           # empty: zeros
    N = 10
    K = np.tile(bits(rng.standard_normal((1, d))), (N, 1)); Vf = np.round(rng.standard_normal((N, d)) * 4) / 4
    _, o64 = oracle.decode_attn(q, K, bits(Vf), N)
    assert np.allclose(o64, np.tile(Vf.mean(0), (4, 1)), atol=1e-14)   # equal keys: mean of V
    q2 = q.copy(); q2[2] = q2[0]
    K = bits(rng.standard_normal((N, d)))
    out, _ = oracle.decode_attn(q2, K, bits(Vf), N)
    assert np.array_equal(out[0], out[2])
    # rows beyond len are ignored
    o_a, _ = oracle.decode_attn(q, K, bits(Vf), 6)
    o_b, _ = oracle.decode_attn(q, K[:6], bits(Vf)[:6], 6)
    assert np.array_equal(o_a, o_b)


def test_o7_closed_form_and_library():
    # two tokens, d=4: weights (sigmoid(c), sigmoid(-c)) as in the O1 pin
    K = bits([[2, 0, 0, 0], [0, 0, 0, 0]]); V = bits([[1, 0, 2, 0], [0, 1, 0, 4]])
    _, o = oracle.decode_attn(bits([[1, 0, 0, 0]]), K, V, 2)
    p = sigm(1.0)
    assert np.allclose(o[0], [p, 1 - p, 2 * p, 4 * (1 - p)], atol=1e-15)
    N, d = 77, 128
    qb, Kb, Vb = bits(rng.standard_normal((4, d))), bits(rng.standard_normal((N, d))), bits(rng.standard_normal((N, d)))
    out, o64 = oracle.decode_attn(qb, Kb, Vb, N)
    q, K, V = (torch.from_numpy(unbits(x)) for x in (qb, Kb, Vb))
    ref = torch.softmax(q @ K.T / math.sqrt(d), dim=-1) @ V
    assert np.allclose(o64, ref.numpy(), rtol=1e-12, atol=1e-15)
    assert np.abs(unbits(out) - o64).max() <= np.abs(o64).max() * 2.0 ** -8


# ------------------------------------------------------------------ O8 steering
def test_o8_bit_exact_rounding():
    one, ulp = 1.0, 2.0 ** -7                     # bf16 spacing at 1.0
    h = bits([[one, one + ulp, one, 3.0], [one, one, one, one]])
    v = bits([2.0 ** -8, 2.0 ** -8, 0.5, -1.5])
    out = oracle.steer(h, v, np.array([1.0, 9.0], np.float32), np.array([1, 0], np.uint8))
    # ties to even: 1 + half ulp -> 1 ; (1+ulp) + half ulp -> 1 + 2 ulp ; plain sums exact
    assert unbits(out)[0].tolist() == [1.0, 1.0 + 2 * ulp, 1.5, 1.5]
    assert np.array_equal(out[1], h[1])            # flag 0: untouched
    # one fused rounding, against float64 arithmetic (exact here) and torch's bf16 rounding
    r = np.random.default_rng(9)
    hb = bits(r.standard_normal((3, 64))); vb = bits(0.01 * r.standard_normal(64))
    a = np.array([1.0, 1.26, 1.78], np.float32)
    out = oracle.steer(hb, vb, a, np.ones(3, np.uint8))
    ref32 = (a.astype(np.float64)[:, None] * unbits(vb)[None, :] + unbits(hb)).astype(np.float32)
    assert np.array_equal(out, bits(ref32))


# ------------------------------------------------------------------ batch drivers == per-slab functions
# ------------------------------------------------------------------ O9-O11 lookup table and Phi
def test_o9_table_closed_form():
    """Hand-built hidden states whose sentence means are known vectors."""
    d = 8
    e = np.eye(d)
    c = 0.96
    u = 24 * e[0] + 7 * e[1]                              # |u| = 25, cos(u, e0) = 0.96, exact in bf16
    rows = [2 * e[0], 4 * e[0],                           # sentence 0: mean 3 e0
            e[2], e[2], e[2],                             # sentence 1: e2
            u + 0.5 * e[3], u - 0.5 * e[3],               # sentence 2: mean u (the e3 parts cancel)
            8 * e[0]]                                     # sentence 3: e0 direction again
    off = np.array([0, 2, 5, 7, 8], np.int32)
    T, G = oracle.lookup_table(bits(np.array(rows)), off, 0.95, eps=0.0)
    assert np.allclose(G[0], [1, 0, c, 1], atol=1e-15) and np.allclose(G[2, 3], c, atol=1e-15)
    # sentence 0 repeats as sentence 3 (cos 1) and nearly as sentence 2 (0.96): the largest later one counts;
    # sentence 2 is flagged through sentence 3; sentence 1 is unrelated; the last sentence has no later one
    assert np.allclose(T, [1.0, 0.0, c, 0.0], atol=1e-15)
    # with the threshold above 0.96 only the exact repeat is flagged
    T2, _ = oracle.lookup_table(bits(np.array(rows)), off, 0.97, eps=0.0)
    assert np.allclose(T2, [1.0, 0.0, 0.0, 0.0], atol=1e-15)
    # mean pooling, not sum or last row: sentence 2 would otherwise not be the direction of u
    assert np.allclose(G[2, 2], 1.0, atol=1e-15) and abs(G[1, 2]) < 1e-15


def test_o9_matches_torch_and_incremental_form():
    """Against torch fp64 ops, and against the running form (each closing sentence compared with
    the earlier ones only, keeping the running maximum), which must give the same table."""
    d, lens = 64, [3, 1, 7, 2, 5, 4, 1, 6]
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    H = rng.standard_normal((off[-1], d))
    H[off[4]:off[5]] = H[off[0]:off[0] + 1] + 0.05 * rng.standard_normal((lens[4], d))  # 4 ~ first row of 0
    H[off[6]:off[7]] = np.mean(H[off[2]:off[3]], axis=0)                                # 6 repeats 2's mean
    Hb = bits(H)
    tau = 0.5
    T, G = oracle.lookup_table(Hb, off, tau)
    Hd = torch.from_numpy(unbits(Hb))
    m = torch.stack([Hd[off[i]:off[i + 1]].mean(dim=0) for i in range(len(lens))])
    v = m / (m.norm(dim=1, keepdim=True) + 1e-6)
    Gt = (v @ v.T).numpy()
    assert np.allclose(G, Gt, atol=1e-13)
    run = np.zeros(len(lens))
    for j in range(len(lens)):
        for i in range(j):
            if Gt[i, j] > tau:
                run[i] = max(run[i], Gt[i, j])
    assert np.allclose(T, run, atol=1e-13)
    assert T[2] > 0.99 and T[-1] == 0.0


def test_o10_phi_lookup_and_compaction():
    T = np.array([0.0, 0.97, 0.0, 0.99, 0.96])
    assert np.array_equal(oracle.map_table(T, [3, 0, 4, 4, 1]), [0.99, 0.0, 0.96, 0.96, 0.97])
    assert np.array_equal(oracle.map_table(T, [-1, 5, 2, 100]), [0, 0, 0, 0])     # no entry -> no penalty
    # after an eviction the surviving cache-space sentences still find their own entries
    d, lens = 8, [2, 3, 1, 4, 2]
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    K = bits(rng.standard_normal((off[-1], d))); V = bits(rng.standard_normal((off[-1], d)))
    keep = np.array([1, 0, 1, 0, 1], np.uint8)
    sid = np.arange(5, dtype=np.int32)
    _, _, _, _, nsid = oracle.compact(K, V, keep, off, sid)
    assert np.array_equal(oracle.map_table(T, nsid), oracle.map_table(T, sid)[keep == 1])


def test_o11_score_with_table():
    d, lens = 16, [4, 6, 3, 5]
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    K = bits(rng.standard_normal((off[-1], d))); Q = bits(rng.standard_normal((2, 3, d)))
    T = np.array([0.0, 0.0, 0.98, 0.0, 0.0, 0.96])
    sid = np.array([1, 2, 4, 5], np.int32)
    imp, red, lam, sc = oracle.score_with_table(K, Q, off, sid, T, 0.1, 0.95)
    tok = oracle.token_importance(K, Q)
    imp0, vbar = oracle.pool(K, off, tok)
    _, red0, lam_keys = oracle.gram_terms(vbar, 0.95)
    assert np.array_equal(imp, imp0) and np.array_equal(red, red0)       # importance and redundancy unchanged
    assert np.array_equal(lam, [0.0, 0.98, 0.0, 0.96]) and not lam_keys.any()
    expect = (0.1 * imp - 0.9 * red - lam).astype(np.float32)
    assert np.array_equal(sc, expect)
    # a flagged sentence ranks below every unflagged one whatever its importance
    assert sc[[1, 3]].max() < sc[[0, 2]].min()


# ------------------------------------------------------------------ O12-O13 exactly-B retention
def test_o12_hand_example():
    lens = [3, 4, 2, 5]
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    score = np.array([0.5, 0.1, 0.9, 0.3], np.float32)          # rank: 2, 0, 3, 1
    tok = np.zeros(14, np.float32)
    tok[9:14] = [0.2, 0.7, 0.7, 0.1, 0.4]                        # sentence 3
    # budget 8: sentences 2 and 0 fit (5 tokens); sentence 3 (5 tokens) does not: its 3 best tokens stay,
    # the tie 0.7 / 0.7 keeps both, then 0.4
    keep, tk, nl = oracle.select_fill(score, off, tok, 8, 0)
    assert np.array_equal(keep, [1, 0, 1, 2]) and nl == 8
    assert np.array_equal(np.nonzero(tk)[0], [0, 1, 2, 7, 8, 10, 11, 13])
    # budget 7: two tokens of the cut sentence; among the equal pair the earlier comes first, both fit
    keep, tk, nl = oracle.select_fill(score, off, tok, 7, 0)
    assert np.array_equal(np.nonzero(tk)[0], [0, 1, 2, 7, 8, 10, 11]) and nl == 7
    # budget 6: one token: the earlier of the equal pair
    keep, tk, nl = oracle.select_fill(score, off, tok, 6, 0)
    assert np.array_equal(np.nonzero(tk)[0], [0, 1, 2, 7, 8, 10]) and keep[3] == 2
    # budget 5: no slack, nothing partial: identical to the whole-sentence rule
    keep, tk, nl = oracle.select_fill(score, off, tok, 5, 0)
    assert np.array_equal(keep, [1, 0, 1, 0]) and nl == 5
    # fits already
    keep, tk, nl = oracle.select_fill(score, off, tok, 14, 0)
    assert keep.all() and tk.all() and nl == 14


def test_o12_token_level_redundancy_orders_the_cut_sentence():
    """With a token-level redundancy the cut sentence gives up its tokens in the order of
    sigma * I - (1 - sigma) * R (Eq. "I_final" per token): hand example where the redundancy overturns the
    importance order, the limits sigma = 1 (importance alone) and R constant (importance alone again)."""
    lens = [2, 5]
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    score = np.array([0.9, 0.1], np.float32)                     # sentence 0 first, sentence 1 is cut
    imp = np.array([0, 0, 0.50, 0.40, 0.30, 0.20, 0.10], np.float32)
    red = np.array([0, 0, 0.90, 0.10, 0.80, 0.00, 0.05], np.float32)
    # sigma = 0.5: keys 0.5*I - 0.5*R = -0.20, 0.15, -0.25, 0.10, 0.025 -> order of tokens 3, 5, 6, 2, 4
    keep, tk, nl = oracle.select_fill(score, off, imp, 4, 0, tok_red=red, sigma=0.5)
    assert np.array_equal(keep, [1, 2]) and nl == 4
    assert np.array_equal(np.nonzero(tk)[0], [0, 1, 3, 5])
    keep, tk, nl = oracle.select_fill(score, off, imp, 6, 0, tok_red=red, sigma=0.5)
    assert np.array_equal(np.nonzero(tk)[0], [0, 1, 2, 3, 5, 6])   # the most redundant token (4) goes first
    # sigma = 1: the redundancy has no weight
    k1, t1, _ = oracle.select_fill(score, off, imp, 4, 0, tok_red=red, sigma=1.0)
    k0, t0, _ = oracle.select_fill(score, off, imp, 4, 0)
    assert np.array_equal(t1, t0) and np.array_equal(np.nonzero(t0)[0], [0, 1, 2, 3])
    # a constant redundancy shifts every key alike (in exact arithmetic; here with values that stay exact in fp32)
    kc, tc, _ = oracle.select_fill(score, off, imp, 4, 0, tok_red=np.full(7, 0.25, np.float32), sigma=0.5)
    assert np.array_equal(tc, t0)
    # the key itself: each operation rounded to fp32
    key = oracle.token_final_key(imp, red, 0.5)
    assert key.dtype == np.float32
    want = [np.float32(np.float32(0.5) * i) - np.float32(np.float32(0.5) * r) for i, r in zip(imp, red)]
    assert np.array_equal(key, np.array(want, np.float32))


def test_o12_random_properties():
    r = np.random.default_rng(7)
    for trial in range(60):
        S = int(r.integers(1, 12))
        lens = r.integers(0, 7, size=S)
        off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
        N = int(off[-1])
        score = r.choice(np.array([-1.0, -0.5, 0.0, 0.25, 0.5], np.float32), size=S)
        tok = r.choice(np.array([0.0, 0.1, 0.2, 0.3], np.float32), size=N)
        budget = int(r.integers(0, N + 2)); pt = int(r.integers(0, 4))
        keep, tk, nl = oracle.select_fill(score, off, tok, budget, pt)
        k5, _, nl5 = oracle.select(score, off, budget, pt)
        assert np.array_equal(keep == 1, k5 == 1)                 # the whole sentences are those of O5
        assert nl == int(tk.sum()) and nl5 <= nl <= max(budget, nl5)
        if N > budget:
            assert nl == budget                                   # exactly B
        cut = np.nonzero(keep == 2)[0]
        assert len(cut) <= 1
        for i in range(S):
            span = tk[off[i]:off[i + 1]]
            if keep[i] == 1: assert span.all()
            if keep[i] == 0: assert not span.any()
        if len(cut):
            c = int(cut[0]); b, e = int(off[c]), int(off[c + 1])
            inside, outside = tok[b:e][tk[b:e] == 1], tok[b:e][tk[b:e] == 0]
            assert 0 < len(inside) < e - b
            assert inside.min() >= outside.max()                  # no evicted token outranks a kept one
            # among equal values the earlier tokens are the kept ones
            v = inside.min()
            eq = np.nonzero(tok[b:e] == v)[0]
            flags = tk[b:e][eq]
            assert (np.diff(flags.astype(int)) <= 0).all()


def test_o13_matches_o6_and_gather():
    r = np.random.default_rng(11)
    d = 8
    for trial in range(30):
        S = int(r.integers(1, 9))
        lens = r.integers(0, 6, size=S)
        off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
        N = int(off[-1])
        K = bits(r.standard_normal((max(N, 1), d)))[:N]; V = bits(r.standard_normal((max(N, 1), d)))[:N]
        sid = r.permutation(50)[:S].astype(np.int32)
        # whole-sentence survivors: must agree with the sentence-level compaction
        keep = r.integers(0, 2, size=S).astype(np.uint8)
        tk = np.zeros(N, np.uint8)
        for i in range(S):
            tk[off[i]:off[i + 1]] = keep[i]
        Ko, Vo, im, nso, nsid = oracle.compact_tokens(K, V, tk, off, sid)
        if N:
            K6, V6, im6, nso6, nsid6 = oracle.compact(K, V, keep, off, sid)
            assert np.array_equal(Ko, K6) and np.array_equal(Vo, V6) and np.array_equal(im, im6)
            assert np.array_equal(nso, nso6) and np.array_equal(nsid, nsid6)
        # arbitrary token survivors: numpy gather and per-sentence counts
        tk = r.integers(0, 2, size=N).astype(np.uint8)
        Ko, Vo, im, nso, nsid = oracle.compact_tokens(K, V, tk, off, sid)
        assert np.array_equal(Ko, K[tk == 1]) and np.array_equal(Vo, V[tk == 1])
        assert np.array_equal(im, np.nonzero(tk)[0])
        counts = np.array([int(tk[off[i]:off[i + 1]].sum()) for i in range(S)])
        assert np.array_equal(np.diff(nso), counts[counts > 0]) and np.array_equal(nsid, sid[counts > 0])


def test_o13_hand_example():
    off = np.array([0, 3, 5, 9], np.int32)
    K = bits(np.arange(9 * 2).reshape(9, 2)); V = bits(-np.arange(9 * 2).reshape(9, 2))
    tk = np.array([1, 1, 1, 0, 0, 0, 1, 0, 1], np.uint8)          # sentence 1 evicted, sentence 2 keeps tokens 6 and 8
    Ko, Vo, im, nso, nsid = oracle.compact_tokens(K, V, tk, off, np.array([4, 5, 6], np.int32))
    assert np.array_equal(im, [0, 1, 2, 6, 8]) and np.array_equal(nso, [0, 3, 5]) and np.array_equal(nsid, [4, 6])
    assert np.array_equal(unbits(Ko)[:, 0], [0, 2, 4, 12, 16])


# ------------------------------------------------------------------ O14 token-level redundancy
def test_o14_closed_form_and_library():
    e = np.eye(4)
    # keys 0 and 1 point the same way (different lengths), key 2 is orthogonal: the 3-sentence closed form of O3
    R = oracle.token_redundancy(bits(np.stack([2 * e[0], 8 * e[0], 4 * e[1]])), eps=0.0)
    E = math.e
    assert np.allclose(R, [(E / (E + 1) + 0.5) / 3, (E / (E + 1) + 0.5) / 3, (2 / (E + 1)) / 3], atol=1e-15)
    assert oracle.token_redundancy(bits(e[:1]))[0] == 0.0            # a single token has nothing to repeat
    N, d = 37, 16
    Kb = bits(rng.standard_normal((N, d)))
    R = oracle.token_redundancy(Kb)
    Kd = torch.from_numpy(unbits(Kb))
    Kn = Kd / (Kd.norm(dim=1, keepdim=True) + 1e-6)
    Gt = (Kn @ Kn.T).masked_fill(torch.eye(N, dtype=torch.bool), float("-inf"))
    ref = torch.softmax(Gt, dim=1).sum(dim=0) / N
    assert np.allclose(R, ref.numpy(), rtol=1e-12) and abs(R.sum() - 1.0) < 1e-13
    # scaling a key changes nothing (cosine), repeating it raises its redundancy above an unrelated key's
    K2 = unbits(Kb).copy(); K2[5] *= 4.0
    assert np.allclose(oracle.token_redundancy(bits(K2)), R, rtol=1e-6)
    K3 = unbits(Kb).copy(); K3[7] = K3[3]
    R3 = oracle.token_redundancy(bits(K3))
    assert R3[3] > R[3] and R3[7] > np.median(R3)


# ------------------------------------------------------------------ O15 range append
def test_o15_append_token_hand_example():
    off, ids = np.array([0, 3, 5], np.int32), np.array([7, 9], np.int32)
    o1, i1 = oracle.append_token(off, ids, False, 11)                 # token 5 extends sentence 9
    assert np.array_equal(o1, [0, 3, 6]) and np.array_equal(i1, [7, 9])
    o2, i2 = oracle.append_token(o1, i1, True, 11)                    # token 6 starts sentence 11
    assert np.array_equal(o2, [0, 3, 6, 7]) and np.array_equal(i2, [7, 9, 11])
    o3, i3 = oracle.append_token(o2, i2, False, 12)
    assert np.array_equal(o3, [0, 3, 6, 8]) and np.array_equal(i3, [7, 9, 11])
    o0, i0 = oracle.append_token(np.array([0], np.int32), np.array([], np.int32), False, 4)   # empty cache
    assert np.array_equal(o0, [0, 1]) and np.array_equal(i0, [4])
    # a stream of tokens with delimiters reproduces the lengths of the sentences
    lens = [4, 1, 6, 2]
    off, ids = np.array([0], np.int32), np.array([], np.int32)
    g = 0
    for n, ln in enumerate(lens):
        for t in range(ln):
            off, ids = oracle.append_token(off, ids, t == 0, n)
    assert np.array_equal(np.diff(off), lens) and np.array_equal(ids, [0, 1, 2, 3])


def test_batch_drivers_match_slab_functions():
    cfg = W.config(0)
    L = W.make_layer(cfg)
    shape = dict(batch=cfg.batch, Hq=cfg.n_q_heads, Hk=cfg.n_kv_heads, d=cfg.head_dim, alpha=cfg.window,
                 max_sent=L["max_sent"], slab_off=L["slab_off"], cap=L["cap"])
    Kb, Vb = W.bf16_bits(L["K"]), W.bf16_bits(L["V"])
    res = oracle.score_batch(shape, Kb, W.bf16_bits(L["q_win"]), L["kv_len"], L["sent_off"], L["n_sent"],
                             0.1, 0.95, 1e-6, want_tok_imp=True)
    sel = oracle.select_batch(res["score"], L["sent_off"], L["n_sent"], cfg.budget, cfg.window)
    cmp_ = oracle.compact_batch(shape, Kb, Vb, sel["keep"], L["sent_off"], L["sent_id"], L["n_sent"], L["kv_len"])
    dec, _ = oracle.decode_attn_batch(shape, W.bf16_bits(L["q"]), cmp_["K"], cmp_["V"], cmp_["kv_len"])
    g = cfg.group
    for b in range(cfg.batch):
        for h in range(cfg.n_kv_heads):
            sl = W.slab_rows(L, b, h)
            n, S = int(L["kv_len"][b, h]), int(L["n_sent"][b, h])
            off = L["sent_off"][b, h, :S + 1]
            ti = oracle.token_importance(Kb[sl][:n], W.bf16_bits(L["q_win"][b, h * g:(h + 1) * g]))
            assert np.array_equal(ti, res["tok_imp"][sl][:n])
            imp, vbar = oracle.pool(Kb[sl][:n], off, ti)
            _, red, lam = oracle.gram_terms(vbar, 0.95)
            sc = oracle.final_score(imp, red, lam, 0.1)
            assert np.array_equal(sc, res["score"][b, h, :S])
            keep, kept, nl = oracle.select(sc, off, cfg.budget, cfg.window)
            assert np.array_equal(keep, sel["keep"][b, h, :S]) and nl == sel["new_len"][b, h] <= cfg.budget
            Ko, Vo, im, nso, nsid = oracle.compact(Kb[sl][:n], Vb[sl][:n], keep, off, L["sent_id"][b, h, :S])
            assert np.array_equal(Ko, cmp_["K"][sl][:nl]) and np.array_equal(im, cmp_["index_map"][sl][:nl])
            assert cmp_["kv_len"][b, h] == nl and cmp_["n_sent"][b, h] == len(nsid)
            assert np.array_equal(nso, cmp_["sent_off"][b, h, :len(nsid) + 1])
            o, _ = oracle.decode_attn(W.bf16_bits(L["q"][b, h * g:(h + 1) * g]), Ko, Vo, nl)
            assert np.array_equal(o, dec[b, h * g:(h + 1) * g])


# ------------------------------------------------------------------ stored values
def test_golden_oracle_outputs_unchanged():
    """The oracle still produces the stored outputs for the seeded tiny slab (the file is written by
    tests/golden/make_golden.py from the oracle alone)."""
    import importlib.util, json, os
    here = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(here, "make_golden.py"))
    mod = importlib.util.module_from_spec(spec); spec.loader.exec_module(mod)
    now, stored = mod.compute(), json.load(open(os.path.join(here, "oracle_tiny_slab.json")))
    assert now.keys() == stored.keys()
    for k, v in stored.items():
        if isinstance(v, list) and v and isinstance(v[0], float):
            assert np.allclose(now[k], v, rtol=1e-10, atol=0.0), k
        elif isinstance(v, float):
            assert abs(now[k] - v) <= 1e-10 * abs(v), k
        else:
            assert now[k] == v, k


def test_paper_hyperparameters_are_the_defaults():
    """Values the paper prints (appendix, "Hyper-parameters") against the defaults of the binding and workloads."""
    import os
    from paper_2512_07993_b200 import binding
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "paper_hyperparameters.txt")
    hp = {}
    for line in open(path):
        if "=" in line and not line.startswith("#"):
            k, v = line.split("=")
            hp[k.strip()] = float(v)
    p = binding.make_params()
    assert abs(p.sigma - hp["sigma"]) < 1e-7 and hp["tau_low"] - 1e-7 <= p.tau <= hp["tau_high"]
    cfg = W.config(4)
    assert cfg.layers == 32 and hp["steer_layer_7b_8b"] < cfg.layers
    L = W.make_layer(W.config(0))
    k = (L["alpha"].astype(np.float64) - hp["alpha0_a"]) / hp["gamma"]           # alpha_t = alpha_0 + gamma * N_o
    assert np.allclose(k, np.round(k), atol=1e-4) and (k >= 0).all()
