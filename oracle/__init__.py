"""ctypes front end of the CPU oracle (``skipkv_oracle.cpp``).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's cpu-baseline / reference legs may
import this package; the CUDA product path never does.  It takes and returns numpy
arrays (bf16 tensors travel as ``uint16`` bit patterns) and shares no code with the
CUDA library.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "skipkv_oracle.cpp")
_LIB = os.path.join(_HERE, "libskipkv_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ -O2 -fopenmp (no fast-math) if it is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(["g++", "-std=c++17", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC],
                       check=True)
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_select.restype = C.c_int
        _lib.oracle_compact.restype = C.c_int
        _lib.oracle_compact_batch.restype = C.c_int
        _lib.oracle_max_threads.restype = C.c_int
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dt):
    a = np.ascontiguousarray(a, dtype=dt)
    return a


def max_threads() -> int:
    return int(lib().oracle_max_threads())


def set_threads(n: int) -> None:
    lib().oracle_set_threads(C.c_int(n))


# ------------------------------------------------------------------ per-slab functions
def token_importance(K_bits, Q_bits):
    """K_bits uint16 [N,d]; Q_bits uint16 [n,alpha,d] -> tok_imp float64 [N]."""
    K_bits = _c(K_bits, np.uint16); Q_bits = _c(Q_bits, np.uint16)
    N, d = K_bits.shape
    n, alpha, d2 = Q_bits.shape
    assert d == d2
    out = np.zeros(N, np.float64)
    lib().oracle_token_importance(_p(K_bits), _p(Q_bits), N, n, alpha, d, _p(out))
    return out


def pool(K_bits, sent_off, tok_imp, eps=1e-6):
    K_bits = _c(K_bits, np.uint16); sent_off = _c(sent_off, np.int32); tok_imp = _c(tok_imp, np.float64)
    S = len(sent_off) - 1
    d = K_bits.shape[1]
    imp = np.zeros(S, np.float64); vbar = np.zeros((S, d), np.float64)
    lib().oracle_pool(_p(K_bits), d, _p(sent_off), S, _p(tok_imp), C.c_double(eps), _p(imp), _p(vbar))
    return imp, vbar


def gram_terms(vbar, tau):
    vbar = _c(vbar, np.float64)
    S, d = vbar.shape
    G = np.zeros((S, S), np.float64); red = np.zeros(S, np.float64); lam = np.zeros(S, np.float64)
    lib().oracle_gram_terms(_p(vbar), S, d, C.c_double(tau), _p(G), _p(red), _p(lam))
    return G, red, lam


def final_score(imp, red, lam, sigma):
    imp = _c(imp, np.float64); red = _c(red, np.float64); lam = _c(lam, np.float64)
    out = np.zeros(len(imp), np.float32)
    lib().oracle_final_score(_p(imp), _p(red), _p(lam), len(imp), C.c_double(sigma), _p(out))
    return out


def select(score, sent_off, budget, protect_tail):
    score = _c(score, np.float32); sent_off = _c(sent_off, np.int32)
    S = len(sent_off) - 1
    keep = np.zeros(S, np.uint8); kept = np.zeros(max(S, 1), np.int32); nl = np.zeros(1, np.int32)
    nk = lib().oracle_select(_p(score), _p(sent_off), S, int(budget), int(protect_tail), _p(keep), _p(kept), _p(nl))
    return keep, kept[:nk].copy(), int(nl[0])


def compact(K_bits, V_bits, keep, sent_off, sent_id):
    K_bits = _c(K_bits, np.uint16); V_bits = _c(V_bits, np.uint16)
    keep = _c(keep, np.uint8); sent_off = _c(sent_off, np.int32); sent_id = _c(sent_id, np.int32)
    S = len(sent_off) - 1
    N, d = K_bits.shape
    Ko = np.zeros_like(K_bits); Vo = np.zeros_like(V_bits)
    im = np.zeros(max(N, 1), np.int32); nso = np.zeros(S + 1, np.int32); nsid = np.zeros(max(S, 1), np.int32)
    nl = np.zeros(1, np.int32)
    ns = lib().oracle_compact(_p(K_bits), _p(V_bits), d, _p(keep), _p(sent_off), _p(sent_id), S, _p(Ko), _p(Vo),
                              _p(im), _p(nso), _p(nsid), _p(nl))
    if ns < 0:
        raise AssertionError("literal range remap disagrees with the prefix-sum form")
    n = int(nl[0])
    return Ko[:n], Vo[:n], im[:n], nso[:ns + 1], nsid[:ns]


def decode_attn(q_bits, K_bits, V_bits, length):
    q_bits = _c(q_bits, np.uint16); K_bits = _c(K_bits, np.uint16); V_bits = _c(V_bits, np.uint16)
    n, d = q_bits.shape
    out = np.zeros((n, d), np.uint16); o64 = np.zeros((n, d), np.float64)
    lib().oracle_decode_attn(_p(q_bits), _p(K_bits), _p(V_bits), int(length), n, d, _p(out), _p(o64))
    return out, o64


def steer(hidden_bits, v_bits, alpha, flag):
    h = _c(hidden_bits, np.uint16).copy(); v = _c(v_bits, np.uint16)
    alpha = _c(alpha, np.float32); flag = _c(flag, np.uint8)
    b, dm = h.shape
    lib().oracle_steer(b, dm, _p(h), _p(v), _p(alpha), _p(flag))
    return h


# ------------------------------------------------------------------ generation-space lookup table
def lookup_table(H_bits, gen_off, tau, eps=1e-6):
    """O9  Lookup table T (Section 4.1, "Sentence Similarity Score" and the sentence-score
    table of Eq. "sentence-score-input"): sentence embeddings are the mean of the LAST-LAYER
    hidden-state rows of each generation-space sentence (normalised as in O2), G is their
    pairwise similarity (Eq. "PSS"), and T[i] = max_{j>i} G_ij when that exceeds tau, else 0
    (the earlier sentence of a redundant pair is flagged, the later one kept).

    H_bits uint16 [N, d_model] (bf16 bits, one sequence); gen_off int32 [S+1] CSR ranges of the
    closed sentences.  Returns (T float64 [S], G float64 [S, S]).
    """
    H_bits = _c(H_bits, np.uint16); gen_off = _c(gen_off, np.int32)
    _, vbar = pool(H_bits, gen_off, np.zeros(H_bits.shape[0], np.float64), eps)
    G, _, T = gram_terms(vbar, tau)
    return T, G


def map_table(T, sent_id):
    """O10  Phi (Eq. "sentence-score-cache"): the penalty of a cache-space sentence is the table
    entry of the generation-space sentence it came from; a sentence without an entry (index
    outside the table) carries no penalty."""
    T = np.asarray(T, np.float64)
    out = np.zeros(len(sent_id), np.float64)
    for i, g in enumerate(np.asarray(sent_id).tolist()):
        if 0 <= g < len(T):
            out[i] = T[g]
    return out


def score_with_table(K_bits, Q_bits, sent_off, sent_id, T, sigma, tau, eps=1e-6):
    """O11  Eq. "I_final" with the sentence penalty read from the table through Phi instead of
    being derived from the pooled keys: importance (O1, O2) and redundancy (O3) as before.
    Returns (imp, red, lam, score fp32)."""
    tok = token_importance(K_bits, Q_bits)
    imp, vbar = pool(K_bits, sent_off, tok, eps)
    _, red, _ = gram_terms(vbar, tau)
    lam = map_table(T, sent_id)
    return imp, red, lam, final_score(imp, red, lam, sigma)


# ------------------------------------------------------------------ exactly-B retention
def token_final_key(tok_imp, tok_red, sigma):
    """Per-token key of the cut sentence when a token-level redundancy is given (Section 4.1, Eq. "I_final" with the
    token-level R of the "Token Redundancy Score" paragraph; the penalty is the same for all tokens of a sentence and
    drops out of the order): sigma * I - (1 - sigma) * R, each operation rounded to fp32 (the precision in which the
    order is decided)."""
    s = np.float32(sigma)
    return (s * np.asarray(tok_imp, np.float32)).astype(np.float32) - ((np.float32(1) - s) * np.asarray(tok_red, np.float32)).astype(np.float32)


def select_fill(score, sent_off, tok_imp, budget, protect_tail, tok_red=None, sigma=None):
    """O12  Selection that retains exactly B tokens (Section 4.1: tokens are evicted in increasing
    order of the final score until the cache meets the budget).  Whole sentences are kept in rank
    order as in O5; the first sentence that does not fit (the cut sentence) then gives up only its
    lowest-scoring tokens: redundancy and penalty are the same for all tokens of a sentence, so
    inside it the final-score order is the token-importance order.  Its `slack = B - kept` tokens of
    largest tok_imp survive (equal values: the earlier token first).  With tok_red (token-level redundancy, O14)
    the tokens of the cut sentence are ordered by token_final_key instead.

    score fp32 [S], sent_off int32 [S+1], tok_imp fp32 [N].  Returns (keep uint8 [S] with 1 = whole
    sentence kept, 2 = cut sentence partly kept; tok_keep uint8 [N]; new_len)."""
    score = np.asarray(score, np.float32); sent_off = np.asarray(sent_off, np.int64)
    tok_imp = np.asarray(tok_imp, np.float32)
    if tok_red is not None:
        tok_imp = token_final_key(tok_imp, tok_red, sigma)
    S = len(sent_off) - 1
    total = int(sent_off[S]) if S > 0 else 0
    keep = np.zeros(S, np.uint8); tok_keep = np.zeros(total, np.uint8)
    if total <= budget:
        keep[:] = 1; tok_keep[:] = 1
        return keep, tok_keep, total
    forced = [protect_tail > 0 and sent_off[i + 1] > total - protect_tail and sent_off[i + 1] > sent_off[i]
              for i in range(S)]
    order = [i for i in range(S) if forced[i]]
    order += sorted((i for i in range(S) if not forced[i]), key=lambda i: (-float(score[i]), i))
    kept = 0
    for i in order:
        b, e = int(sent_off[i]), int(sent_off[i + 1])
        if kept + (e - b) > budget:
            slack = budget - kept
            if slack > 0:
                best = sorted(range(b, e), key=lambda t: (-float(tok_imp[t]), t))[:slack]
                tok_keep[best] = 1
                keep[i] = 2
            break
        kept += e - b
        keep[i] = 1
        tok_keep[b:e] = 1
    return keep, tok_keep, int(tok_keep.sum())


def compact_tokens(K_bits, V_bits, tok_keep, sent_off, sent_id):
    """O13  Compaction with token-level survivors (Section 4.1, "Updating Cache Ranges After
    Eviction", Eq. "after", evaluated literally): survivors p_1 < ... < p_B' are the kept token
    indices; row k of the new cache is old row p_k; sentence (b, e) (inclusive ends) becomes
    (min{k : p_k >= b}, max{k : p_k <= e}) and disappears when no survivor lies inside it.
    Returns (K, V, index_map, new sent_off CSR, new sent_id)."""
    K_bits = _c(K_bits, np.uint16); V_bits = _c(V_bits, np.uint16)
    p = [t for t in range(len(tok_keep)) if tok_keep[t]]
    new_off = [0]; new_id = []
    for i in range(len(sent_off) - 1):
        b, e = int(sent_off[i]), int(sent_off[i + 1]) - 1
        if e < b:
            continue
        lo = [k for k, pk in enumerate(p) if pk >= b]
        hi = [k for k, pk in enumerate(p) if pk <= e]
        if not lo or not hi or min(lo) > max(hi):
            continue
        if min(lo) != new_off[-1]:
            raise AssertionError("remapped ranges are not contiguous")
        new_off.append(max(hi) + 1)
        new_id.append(int(sent_id[i]))
    idx = np.asarray(p, np.int64)
    return (K_bits[idx], V_bits[idx], idx.astype(np.int32), np.asarray(new_off, np.int32),
            np.asarray(new_id, np.int32))


# ------------------------------------------------------------------ token-level redundancy
def token_redundancy(K_bits, eps=1e-6):
    """O14  Token redundancy at token granularity (Section 4.1, token-redundancy equation):
    Kbar_t = K_t / (|K_t|_2 + eps), G = Kbar Kbar^T, R = column mean of the row softmax of G with the
    diagonal excluded -- O2 with every token its own sentence, followed by O3.  K_bits uint16 [N, d].
    Returns R float64 [N]."""
    K_bits = _c(K_bits, np.uint16)
    N = K_bits.shape[0]
    _, kbar = pool(K_bits, np.arange(N + 1, dtype=np.int32), np.zeros(N, np.float64), eps)
    _, red, _ = gram_terms(kbar, 2.0)
    return red


# ------------------------------------------------------------------ per-token range append
def append_token(sent_off, sent_id, new_sentence, gen_id):
    """O15  Pre-eviction update of the cache-space range list for one appended token (Algorithm 1;
    Section 4.1, "Updating Cache Ranges Before Eviction", Eq. "before" applied as soon as a token
    arrives, i.e. with no tokens generated since: the range of the sentence the token belongs to ends
    at the current cache length, and a new sentence begins right after the end of the previous one).
    The cache stays fully partitioned: the trailing, still open sentence is the last range.

    sent_off int32 [S+1] (CSR), sent_id int32 [S].  Returns the new (sent_off, sent_id)."""
    off = [int(x) for x in sent_off]; ids = [int(x) for x in sent_id]
    length = off[-1] if off else 0
    ranges = [(off[i], off[i + 1] - 1) for i in range(len(ids))]              # inclusive (b, e)
    if new_sentence or not ranges:
        b = ranges[-1][1] + 1 if ranges else 0                                # b_i = e_{i-1} + 1
        ranges.append((b, length))                                            # e_i = new length - 1
        ids.append(int(gen_id))
    else:
        ranges[-1] = (ranges[-1][0], length)
    new_off = [0] + [e + 1 for (_, e) in ranges]
    assert all(ranges[i][0] == new_off[i] for i in range(len(ranges)))        # still a partition
    return np.asarray(new_off, np.int32), np.asarray(ids, np.int32)


# ------------------------------------------------------------------ batch drivers
def score_batch(shape, K_bits, qwin_bits, kv_len, sent_off, n_sent, sigma, tau, eps, want_tok_imp=False):
    """shape: dict(batch,Hq,Hk,d,alpha,max_sent,slab_off,cap).  Returns dict of arrays."""
    b, Hq, Hk, d, alpha, ms = (shape[k] for k in ("batch", "Hq", "Hk", "d", "alpha", "max_sent"))
    slab_off = _c(shape["slab_off"], np.int64); cap = _c(shape["cap"], np.int32)
    K_bits = _c(K_bits, np.uint16); qwin_bits = _c(qwin_bits, np.uint16)
    kv_len = _c(kv_len, np.int32); sent_off = _c(sent_off, np.int32); n_sent = _c(n_sent, np.int32)
    ti = np.zeros(K_bits.shape[0], np.float64) if want_tok_imp else None
    imp = np.zeros((b, Hk, ms), np.float64); red = np.zeros_like(imp); lam = np.zeros_like(imp)
    sc = np.zeros((b, Hk, ms), np.float32)
    lib().oracle_score_batch(b, Hq, Hk, d, alpha, ms, _p(slab_off), _p(cap), _p(K_bits), _p(qwin_bits),
                             _p(kv_len), _p(sent_off), _p(n_sent), C.c_double(sigma), C.c_double(tau),
                             C.c_double(eps), _p(ti), _p(imp), _p(red), _p(lam), _p(sc))
    return dict(tok_imp=ti, imp=imp, red=red, lam=lam, score=sc)


def select_batch(score, sent_off, n_sent, budget, protect_tail):
    score = _c(score, np.float32); sent_off = _c(sent_off, np.int32); n_sent = _c(n_sent, np.int32)
    ms = score.shape[-1]
    ns = int(np.prod(score.shape[:-1]))
    keep = np.zeros(score.shape, np.uint8); kept = np.full(score.shape, -1, np.int32)
    nk = np.zeros(score.shape[:-1], np.int32); nl = np.zeros(score.shape[:-1], np.int32)
    lib().oracle_select_batch(ns, ms, _p(score), _p(sent_off), _p(n_sent), int(budget), int(protect_tail),
                              _p(keep), _p(kept), _p(nk), _p(nl))
    return dict(keep=keep, kept_idx=kept, n_kept=nk, new_len=nl)


def compact_batch(shape, K_bits, V_bits, keep, sent_off, sent_id, n_sent, kv_len, want_index_map=True):
    """Returns new copies: K, V, sent_off, sent_id, n_sent, kv_len, index_map."""
    b, Hk, d, ms = (shape[k] for k in ("batch", "Hk", "d", "max_sent"))
    slab_off = _c(shape["slab_off"], np.int64); cap = _c(shape["cap"], np.int32)
    K = _c(K_bits, np.uint16).copy(); V = _c(V_bits, np.uint16).copy()
    keep = _c(keep, np.uint8)
    so = _c(sent_off, np.int32).copy(); sid = _c(sent_id, np.int32).copy()
    ns = _c(n_sent, np.int32).copy(); kl = _c(kv_len, np.int32).copy()
    im = np.full(K.shape[0], -1, np.int32) if want_index_map else None
    rc = lib().oracle_compact_batch(b, Hk, d, ms, _p(slab_off), _p(cap), _p(K), _p(V), _p(keep), _p(so), _p(sid),
                                    _p(ns), _p(kl), _p(im))
    if rc != 0:
        raise AssertionError("literal range remap disagrees with the prefix-sum form")
    return dict(K=K, V=V, sent_off=so, sent_id=sid, n_sent=ns, kv_len=kl, index_map=im)


def decode_attn_batch(shape, q_bits, K_bits, V_bits, kv_len):
    b, Hq, Hk, d = (shape[k] for k in ("batch", "Hq", "Hk", "d"))
    slab_off = _c(shape["slab_off"], np.int64); cap = _c(shape["cap"], np.int32)
    q_bits = _c(q_bits, np.uint16); K_bits = _c(K_bits, np.uint16); V_bits = _c(V_bits, np.uint16)
    kv_len = _c(kv_len, np.int32)
    out = np.zeros((b, Hq, d), np.uint16); o64 = np.zeros((b, Hq, d), np.float64)
    lib().oracle_decode_attn_batch(b, Hq, Hk, d, _p(slab_off), _p(cap), _p(q_bits), _p(K_bits), _p(V_bits),
                                   _p(kv_len), _p(out), _p(o64))
    return out, o64
