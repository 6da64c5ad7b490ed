"""Seeded synthetic workloads for the SkipKV eviction / decode hot path.

This module only *draws inputs*: sentence lengths, near-duplicate structure, bf16
K/V/Q tensors, the steering vector and the ragged slab layout.  It holds none of the
method's arithmetic (no scoring, selection, compaction or attention), so that both the
CPU oracle's tests and the CUDA path's tests can be fed from it without sharing any
code of the method itself.

Layout produced (the layout the C-ABI library consumes):

* ``K``/``V``: one bf16 buffer per layer, shape ``[total_rows, head_dim]``.  Sequence
  ``b`` owns rows ``[slab_off[b]*Hk, (slab_off[b]+cap[b])*Hk)``; inside it KV head ``h``
  owns ``cap[b]`` consecutive rows, of which the first ``kv_len[b,h]`` are live.
* sentence tables per (b, h): ``sent_off[b,h,0..n_sent]`` (token offsets, CSR),
  ``sent_id[b,h,:]`` (generation-space sentence index) and ``n_sent[b,h]``.

Every value is a pure function of ``(cfg.seed, layer, sequence, stream kind)`` through
numpy's counter-based Philox generator, so any single sequence of any layer can be
regenerated on its own.
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass
from typing import Dict, List, Optional

import numpy as np
import torch

# stream kinds (sub-keys of the Philox seed sequence)
_K_STRUCT, _K_KEYS, _K_VALS, _K_NOISE, _K_QWIN, _K_QDEC, _K_HID, _K_STEER, _K_LENS, _K_MISC, _K_GEN, _K_GENNOISE = range(12)


@dataclass(frozen=True)
class Workload:
    """Shape and distribution of one synthetic configuration."""
    name: str
    seed: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    window: int            # observation window (number of recent queries)
    d_model: int
    budget: int            # KV budget B in tokens
    ctx_lo: int            # cached tokens per sequence, uniform in [ctx_lo, ctx_hi]
    ctx_hi: int
    sent_lo: int
    sent_hi: int
    sent_dist: str         # "uniform" | "geometric"
    geo_mean_extra: float  # geometric: mean of the part added to sent_lo
    dup_rate: float        # fraction of sentences that are noisy copies of an earlier one
    dup_noise: float       # std of the noise added to the copied keys
    layers: int = 1
    dup_rate_hi: Optional[float] = None   # if set, dup rate varies linearly over layers
    cap_extra: int = 0     # spare rows per (sequence, head) beyond the cached tokens
    protect_tail: Optional[int] = None    # defaults to the window

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    def dup_rate_at(self, layer: int) -> float:
        if self.dup_rate_hi is None or self.layers <= 1:
            return self.dup_rate
        return self.dup_rate + (self.dup_rate_hi - self.dup_rate) * layer / (self.layers - 1)


def config(index: int, **over) -> Workload:
    """The five benchmark configurations (index 1..5) plus 0 = a very small smoke case."""
    base = {
        0: Workload("smoke", 1000, 2, 8, 2, 128, 8, 256, 96, 300, 420, 4, 24, "uniform", 0.0,
                    0.25, 0.05),
        1: Workload("tiny", 1001, 1, 32, 8, 128, 32, 4096, 512, 2048, 2048, 8, 64, "uniform",
                    0.0, 0.25, 0.05),
        2: Workload("llama8b-32k-b10", 1002, 10, 32, 8, 128, 32, 4096, 4096, 16384, 32768, 8, 96,
                    "uniform", 0.0, 0.30, 0.05),
        3: Workload("llama8b-32k-b10-32layers", 1003, 10, 32, 8, 128, 32, 4096, 4096, 16384,
                    32768, 8, 96, "uniform", 0.0, 0.10, 0.05, layers=32, dup_rate_hi=0.50),
        4: Workload("decode-loop", 1004, 10, 32, 8, 128, 32, 4096, 2048, 8192, 8192, 8, 96,
                    "uniform", 0.0, 0.20, 0.05, layers=32, cap_extra=256),
        5: Workload("qwen14b-64k-b16", 1005, 16, 40, 8, 128, 64, 5120, 8192, 32768, 65536, 4, 128,
                    "geometric", 20.0, 0.40, 0.05, layers=48),
    }[index]
    return dataclasses.replace(base, **over) if over else base


def _rng(seed: int, layer: int, seq: int, kind: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(np.random.SeedSequence([seed, layer, seq, kind])))


def to_bf16(x: np.ndarray) -> torch.Tensor:
    """float32 numpy -> torch bf16 (round to nearest even)."""
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """torch bf16 tensor -> numpy uint16 view of the raw bits (no copy)."""
    assert t.dtype == torch.bfloat16
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_bf16(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)


def draw_context_lengths(cfg: Workload) -> np.ndarray:
    r = _rng(cfg.seed, 0, 0, _K_LENS)
    return r.integers(cfg.ctx_lo, cfg.ctx_hi + 1, size=cfg.batch).astype(np.int64)


def draw_sentences(cfg: Workload, layer: int, seq: int, n_tokens: int, per_layer: bool = False):
    """Sentence lengths and near-duplicate sources for one sequence.

    Returns ``(lengths int32[S], dup_src int32[S])``; ``dup_src[i] = -1`` for a fresh
    sentence, else the index of the earlier sentence it copies (it takes that
    sentence's length).  The last sentence is cut so the lengths sum to ``n_tokens``.
    """
    r = _rng(cfg.seed, layer if per_layer else 0, seq, _K_STRUCT)
    rate = cfg.dup_rate_at(layer)
    lengths: List[int] = []
    src: List[int] = []
    total = 0
    while total < n_tokens:
        i = len(lengths)
        is_dup = i > 0 and r.random() < rate
        if is_dup:
            s = int(r.integers(0, i))
            ln = lengths[s]
        else:
            s = -1
            if cfg.sent_dist == "uniform":
                ln = int(r.integers(cfg.sent_lo, cfg.sent_hi + 1))
            else:  # long-tailed: sent_lo + geometric, clipped
                p = 1.0 / (cfg.geo_mean_extra + 1.0)
                ln = int(min(cfg.sent_hi, cfg.sent_lo + (r.geometric(p) - 1)))
        if total + ln > n_tokens:      # ragged tail: a fresh, shorter sentence
            ln = n_tokens - total
            s = -1
        lengths.append(ln)
        src.append(s)
        total += ln
    return np.asarray(lengths, np.int32), np.asarray(src, np.int32)


def _draw_keys(cfg: Workload, layer: int, seq: int, lengths, dup_src) -> torch.Tensor:
    """bf16 keys ``[Hk, N, d]``: N(0,1), duplicate sentences = source + N(0, noise)."""
    n = int(lengths.sum())
    hk, d = cfg.n_kv_heads, cfg.head_dim
    k = to_bf16(_rng(cfg.seed, layer, seq, _K_KEYS).standard_normal((hk, n, d), dtype=np.float32))
    if (dup_src >= 0).any():
        z = _rng(cfg.seed, layer, seq, _K_NOISE)
        off = np.concatenate([[0], np.cumsum(lengths)])
        for i in np.nonzero(dup_src >= 0)[0]:       # ascending, so chains of copies resolve
            s = int(dup_src[i])
            ln = int(lengths[i])
            noise = torch.from_numpy(z.standard_normal((hk, ln, d), dtype=np.float32))
            srcrows = k[:, off[s]:off[s] + ln, :].float()
            k[:, off[i]:off[i] + ln, :] = (srcrows + cfg.dup_noise * noise).to(torch.bfloat16)
    return k


def make_layer(cfg: Workload, layer: int = 0, ctx: Optional[np.ndarray] = None,
               per_layer_sentences: bool = False) -> Dict[str, object]:
    """All inputs of one layer of ``cfg`` as host tensors in the library's layout."""
    hk, hq, d = cfg.n_kv_heads, cfg.n_q_heads, cfg.head_dim
    ctx = draw_context_lengths(cfg) if ctx is None else np.asarray(ctx, np.int64)
    cap = (ctx + cfg.cap_extra).astype(np.int32)
    slab_off = np.concatenate([[0], np.cumsum(cap.astype(np.int64))[:-1]]).astype(np.int64)
    total_rows = int(cap.astype(np.int64).sum()) * hk
    K = torch.zeros((total_rows, d), dtype=torch.bfloat16)
    V = torch.zeros((total_rows, d), dtype=torch.bfloat16)
    sents = [draw_sentences(cfg, layer, b, int(ctx[b]), per_layer_sentences) for b in range(cfg.batch)]
    max_sent = max(len(s[0]) for s in sents)
    sent_off = np.zeros((cfg.batch, hk, max_sent + 1), np.int32)
    sent_id = np.full((cfg.batch, hk, max_sent), -1, np.int32)
    n_sent = np.zeros((cfg.batch, hk), np.int32)
    kv_len = np.zeros((cfg.batch, hk), np.int32)
    dup_src_all = []
    for b in range(cfg.batch):
        lengths, dup_src = sents[b]
        n = int(ctx[b])
        kb = _draw_keys(cfg, layer, b, lengths, dup_src)
        vb = to_bf16(_rng(cfg.seed, layer, b, _K_VALS).standard_normal((hk, n, d), dtype=np.float32))
        for h in range(hk):
            r0 = int(slab_off[b]) * hk + h * int(cap[b])
            K[r0:r0 + n] = kb[h]
            V[r0:r0 + n] = vb[h]
        s = len(lengths)
        off = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
        sent_off[b, :, :s + 1] = off
        sent_off[b, :, s + 1:] = off[-1]
        sent_id[b, :, :s] = np.arange(s, dtype=np.int32)
        n_sent[b, :] = s
        kv_len[b, :] = n
        dup_src_all.append(dup_src)
    q_win = to_bf16(_rng(cfg.seed, layer, 0, _K_QWIN).standard_normal(
        (cfg.batch, hq, cfg.window, d), dtype=np.float32))
    q = to_bf16(_rng(cfg.seed, layer, 0, _K_QDEC).standard_normal((cfg.batch, hq, d), dtype=np.float32))
    hidden = to_bf16(_rng(cfg.seed, layer, 0, _K_HID).standard_normal((cfg.batch, cfg.d_model),
                                                                        dtype=np.float32))
    steer_vec = to_bf16(0.01 * _rng(cfg.seed, 0, 0, _K_STEER).standard_normal(cfg.d_model,
                                                                               dtype=np.float32))
    m = _rng(cfg.seed, layer, 0, _K_MISC)
    alpha = (1.0 + 0.02 * m.integers(0, 40, size=cfg.batch)).astype(np.float32)
    flag = (m.random(cfg.batch) < 0.6).astype(np.uint8)
    if cfg.batch >= 1:
        flag[0] = 1
    return dict(cfg=cfg, layer=layer, ctx=ctx, cap=cap, slab_off=slab_off, K=K, V=V,
                sent_off=sent_off, sent_id=sent_id, n_sent=n_sent, kv_len=kv_len,
                max_sent=max_sent, q_win=q_win, q=q, hidden=hidden, steer_vec=steer_vec,
                alpha=alpha, flag=flag, dup_src=dup_src_all)


def slab_rows(layer: Dict[str, object], b: int, h: int) -> slice:
    """Row range of (sequence b, KV head h) inside the layer's K / V buffers."""
    cfg = layer["cfg"]
    r0 = int(layer["slab_off"][b]) * cfg.n_kv_heads + h * int(layer["cap"][b])
    return slice(r0, r0 + int(layer["cap"][b]))


def make_generation(cfg: Workload, steps: int, d_model: Optional[int] = None, noise_hi: float = 0.6) -> Dict[str, object]:
    """Last-layer hidden states of ``steps`` generated tokens per sequence, with sentence structure.

    Sentences are drawn as for the cache (same length distribution and duplicate rate).  Tokens of a fresh
    sentence are N(0,1); a duplicate sentence is its source plus N(0, s^2) noise with s uniform in
    [0, noise_hi], so that the cosine of the two sentence means, about 1/sqrt(1+s^2), falls on both sides
    of the usual threshold.  The last sentence of every even sequence is left open (no closing delimiter).
    Returns H bf16 ``[batch, steps, d_model]``, flag uint8 ``[steps, batch]`` (1 = the token closes a
    sentence) and gen_off (per sequence, int32 CSR ranges of the closed sentences).
    """
    dm = cfg.d_model if d_model is None else d_model
    H = torch.zeros((cfg.batch, steps, dm), dtype=torch.bfloat16)
    flag = np.zeros((steps, cfg.batch), np.uint8)
    gen_off = []
    for b in range(cfg.batch):
        lengths, dup_src = draw_sentences(cfg, 0, b, steps)
        off = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
        h = to_bf16(_rng(cfg.seed, 0, b, _K_GEN).standard_normal((steps, dm), dtype=np.float32))
        z = _rng(cfg.seed, 0, b, _K_GENNOISE)
        for i in np.nonzero(dup_src >= 0)[0]:
            s0, ln = int(dup_src[i]), int(lengths[i])
            sd = float(z.uniform(0.0, noise_hi))
            noise = torch.from_numpy(z.standard_normal((ln, dm), dtype=np.float32))
            h[off[i]:off[i] + ln] = (h[off[s0]:off[s0] + ln].float() + sd * noise).to(torch.bfloat16)
        H[b] = h
        n_closed = len(lengths) - (1 if b % 2 == 0 else 0)
        flag[off[1:n_closed + 1] - 1, b] = 1
        gen_off.append(off[:n_closed + 1].copy())
    return dict(H=H, flag=flag, gen_off=gen_off, d_model=dm, steps=steps)
