"""Thin ctypes binding of the C-ABI CUDA library (``libskipkv.so``): argument marshalling only.

Every function has the name and argument order of its C counterpart in ``include/skipkv.h``
and takes ``torch`` CUDA tensors (used purely as device memory) whose ``data_ptr()`` is
passed through.  There is no CPU fallback: if the library has not been built, or a call
returns an error code, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libskipkv.so")
_lib = None

ERRORS = {-1: "SKIPKV_ERR_INVALID_ARG", -2: "SKIPKV_ERR_UNSUPPORTED", -3: "SKIPKV_ERR_WORKSPACE",
          -4: "SKIPKV_ERR_CUDA", -5: "SKIPKV_ERR_TIMEOUT"}
SYMBOLS = ["skipkv_workspace_bytes", "skipkv_workspace_init", "skipkv_status", "skipkv_last_cuda_error",
           "skipkv_score", "skipkv_select", "skipkv_compact", "skipkv_decode_attn", "skipkv_steer",
           "skipkv_append", "skipkv_decode_attn_static", "skipkv_table_step", "skipkv_score_table",
           "skipkv_select_fill", "skipkv_compact_fill", "skipkv_token_redundancy",
           "skipkv_append_step", "skipkv_decode_attn_paged",
           "skipkv_decode_step", "skipkv_set_wait_limit", "skipkv_wait_probe", "skipkv_select_fill_red",
           "skipkv_score_paged", "skipkv_compact_paged", "skipkv_decode_step_paged"]


class SkipKVError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        super().__init__(f"{where}: {ERRORS.get(code, code)} {detail}".strip())


class Shape(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("window", C.c_int32), ("d_model", C.c_int32),
                ("max_sent", C.c_int32), ("max_cap", C.c_int32), ("total_rows", C.c_int64),
                ("slab_off", C.c_void_p), ("cap", C.c_void_p)]


class Params(C.Structure):
    _fields_ = [("sigma", C.c_float), ("tau", C.c_float), ("eps", C.c_float),
                ("budget", C.c_int32), ("protect_tail", C.c_int32)]


def lib():
    """Load the CUDA library; fails loudly when it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2512_07993_b200.build` "
                               "(there is no CPU fallback)")
        _lib = C.CDLL(LIB_PATH)
        for name in SYMBOLS:
            getattr(_lib, name).restype = C.c_int
        _lib.skipkv_last_cuda_error.restype = C.c_char_p
    return _lib


def _ptr(t: Optional[torch.Tensor], dtype=None):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("device-resident contiguous tensor expected")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"expected {dtype}, got {t.dtype}")
    return C.c_void_p(t.data_ptr())


def _stream(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _check(rc: int, where: str):
    if rc != 0:
        detail = lib().skipkv_last_cuda_error().decode() if rc in (-4, -2) else ""
        raise SkipKVError(rc, where, detail)


def make_shape(batch, n_q_heads, n_kv_heads, head_dim, window, d_model, max_sent, max_cap,
               slab_off: Optional[torch.Tensor], cap: Optional[torch.Tensor], total_rows: Optional[int] = None) -> Shape:
    # total_rows must be the exact row count of the K / V buffers for skipkv_score (it bounds the tiled copies);
    # the default is an upper bound, enough for workspace sizing and for the calls that never tile K
    if total_rows is None:
        total_rows = batch * n_kv_heads * max_cap
    s = Shape(batch, n_q_heads, n_kv_heads, head_dim, window, d_model, max_sent, max_cap, total_rows,
              slab_off.data_ptr() if slab_off is not None else None,
              cap.data_ptr() if cap is not None else None)
    s._keepalive = (slab_off, cap)
    return s


def make_params(sigma=0.1, tau=0.95, eps=1e-6, budget=0, protect_tail=0) -> Params:
    return Params(sigma, tau, eps, budget, protect_tail)


def skipkv_workspace_bytes(shape: Shape) -> int:
    n = C.c_size_t(0)
    _check(lib().skipkv_workspace_bytes(C.byref(shape), C.byref(n)), "skipkv_workspace_bytes")
    return int(n.value)


def skipkv_workspace_init(shape: Shape, ws: torch.Tensor, stream=None) -> None:
    _check(lib().skipkv_workspace_init(C.byref(shape), _ptr(ws), _stream(stream)), "skipkv_workspace_init")


def skipkv_status(ws: torch.Tensor, stream=None, raise_on_error=True) -> int:
    bits = C.c_uint32(0)
    rc = lib().skipkv_status(_ptr(ws), _stream(stream), C.byref(bits))
    if rc != 0 and raise_on_error:
        raise SkipKVError(rc, "skipkv_status", f"status bits 0x{bits.value:x}")
    return int(bits.value)


def skipkv_score(shape, params, K, q_win, kv_len, sent_off, n_sent, tok_imp, sent_imp, sent_red, sent_lam,
                 sent_score, ws, stream=None) -> None:
    _check(lib().skipkv_score(C.byref(shape), C.byref(params), _ptr(K, torch.bfloat16), _ptr(q_win, torch.bfloat16),
                              _ptr(kv_len, torch.int32), _ptr(sent_off, torch.int32), _ptr(n_sent, torch.int32),
                              _ptr(tok_imp, torch.float32), _ptr(sent_imp, torch.float32),
                              _ptr(sent_red, torch.float32), _ptr(sent_lam, torch.float32),
                              _ptr(sent_score, torch.float32), _ptr(ws), _stream(stream)), "skipkv_score")


def skipkv_select(shape, params, sent_score, sent_off, n_sent, keep, kept_idx, n_kept, new_len, ws,
                  stream=None) -> None:
    _check(lib().skipkv_select(C.byref(shape), C.byref(params), _ptr(sent_score, torch.float32),
                               _ptr(sent_off, torch.int32), _ptr(n_sent, torch.int32), _ptr(keep, torch.uint8),
                               _ptr(kept_idx, torch.int32), _ptr(n_kept, torch.int32), _ptr(new_len, torch.int32),
                               _ptr(ws), _stream(stream)), "skipkv_select")


def skipkv_compact(shape, K, V, keep, sent_off, sent_id, n_sent, kv_len, index_map, ws, stream=None) -> None:
    _check(lib().skipkv_compact(C.byref(shape), _ptr(K, torch.bfloat16), _ptr(V, torch.bfloat16),
                                _ptr(keep, torch.uint8), _ptr(sent_off, torch.int32), _ptr(sent_id, torch.int32),
                                _ptr(n_sent, torch.int32), _ptr(kv_len, torch.int32), _ptr(index_map, torch.int32),
                                _ptr(ws), _stream(stream)), "skipkv_compact")


def skipkv_decode_attn(shape, q, K, V, kv_len, out, hidden, steer_vec, alpha, flag, ws, stream=None) -> None:
    _check(lib().skipkv_decode_attn(C.byref(shape), _ptr(q, torch.bfloat16), _ptr(K, torch.bfloat16),
                                    _ptr(V, torch.bfloat16), _ptr(kv_len, torch.int32), _ptr(out, torch.bfloat16),
                                    _ptr(hidden, torch.bfloat16), _ptr(steer_vec, torch.bfloat16),
                                    _ptr(alpha, torch.float32), _ptr(flag, torch.uint8), _ptr(ws),
                                    _stream(stream)), "skipkv_decode_attn")


def skipkv_set_wait_limit(ws, polls: int, stream=None) -> None:
    _check(lib().skipkv_set_wait_limit(_ptr(ws), C.c_uint32(polls), _stream(stream)), "skipkv_set_wait_limit")


def skipkv_wait_probe(ws, stream=None) -> None:
    _check(lib().skipkv_wait_probe(_ptr(ws), _stream(stream)), "skipkv_wait_probe")


def skipkv_steer(batch, d_model, hidden, steer_vec, alpha, flag, stream=None) -> None:
    _check(lib().skipkv_steer(C.c_int32(batch), C.c_int32(d_model), _ptr(hidden, torch.bfloat16),
                              _ptr(steer_vec, torch.bfloat16), _ptr(alpha, torch.float32), _ptr(flag, torch.uint8),
                              _stream(stream)), "skipkv_steer")


def skipkv_append(shape, K, V, k_new, v_new, kv_len, ws, stream=None) -> None:
    _check(lib().skipkv_append(C.byref(shape), _ptr(K, torch.bfloat16), _ptr(V, torch.bfloat16),
                               _ptr(k_new, torch.bfloat16), _ptr(v_new, torch.bfloat16), _ptr(kv_len, torch.int32),
                               _ptr(ws), _stream(stream)), "skipkv_append")


def skipkv_table_step(batch, d_model, max_gen_sent, hidden_last, flag, acc, acc_count, emb, n_gen_sent, closed,
                      lam_table, tau, eps, status=None, stream=None) -> None:
    _check(lib().skipkv_table_step(C.c_int32(batch), C.c_int32(d_model), C.c_int32(max_gen_sent),
                                   _ptr(hidden_last, torch.bfloat16), _ptr(flag, torch.uint8),
                                   _ptr(acc, torch.float32), _ptr(acc_count, torch.int32), _ptr(emb, torch.float32),
                                   _ptr(n_gen_sent, torch.int32), _ptr(closed, torch.int32),
                                   _ptr(lam_table, torch.float32), C.c_float(tau), C.c_float(eps),
                                   _ptr(status, torch.int32), _stream(stream)), "skipkv_table_step")


def skipkv_score_table(shape, params, K, q_win, kv_len, sent_off, sent_id, n_sent, lam_table, table_len, tok_imp,
                       sent_imp, sent_red, sent_lam, sent_score, ws, stream=None) -> None:
    _check(lib().skipkv_score_table(C.byref(shape), C.byref(params), _ptr(K, torch.bfloat16),
                                    _ptr(q_win, torch.bfloat16), _ptr(kv_len, torch.int32),
                                    _ptr(sent_off, torch.int32), _ptr(sent_id, torch.int32),
                                    _ptr(n_sent, torch.int32), _ptr(lam_table, torch.float32),
                                    C.c_int32(table_len), _ptr(tok_imp, torch.float32),
                                    _ptr(sent_imp, torch.float32), _ptr(sent_red, torch.float32),
                                    _ptr(sent_lam, torch.float32), _ptr(sent_score, torch.float32), _ptr(ws),
                                    _stream(stream)), "skipkv_score_table")


def skipkv_select_fill(shape, params, sent_score, tok_imp, sent_off, n_sent, keep, tok_keep, kept_idx, n_kept, new_len,
                       ws, stream=None) -> None:
    _check(lib().skipkv_select_fill(C.byref(shape), C.byref(params), _ptr(sent_score, torch.float32),
                                    _ptr(tok_imp, torch.float32), _ptr(sent_off, torch.int32),
                                    _ptr(n_sent, torch.int32), _ptr(keep, torch.uint8), _ptr(tok_keep, torch.uint8),
                                    _ptr(kept_idx, torch.int32), _ptr(n_kept, torch.int32),
                                    _ptr(new_len, torch.int32), _ptr(ws), _stream(stream)), "skipkv_select_fill")


def skipkv_select_fill_red(shape, params, sent_score, tok_imp, tok_red, sent_off, n_sent, keep, tok_keep, kept_idx,
                           n_kept, new_len, ws, stream=None) -> None:
    _check(lib().skipkv_select_fill_red(C.byref(shape), C.byref(params), _ptr(sent_score, torch.float32),
                                        _ptr(tok_imp, torch.float32), _ptr(tok_red, torch.float32),
                                        _ptr(sent_off, torch.int32), _ptr(n_sent, torch.int32), _ptr(keep, torch.uint8),
                                        _ptr(tok_keep, torch.uint8), _ptr(kept_idx, torch.int32),
                                        _ptr(n_kept, torch.int32), _ptr(new_len, torch.int32), _ptr(ws),
                                        _stream(stream)), "skipkv_select_fill_red")


def skipkv_compact_fill(shape, K, V, keep, tok_keep, sent_off, sent_id, n_sent, kv_len, index_map, ws,
                        stream=None) -> None:
    _check(lib().skipkv_compact_fill(C.byref(shape), _ptr(K, torch.bfloat16), _ptr(V, torch.bfloat16),
                                     _ptr(keep, torch.uint8), _ptr(tok_keep, torch.uint8),
                                     _ptr(sent_off, torch.int32), _ptr(sent_id, torch.int32),
                                     _ptr(n_sent, torch.int32), _ptr(kv_len, torch.int32),
                                     _ptr(index_map, torch.int32), _ptr(ws), _stream(stream)), "skipkv_compact_fill")


def skipkv_token_redundancy(shape, params, K, kv_len, tok_red, ws, stream=None) -> None:
    _check(lib().skipkv_token_redundancy(C.byref(shape), C.byref(params), _ptr(K, torch.bfloat16),
                                         _ptr(kv_len, torch.int32), _ptr(tok_red, torch.float32), _ptr(ws),
                                         _stream(stream)), "skipkv_token_redundancy")


def skipkv_append_step(shape, K, V, k_new, v_new, kv_len, sent_off, sent_id, n_sent, new_sent, gen_id, q_win, q, slot,
                       ws, stream=None) -> None:
    _check(lib().skipkv_append_step(C.byref(shape), _ptr(K, torch.bfloat16), _ptr(V, torch.bfloat16),
                                    _ptr(k_new, torch.bfloat16), _ptr(v_new, torch.bfloat16),
                                    _ptr(kv_len, torch.int32), _ptr(sent_off, torch.int32),
                                    _ptr(sent_id, torch.int32), _ptr(n_sent, torch.int32),
                                    _ptr(new_sent, torch.uint8), _ptr(gen_id, torch.int32),
                                    _ptr(q_win, torch.bfloat16), _ptr(q, torch.bfloat16), C.c_int32(slot), _ptr(ws),
                                    _stream(stream)), "skipkv_append_step")


def skipkv_decode_attn_paged(shape, q, K_pages, V_pages, block_table, max_pages, kv_len, out, hidden, steer_vec, alpha,
                             flag, ws, stream=None) -> None:
    _check(lib().skipkv_decode_attn_paged(C.byref(shape), _ptr(q, torch.bfloat16), _ptr(K_pages, torch.bfloat16),
                                          _ptr(V_pages, torch.bfloat16), _ptr(block_table, torch.int32),
                                          C.c_int32(max_pages), _ptr(kv_len, torch.int32), _ptr(out, torch.bfloat16),
                                          _ptr(hidden, torch.bfloat16), _ptr(steer_vec, torch.bfloat16),
                                          _ptr(alpha, torch.float32), _ptr(flag, torch.uint8), _ptr(ws),
                                          _stream(stream)), "skipkv_decode_attn_paged")


def skipkv_score_paged(shape, params, K_pages, block_table, max_pages, q_win, kv_len, sent_off, n_sent, tok_imp,
                       sent_imp, sent_red, sent_lam, sent_score, ws, stream=None) -> None:
    _check(lib().skipkv_score_paged(C.byref(shape), C.byref(params), _ptr(K_pages, torch.bfloat16),
                                    _ptr(block_table, torch.int32), C.c_int32(max_pages),
                                    _ptr(q_win, torch.bfloat16), _ptr(kv_len, torch.int32),
                                    _ptr(sent_off, torch.int32), _ptr(n_sent, torch.int32),
                                    _ptr(tok_imp, torch.float32), _ptr(sent_imp, torch.float32),
                                    _ptr(sent_red, torch.float32), _ptr(sent_lam, torch.float32),
                                    _ptr(sent_score, torch.float32), _ptr(ws), _stream(stream)),
           "skipkv_score_paged")


def skipkv_compact_paged(shape, K_pages, V_pages, block_table, max_pages, keep, sent_off, sent_id, n_sent, kv_len,
                         index_map, ws, stream=None) -> None:
    _check(lib().skipkv_compact_paged(C.byref(shape), _ptr(K_pages, torch.bfloat16), _ptr(V_pages, torch.bfloat16),
                                      _ptr(block_table, torch.int32), C.c_int32(max_pages),
                                      _ptr(keep, torch.uint8), _ptr(sent_off, torch.int32),
                                      _ptr(sent_id, torch.int32), _ptr(n_sent, torch.int32),
                                      _ptr(kv_len, torch.int32), _ptr(index_map, torch.int32), _ptr(ws),
                                      _stream(stream)), "skipkv_compact_paged")


def skipkv_decode_step_paged(shape, q, k_new, v_new, K_pages, V_pages, block_table, max_pages, kv_len_in, kv_len_out,
                             sent_off, sent_id, n_sent, new_sent, gen_id, q_win, slot, out, hidden, steer_vec, alpha,
                             flag, ws, stream=None) -> None:
    _check(lib().skipkv_decode_step_paged(C.byref(shape), _ptr(q, torch.bfloat16), _ptr(k_new, torch.bfloat16),
                                          _ptr(v_new, torch.bfloat16), _ptr(K_pages, torch.bfloat16),
                                          _ptr(V_pages, torch.bfloat16), _ptr(block_table, torch.int32),
                                          C.c_int32(max_pages), _ptr(kv_len_in, torch.int32),
                                          _ptr(kv_len_out, torch.int32), _ptr(sent_off, torch.int32),
                                          _ptr(sent_id, torch.int32), _ptr(n_sent, torch.int32),
                                          _ptr(new_sent, torch.uint8), _ptr(gen_id, torch.int32),
                                          _ptr(q_win, torch.bfloat16), C.c_int32(slot), _ptr(out, torch.bfloat16),
                                          _ptr(hidden, torch.bfloat16), _ptr(steer_vec, torch.bfloat16),
                                          _ptr(alpha, torch.float32), _ptr(flag, torch.uint8), _ptr(ws),
                                          _stream(stream)), "skipkv_decode_step_paged")


def skipkv_decode_step(shape, q, k_new, v_new, K, V, kv_len_in, kv_len_out, sent_off, sent_id, n_sent, new_sent, gen_id,
                       q_win, slot, out, hidden, steer_vec, alpha, flag, ws, stream=None) -> None:
    _check(lib().skipkv_decode_step(C.byref(shape), _ptr(q, torch.bfloat16), _ptr(k_new, torch.bfloat16),
                                    _ptr(v_new, torch.bfloat16), _ptr(K, torch.bfloat16), _ptr(V, torch.bfloat16),
                                    _ptr(kv_len_in, torch.int32), _ptr(kv_len_out, torch.int32),
                                    _ptr(sent_off, torch.int32), _ptr(sent_id, torch.int32),
                                    _ptr(n_sent, torch.int32), _ptr(new_sent, torch.uint8),
                                    _ptr(gen_id, torch.int32), _ptr(q_win, torch.bfloat16), C.c_int32(slot),
                                    _ptr(out, torch.bfloat16), _ptr(hidden, torch.bfloat16),
                                    _ptr(steer_vec, torch.bfloat16), _ptr(alpha, torch.float32),
                                    _ptr(flag, torch.uint8), _ptr(ws), _stream(stream)), "skipkv_decode_step")


def skipkv_decode_attn_static(shape, q, K, V, kv_len, out, hidden, steer_vec, alpha, flag, status=None,
                              stream=None) -> None:
    """Decode attention without a workspace: scratch is a fixed array inside the library.

    For callers that cannot allocate device memory.  ``status`` is an optional one-element
    uint32-sized (int32) device tensor that receives the status bits."""
    _check(lib().skipkv_decode_attn_static(C.byref(shape), _ptr(q, torch.bfloat16), _ptr(K, torch.bfloat16),
                                           _ptr(V, torch.bfloat16), _ptr(kv_len, torch.int32),
                                           _ptr(out, torch.bfloat16), _ptr(hidden, torch.bfloat16),
                                           _ptr(steer_vec, torch.bfloat16), _ptr(alpha, torch.float32),
                                           _ptr(flag, torch.uint8), _ptr(status, torch.int32), _stream(stream)),
           "skipkv_decode_attn_static")


class DeviceLayer:
    """Device copies of one ``workloads.make_layer`` result plus output buffers and workspace.

    Convenience for tests and the benchmark; it only moves tensors and allocates."""

    def __init__(self, layer: dict, device="cuda", params: Optional[Params] = None):
        cfg = layer["cfg"]
        dev = torch.device(device)
        self.cfg = cfg
        t = lambda a, dt=None: torch.as_tensor(a, dtype=dt).to(dev).contiguous()
        self.slab_off = t(layer["slab_off"], torch.int64)
        self.cap = t(layer["cap"], torch.int32)
        self.K = layer["K"].to(dev)
        self.V = layer["V"].to(dev)
        self.q_win = layer["q_win"].to(dev)
        self.q = layer["q"].to(dev)
        self.hidden = layer["hidden"].to(dev)
        self.steer_vec = layer["steer_vec"].to(dev)
        self.alpha = t(layer["alpha"], torch.float32)
        self.flag = t(layer["flag"], torch.uint8)
        self.kv_len = t(layer["kv_len"], torch.int32)
        self.sent_off = t(layer["sent_off"], torch.int32)
        self.sent_id = t(layer["sent_id"], torch.int32)
        self.n_sent = t(layer["n_sent"], torch.int32)
        ms = int(layer["max_sent"])
        self.max_sent = ms
        self.shape = make_shape(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.window, cfg.d_model,
                                ms, int(layer["cap"].max()), self.slab_off, self.cap, int(self.K.shape[0]))
        pt = cfg.window if cfg.protect_tail is None else cfg.protect_tail
        self.params = params or make_params(0.1, 0.95, 1e-6, cfg.budget, pt)
        bh = (cfg.batch, cfg.n_kv_heads)
        f32 = dict(dtype=torch.float32, device=dev)
        self.tok_imp = torch.zeros(self.K.shape[0], **f32)
        self.sent_imp = torch.zeros(*bh, ms, **f32)
        self.sent_red = torch.zeros(*bh, ms, **f32)
        self.sent_lam = torch.zeros(*bh, ms, **f32)
        self.sent_score = torch.zeros(*bh, ms, **f32)
        self.keep = torch.zeros(*bh, ms, dtype=torch.uint8, device=dev)
        self.kept_idx = torch.zeros(*bh, ms, dtype=torch.int32, device=dev)
        self.n_kept = torch.zeros(*bh, dtype=torch.int32, device=dev)
        self.new_len = torch.zeros(*bh, dtype=torch.int32, device=dev)
        self.index_map = torch.full((self.K.shape[0],), -1, dtype=torch.int32, device=dev)
        self.out = torch.zeros(cfg.batch, cfg.n_q_heads, cfg.head_dim, dtype=torch.bfloat16, device=dev)
        self.ws = torch.empty(skipkv_workspace_bytes(self.shape), dtype=torch.uint8, device=dev)
        skipkv_workspace_init(self.shape, self.ws)

    def score(self, stream=None):
        skipkv_score(self.shape, self.params, self.K, self.q_win, self.kv_len, self.sent_off, self.n_sent,
                     self.tok_imp, self.sent_imp, self.sent_red, self.sent_lam, self.sent_score, self.ws, stream)

    def select(self, stream=None):
        skipkv_select(self.shape, self.params, self.sent_score, self.sent_off, self.n_sent, self.keep,
                      self.kept_idx, self.n_kept, self.new_len, self.ws, stream)

    def compact(self, stream=None):
        skipkv_compact(self.shape, self.K, self.V, self.keep, self.sent_off, self.sent_id, self.n_sent,
                       self.kv_len, self.index_map, self.ws, stream)

    def decode_attn(self, steer=True, stream=None):
        skipkv_decode_attn(self.shape, self.q, self.K, self.V, self.kv_len, self.out,
                           self.hidden if steer else None, self.steer_vec, self.alpha, self.flag, self.ws, stream)

    def status(self):
        return skipkv_status(self.ws)
