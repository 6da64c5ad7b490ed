#!/usr/bin/env python
"""Benchmark of the SkipKV hot path on B200: one step = score + select + compact + decode
attention (with the fused steering add) over one layer of the Llama-8B-shaped workload
(batch 10, 8 KV / 32 query heads, head_dim 128, ragged 16K-32K cached tokens, budget 4096).

    python bench.py --gpus N --steps K --warmup W          # this library (CUDA path)
    python bench.py --impl reference ...                   # the CPU oracle on the host cores

Prints ONE JSON line.  `value` is the eviction time (score+select+compact) per layer in
microseconds with inputs resident in HBM; the decode-attention bandwidth and the per-step
rooflines ride along in the same line.  A step runs every leg over `--layers` independently
seeded layers back to back (the order of a multi-layer eviction pass and of a decode step), so
no launch finds its K/V in L2 and a leg's time divided by the layer count is the average launch.  With N > 1 every rank runs an independent replica of
the workload (the path has no exchange step); the time is the max over ranks and the value is
that time divided by the N layers processed.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2512_07993_b200 import workloads as W  # noqa: E402

METRIC = "SkipKV compress+compact µs/layer and decode-attn HBM GB/s, 32K ctx, batch 10"
UNIT = "us/layer (score+select+compact); decode-attn GB/s in decode_attn_gbs"
LAUNCHES_PER_STEP = {"score": 5, "select": 1, "compact": 2, "decode_attn": 1, "decode_attn_full_ctx": 1}   # kernels per layer


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d.get("bf16_tflops", 0.0)), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, source="fallback")


def ncu_traffic():
    """DRAM bytes per launch from the committed ncu summaries (None when not captured)."""
    p = os.path.join(ROOT, "profiles", "dram_traffic.json")
    return json.load(open(p)) if os.path.exists(p) else {}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.lines, self.proc = index, [], None

    def start(self):
        self.t_start = time.time()
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "100"], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return None
        if self.proc.poll() is None:
            time.sleep(0.15)
            self.proc.terminate()
        sm, mx, reasons = [], [], set()
        for ts, line in self.lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9 or not (t0 - 0.1 <= ts <= t1 + 0.2):
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return None
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm),
                "window": "warm-up + timed region" if t0 < self.t_start + 1e-3 else "timed region"}


def max_over_ranks(values, dist, device):
    """Element-wise maximum of a list of floats over all ranks (the replicas are independent: the slowest one
    defines the job's time); identity without a process group."""
    if dist is None:
        return list(values)
    tt = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return tt.tolist()


def replica_value(per_replica_us, world):
    """Whole-job value for `world` independent replicas that each process one layer per per_replica_us:
    microseconds per layer of the job = slowest replica's time / layers processed concurrently."""
    return per_replica_us / world


def oracle_shape(L):
    cfg = L["cfg"]
    return dict(batch=cfg.batch, Hq=cfg.n_q_heads, Hk=cfg.n_kv_heads, d=cfg.head_dim, alpha=cfg.window,
                max_sent=L["max_sent"], slab_off=L["slab_off"], cap=L["cap"])


def sub_layer(L, n_seq):
    """The first n_seq sequences of a layer as a layer of their own (views, no arithmetic)."""
    cfg = L["cfg"]
    import dataclasses
    rows = int((L["slab_off"][n_seq - 1] + L["cap"][n_seq - 1]) * cfg.n_kv_heads)
    out = dict(L)
    out["cfg"] = dataclasses.replace(cfg, batch=n_seq)
    for k in ("cap", "slab_off", "sent_off", "sent_id", "n_sent", "kv_len", "q_win", "q", "hidden", "alpha", "flag", "ctx"):
        out[k] = L[k][:n_seq]
    out["K"], out["V"] = L["K"][:rows], L["V"][:rows]
    return out


def time_oracle(L, n_seq=None, threads=None):
    """One pass of the whole path by the CPU oracle over the layer (or its first n_seq sequences) with the given
    number of threads (default: all); seconds per leg, the fraction of the layer's tokens covered, threads at work."""
    import oracle
    S = sub_layer(L, n_seq) if n_seq else L
    cfg = S["cfg"]
    sh = oracle_shape(S)
    Kb, Vb = W.bf16_bits(S["K"]), W.bf16_bits(S["V"])
    all_threads = oracle.max_threads()
    oracle.set_threads(threads or all_threads)
    try:
        t = [time.perf_counter()]
        sc = oracle.score_batch(sh, Kb, W.bf16_bits(S["q_win"]), S["kv_len"], S["sent_off"], S["n_sent"],
                                float(np.float32(0.1)), float(np.float32(0.95)), float(np.float32(1e-6)))
        t.append(time.perf_counter())
        sel = oracle.select_batch(sc["score"], S["sent_off"], S["n_sent"], cfg.budget, cfg.window)
        t.append(time.perf_counter())
        cp = oracle.compact_batch(sh, Kb, Vb, sel["keep"], S["sent_off"], S["sent_id"], S["n_sent"], S["kv_len"])
        t.append(time.perf_counter())
        oracle.decode_attn_batch(sh, W.bf16_bits(S["q"]), cp["K"], cp["V"], cp["kv_len"])
        oracle.steer(W.bf16_bits(S["hidden"]), W.bf16_bits(S["steer_vec"]), S["alpha"], S["flag"])
        t.append(time.perf_counter())
    finally:
        oracle.set_threads(all_threads)
    legs = dict(zip(("score", "select", "compact", "decode_attn"), np.diff(t)))
    frac = float(S["kv_len"].sum()) / float(L["kv_len"].sum())
    # the oracle's only parallel loop runs over the (sequence, head) slabs: that many threads can be busy at most
    busy = min(threads or all_threads, cfg.batch * cfg.n_kv_heads)
    return legs, frac, busy


def workload_config(cfg, config_index, tokens_before, tokens_after, layers_per_step, replicas):
    """The `config` object of the JSON line; both arms print the same keys for the same workload."""
    return {"workload": f"configs[{config_index - 1}]: {cfg.name}", "batch": cfg.batch, "kv_heads": cfg.n_kv_heads,
            "q_heads": cfg.n_q_heads, "head_dim": cfg.head_dim, "window": cfg.window, "budget": cfg.budget,
            "tokens_before": tokens_before, "tokens_after": tokens_after, "layers_per_step": layers_per_step,
            "order": "each leg (score, select, compact, decode) runs over all layers back to back; "
                     "per-layer time = leg time / layers",
            "l2": "256 MiB written then 256 MiB read between iterations; each layer's inputs (1 GB) exceed L2",
            "replicas": replicas}


def run_reference(args, rank):
    """The CPU oracle as the reference arm (rank 0 only): every step is one pass of the whole path over one full layer
    of the workload with all host threads, timed by the wall clock; nothing is sampled or scaled."""
    if rank != 0:
        return
    import oracle
    cfg = W.config(args.config)
    L = W.make_layer(cfg)
    sh = oracle_shape(L)
    times = []
    for i in range(args.warmup + args.steps):
        legs, frac, cores = time_oracle(L)
        if i >= args.warmup:
            times.append(legs)
    evict_us = statistics.mean((x["score"] + x["select"] + x["compact"]) for x in times) * 1e6
    dec_s = statistics.mean(x["decode_attn"] for x in times)
    step_ms = statistics.mean(sum(x.values()) for x in times) * 1e3
    # the kept-token count comes from the oracle's own selection
    sc = oracle.score_batch(sh, W.bf16_bits(L["K"]), W.bf16_bits(L["q_win"]), L["kv_len"], L["sent_off"], L["n_sent"],
                            float(np.float32(0.1)), float(np.float32(0.95)), float(np.float32(1e-6)))
    sel = oracle.select_batch(sc["score"], L["sent_off"], L["n_sent"], cfg.budget, cfg.window)
    sample = "one full layer per step, all sequences, no scaling"
    line = {"impl": "reference", "metric": METRIC, "value": evict_us, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(cfg, args.config, int(L["kv_len"].sum() // cfg.n_kv_heads),
                                      int(sel["new_len"].sum() // cfg.n_kv_heads), 1, 1),
            "decode_attn_us": dec_s * 1e6,
            "cpu_baseline": {"value": evict_us, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                             "host_cores": os.cpu_count()},
            "e2e": {"value": evict_us, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def time_extras(cfg, B, flush, clean, peaks, reps=10):
    """CUDA-event times (median, L2 flushed before every call) of the entry points beside the main path."""
    def timed(fn, before=lambda: None):
        ts = []
        for _ in range(reps):
            before()
            flush.fill_(1); clean.sum()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) * 1e3)
        return statistics.median(ts[3:])

    out = {}
    dev = "cuda"
    # lookup-table step: every sequence closes a sentence that is compared with n_prev earlier ones
    bt, dm, mg, n_prev = cfg.batch, cfg.d_model, 2048, 1300
    emb = torch.randn(bt, mg, dm, device=dev); emb /= emb.norm(dim=-1, keepdim=True)
    acc = torch.zeros(bt, dm, device=dev); cnt = torch.zeros(bt, dtype=torch.int32, device=dev)
    T = torch.zeros(bt, mg, device=dev); closed = torch.zeros(bt, dtype=torch.int32, device=dev)
    h = torch.randn(bt, dm, device=dev).bfloat16(); flag = torch.ones(bt, dtype=torch.uint8, device=dev)
    n = torch.empty(bt, dtype=torch.int32, device=dev)
    us = timed(lambda: B.skipkv_table_step(bt, dm, mg, h, flag, acc, cnt, emb, n, closed, T, 0.95, 1e-6),
               before=lambda: n.fill_(n_prev))
    byt = bt * n_prev * dm * 4
    out["table_step"] = {"us": us, "earlier_sentences": n_prev, "d_model": dm, "algorithmic_bytes": byt,
                         "bound": "hbm", "achieved": byt / us / 1e3, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": byt / us / 1e3 / peaks["hbm_gbs"]}
    del emb
    # exactly-B variants on one layer of the workload, beside the plain calls timed the same way
    L = W.make_layer(cfg)
    D = B.DeviceLayer(L)
    tok_keep = torch.zeros(D.K.shape[0], dtype=torch.uint8, device=dev)
    keys = ("K", "V", "sent_off", "sent_id", "n_sent", "kv_len")
    pristine = {k: getattr(D, k).clone() for k in keys}
    def restore():
        for k, v in pristine.items():
            getattr(D, k).copy_(v)
    select_fill = lambda: B.skipkv_select_fill(D.shape, D.params, D.sent_score, D.tok_imp, D.sent_off, D.n_sent, D.keep,
                                               tok_keep, D.kept_idx, D.n_kept, D.new_len, D.ws)
    compact_fill = lambda: B.skipkv_compact_fill(D.shape, D.K, D.V, D.keep, tok_keep, D.sent_off, D.sent_id, D.n_sent,
                                                 D.kv_len, D.index_map, D.ws)
    D.score()
    out["select_us"] = timed(D.select, restore)
    out["select_fill_us"] = timed(select_fill, restore)
    restore(); D.select()
    out["compact_us"] = timed(D.compact, restore)
    restore(); select_fill()
    out["compact_fill_us"] = timed(compact_fill, restore)
    # decode attention over the cache just compacted (exactly B rows per slab): contiguous slabs against the same
    # number of rows behind a shuffled block table (page contents do not matter for the time)
    slabs = cfg.batch * cfg.n_kv_heads
    max_pages = (int(D.kv_len.max().item()) + 127) // 128
    pool_pages = slabs * max_pages
    Kp = torch.randn(pool_pages * 128, 128, device=dev).bfloat16(); Vp = torch.randn(pool_pages * 128, 128, device=dev).bfloat16()
    table = torch.randperm(pool_pages, device=dev).to(torch.int32).reshape(cfg.batch, cfg.n_kv_heads, max_pages).contiguous()
    out["decode_attn_us"] = timed(lambda: D.decode_attn(steer=True))
    out["decode_attn_paged_us"] = timed(lambda: B.skipkv_decode_attn_paged(
        D.shape, D.q, Kp, Vp, table, max_pages, D.kv_len, D.out, D.hidden, D.steer_vec, D.alpha, D.flag, D.ws))
    D.status()
    del Kp, Vp
    del D, pristine, tok_keep
    torch.cuda.empty_cache()
    # one decode step of the decode-loop workload (cache a little above its budget of 2048): two launches against one
    cfg4 = W.config(4, ctx_lo=2112, ctx_hi=2112, batch=cfg.batch)
    D = B.DeviceLayer(W.make_layer(cfg4))
    k_new = torch.randn(cfg4.batch, cfg4.n_kv_heads, 128, device=dev).bfloat16(); v_new = torch.randn_like(k_new)
    zeros8 = torch.zeros(cfg4.batch, dtype=torch.uint8, device=dev); gen = torch.zeros(cfg4.batch, dtype=torch.int32, device=dev)
    kv_in, kv_out = D.kv_len.clone(), torch.zeros_like(D.kv_len)
    def two_launches():
        D.kv_len.copy_(kv_in)
        B.skipkv_append_step(D.shape, D.K, D.V, k_new, v_new, D.kv_len, D.sent_off, D.sent_id, D.n_sent, zeros8, gen, D.q_win,
                             D.q, 0, D.ws)
        D.decode_attn(steer=True)
    def one_launch():
        B.skipkv_decode_step(D.shape, D.q, k_new, v_new, D.K, D.V, kv_in, kv_out, D.sent_off, D.sent_id, D.n_sent, zeros8, gen,
                             D.q_win, 0, D.out, D.hidden, D.steer_vec, D.alpha, D.flag, D.ws)
    out["decode_step_two_launches_us"] = timed(two_launches)
    out["decode_step_fused_us"] = timed(one_launch)
    D.status()
    del D
    torch.cuda.empty_cache()
    # the decode loop itself (Algorithm 2): fused steps over a few layers, one sentence opened every 16 tokens, an eviction
    # pass (score, select, compact on every layer) every 128 steps; event times, the host loop's gaps included
    n_layers, steps, interval = 4, 256, 128
    cfgl = W.config(4, ctx_lo=2048, ctx_hi=2048, batch=cfg.batch)
    Ds = []
    for l in range(n_layers):
        Ll = W.make_layer(cfgl, layer=l)
        ms = int(Ll["max_sent"]) + steps                    # room for the sentences the loop opens
        for key in ("sent_off", "sent_id"):
            old = Ll[key]
            new = np.zeros(old.shape[:2] + (ms + (1 if key == "sent_off" else 0),), np.int32)
            new[..., :old.shape[2]] = old
            new[..., old.shape[2]:] = old[..., -1:] if key == "sent_off" else -1
            Ll[key] = new
        Ll["max_sent"] = ms
        Ds.append(B.DeviceLayer(Ll))
    other = [torch.zeros_like(D.kv_len) for D in Ds]
    k_new = torch.randn(cfgl.batch, cfgl.n_kv_heads, 128, device=dev).bfloat16(); v_new = torch.randn_like(k_new)
    opens = [torch.full((cfgl.batch,), 1 if t % 16 == 0 else 0, dtype=torch.uint8, device=dev) for t in range(2)]
    gen = torch.zeros(cfgl.batch, dtype=torch.int32, device=dev)
    ev = lambda: torch.cuda.Event(enable_timing=True)
    t_step, t_evict, n_evict = 0.0, 0.0, 0
    marks = []
    e_prev = ev(); e_prev.record()
    for t in range(steps):
        for l, D in enumerate(Ds):
            B.skipkv_decode_step(D.shape, D.q, k_new, v_new, D.K, D.V, D.kv_len, other[l], D.sent_off, D.sent_id, D.n_sent,
                                 opens[1 if t % 16 else 0], gen, D.q_win, t % cfgl.window, D.out, D.hidden, D.steer_vec,
                                 D.alpha, D.flag, D.ws)
            D.kv_len, other[l] = other[l], D.kv_len
        if (t + 1) % interval == 0:
            e0 = ev(); e0.record()
            for D in Ds:
                D.score(); D.select(); D.compact()
            e1 = ev(); e1.record()
            marks.append((e_prev, e0, e1))
            e_prev = e1
    e_end = ev(); e_end.record()
    torch.cuda.synchronize()
    for a0, b0, c0 in marks:
        t_step += a0.elapsed_time(b0); t_evict += b0.elapsed_time(c0); n_evict += 1
    t_step += e_prev.elapsed_time(e_end)
    for D in Ds:
        D.status()
    out["decode_loop"] = {"layers": n_layers, "steps": steps, "evictions": n_evict, "rows_per_slab": "2048 .. 2176",
                          "us_per_layer_step": t_step * 1e3 / (steps * n_layers),
                          "us_per_layer_eviction": t_evict * 1e3 / max(n_evict * n_layers, 1),
                          "note": "CUDA events around a Python loop of C-ABI calls: launch gaps of the host loop included"}
    del Ds, other
    torch.cuda.empty_cache()
    # token-level redundancy at the steady-state length of a budgeted cache: budget + 128 rows per slab
    n_tok = cfg.budget + 128
    cfg_ss = W.config(0, batch=cfg.batch, n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads, window=cfg.window,
                      d_model=cfg.d_model, budget=cfg.budget, ctx_lo=n_tok, ctx_hi=n_tok, sent_lo=cfg.sent_lo,
                      sent_hi=cfg.sent_hi, seed=cfg.seed)
    D = B.DeviceLayer(W.make_layer(cfg_ss))
    red = torch.zeros(D.K.shape[0], dtype=torch.float32, device=dev)
    us = timed(lambda: B.skipkv_token_redundancy(D.shape, D.params, D.K, D.kv_len, red, D.ws))
    D.status()
    nb = (n_tok + 127) // 128
    tiles = nb * (nb + 1) // 2                                              # every pair of 128-row blocks once (G is symmetric)
    exps = cfg.batch * cfg.n_kv_heads * float(tiles) * 128 * 128 * 2        # exponentials evaluated over both passes
    elems = cfg.batch * cfg.n_kv_heads * float(n_tok) * n_tok * 2          # matrix elements covered over both passes
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    mufu_peak = sms * 16 * peaks.get("sm_max_mhz", 1965.0) * 1e6 / 1e12     # 16 special-function results per SM per clock
    out["token_redundancy"] = {"us": us, "rows_per_slab": n_tok, "bound": "alu", "achieved": exps / us / 1e6,
                               "peak": mufu_peak, "unit": "T exp/s", "frac": exps / us / 1e6 / mufu_peak,
                               "matrix_elements_T_per_s": elems / us / 1e6, "tensor_tflops": exps * 256 / us / 1e6,
                               "note": "each block pair is evaluated once; the column sums (a butterfly per 32 columns) "
                                       "make the issue slots, not the exponentials, the limit"}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="skipkv", choices=["skipkv", "reference"])
    ap.add_argument("--config", type=int, default=2, help="workload index (2 = the headline configuration)")
    ap.add_argument("--batch", type=int, default=0, help="override the number of sequences (profiling captures)")
    ap.add_argument("--layers", type=int, default=4, help="layers (independent K/V buffers) each leg of a step runs over")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--extras", action="store_true",
                    help="also time the entry points beside the main path (lookup table, exactly-B variants, "
                         "token-level redundancy); reported under \"extras\", not part of `value`")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "skipkv" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
        return

    from paper_2512_07993_b200 import binding as B, build
    if not os.path.exists(B.LIB_PATH):
        build.build()
    B.lib()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    cfg = W.config(args.config, batch=args.batch) if args.batch else W.config(args.config)
    NL = max(1, args.layers)
    # NL independently seeded layers of the workload, each with its own K/V: every leg of a step runs
    # over all of them back to back, so a launch never finds its inputs in L2 (1 GB per layer)
    Ls = [W.make_layer(cfg, layer=l) for l in range(NL)]
    Ds = [B.DeviceLayer(L) for L in Ls]
    L, D = Ls[0], Ds[0]
    keys = ("K", "V", "sent_off", "sent_id", "n_sent", "kv_len", "hidden")
    pristine = [{k: getattr(Dl, k).clone() for k in keys} for Dl in Ds]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    clean = torch.ones(256 << 20, dtype=torch.uint8, device="cuda")

    def restore():
        for Dl, pr in zip(Ds, pristine):
            for k, v in pr.items():
                getattr(Dl, k).copy_(v)
        flush.fill_(1)                      # evict whatever the restore left in L2 ...
        clean.sum()                         # ... then read a clean buffer: no dirty lines are left to write back

    # decode_attn_full_ctx: the same decode call over the cache before eviction (every cached token live), for
    # comparison with decode_attn over the compacted cache; it is not part of `value` or of `ms_per_step`
    legs = ("decode_attn_full_ctx", "score", "select", "compact", "decode_attn")
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(6)] for _ in range(args.steps)]
    scratch_out = torch.empty_like(D.out)

    def step(events=None):
        rec = (lambda i: events[i].record()) if events else (lambda i: None)
        rec(0)
        for Dl in Ds:
            B.skipkv_decode_attn(Dl.shape, Dl.q, Dl.K, Dl.V, Dl.kv_len, scratch_out, None, None, None, None, Dl.ws)
        rec(1)
        for Dl in Ds: Dl.score()
        rec(2)
        for Dl in Ds: Dl.select()
        rec(3)
        for Dl in Ds: Dl.compact()
        rec(4)
        for Dl in Ds: Dl.decode_attn(steer=True)
        rec(5)

    clocks = ClockSampler(local_rank); clocks.start()      # nvidia-smi needs a moment to deliver its first sample
    for _ in range(args.warmup):
        restore(); step()
    torch.cuda.synchronize()
    for Dl in Ds: Dl.status()
    if dist: dist.barrier()
    torch.cuda.synchronize()
    t0 = time.time()
    for i in range(args.steps):
        restore(); step(ev[i])
    torch.cuda.synchronize()
    if dist: dist.barrier()
    torch.cuda.synchronize()
    t1 = time.time()
    clk = clocks.stop(t0, t1)
    if clk is None:                 # timed region shorter than the sampling period: use the warm-up samples too (same load)
        clk = clocks.stop(clocks.t_start, t1)
    for Dl in Ds: Dl.status()

    # per-launch (= per-layer) times: a leg's elapsed time over its NL back-to-back calls
    per = {leg: [ev[i][k].elapsed_time(ev[i][k + 1]) * 1e3 / NL for i in range(args.steps)] for k, leg in enumerate(legs)}
    us = {leg: statistics.mean(v) for leg, v in per.items()}
    us_med = {leg: statistics.median(v) for leg, v in per.items()}
    evict_us = us["score"] + us["select"] + us["compact"]
    step_ms = (evict_us + us["decode_attn"]) * NL / 1e3
    evict_us, step_ms, dec_us_max = max_over_ranks([evict_us, step_ms, us["decode_attn"]], dist, "cuda")

    # algorithmic bytes per layer from the actual lengths (mean over the NL layers)
    kv0 = np.stack([Ll["kv_len"].astype(np.int64) for Ll in Ls])
    kv1 = np.stack([Dl.kv_len.cpu().numpy().astype(np.int64) for Dl in Ds])
    row = 2 * cfg.head_dim
    bytes_alg = {"score": int(kv0.sum()) * row // NL,                 # K read once
                 "compact": int(kv1.sum()) * row * 2 * 2 // NL,       # kept K and V rows read and written
                 "decode_attn": int(kv1.sum()) * row * 2 // NL,       # live K and V rows read once
                 "decode_attn_full_ctx": int(kv0.sum()) * row * 2 // NL}
    peaks = measured_peaks()
    traffic = ncu_traffic()
    roof = {}
    for leg in ("score", "compact", "decode_attn", "decode_attn_full_ctx"):
        gbs = bytes_alg[leg] / (us[leg] * 1e-6) / 1e9
        roof[leg] = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": gbs / peaks["hbm_gbs"], "peak_source": peaks["source"], "us": us[leg],
                     "us_median": us_med[leg], "algorithmic_bytes": bytes_alg[leg],
                     "frac_of_nominal_8TBs": gbs / 8000.0, "traffic": traffic.get(leg)}
    dominant = max(("score", "compact", "decode_attn"), key=lambda k: us[k])

    line = {"metric": METRIC, "value": replica_value(evict_us, world), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16 storage, f32 arithmetic", "data": "synthetic",
            # token counts of the first layer (the layer the reference arm runs), so that both arms name the same numbers
            "config": workload_config(cfg, args.config, int(kv0[0].sum() // cfg.n_kv_heads),
                                      int(kv1[0].sum() // cfg.n_kv_heads), NL, world),
            "us": us, "decode_attn_us": dec_us_max, "decode_attn_gbs": bytes_alg["decode_attn"] / (dec_us_max * 1e-6) / 1e9,
            "roofline": dict(roof[dominant], kernel=dominant), "roofline_by_step": roof,
            "gpu_launches": sum(LAUNCHES_PER_STEP.values()) * NL * args.steps, "clocks": clk}

    # ---- end to end through the C ABI with host buffers (pinned), copies inside the timed region
    if not args.no_e2e:
        host_in = {k: pristine[0][k].cpu().pin_memory() for k in keys}
        host_in["q_win"] = D.q_win.cpu().pin_memory(); host_in["q"] = D.q.cpu().pin_memory()
        outs = ("out", "kv_len", "n_sent", "sent_off", "sent_id", "hidden")
        host_out = {k: torch.empty_like(getattr(D, k), device="cpu").pin_memory() for k in outs}
        h2d = sum(v.numel() * v.element_size() for v in host_in.values())
        d2h = sum(v.numel() * v.element_size() for v in host_out.values())
        n_e2e = max(3, min(args.steps, 5))
        e2e_t = []
        for i in range(1 + n_e2e):
            flush.fill_(1)
            torch.cuda.synchronize()
            a, b_, c = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            a.record()
            for k, v in host_in.items():
                getattr(D, k).copy_(v, non_blocking=True)
            D.score(); D.select(); D.compact()
            b_.record()
            D.decode_attn(steer=True)
            for k in outs:
                host_out[k].copy_(getattr(D, k), non_blocking=True)
            c.record()
            torch.cuda.synchronize()
            if i:
                e2e_t.append((a.elapsed_time(b_) * 1e3, a.elapsed_time(c) * 1e3))
        e2e_evict = statistics.mean(x[0] for x in e2e_t)
        e2e_all = statistics.mean(x[1] for x in e2e_t)
        e2e_evict, e2e_all = max_over_ranks([e2e_evict, e2e_all], dist, "cuda")
        line["e2e"] = {"value": replica_value(e2e_evict, world), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                       "whole_step_us": e2e_all / world,
                       "note": "host->device copy of K, V, queries and tables from pinned memory, the four calls, "
                               "device->host read of the attention output, hidden state and tables"}

    # ---- the oracle on this machine's host cores (rank 0, single GPU runs only): one warm-up and one timed pass over the
    # whole layer with all threads (every thread has slabs to work on), and one sequence on a single thread
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        time_oracle(L)
        legs_s, _, cores = time_oracle(L)
        legs_1, frac_1, _ = time_oracle(L, n_seq=1, threads=1)
        line["cpu_baseline"] = {"value": (legs_s["score"] + legs_s["select"] + legs_s["compact"]) * 1e6,
                                "unit": UNIT, "cores": cores, "kind": "oracle", "host_cores": os.cpu_count(),
                                "decode_attn_us": legs_s["decode_attn"] * 1e6,
                                "sample": "one full layer (all sequences), second of two passes, no scaling",
                                "one_core": {"value": (legs_1["score"] + legs_1["select"] + legs_1["compact"]) / frac_1 * 1e6,
                                             "cores": 1,
                                             "sample": f"first sequence ({frac_1:.3f} of the tokens), time scaled by token count"}}
    if args.extras and world == 1:
        del Ds, D, pristine
        torch.cuda.empty_cache()
        line["extras"] = time_extras(cfg, B, flush, clean, peaks)
    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
