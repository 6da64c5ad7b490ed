// skipkv_compact: in-place stream compaction of the surviving K/V rows (paper Algorithm 1,
// eviction + post-eviction range update, Eq. "after").
//
// Two launches on the caller's stream:
//   plan  one CTA per (sequence, head) slab.  Block-wide scans over the keep flags turn the
//         sentence table into (a) the rewritten tables and (b) a list of runs: maximal groups
//         of adjacent kept sentences, each a contiguous source block that lands on a
//         contiguous destination block.
//   move  persistent CTAs.  K and V of a slab are two independent streams; a stream's
//         destination range is cut into segments of kSegRows rows which are handed out in
//         ascending order by an atomic ticket.  A CTA pulls every source piece of its segment
//         into shared memory with bulk asynchronous copies (one copy per run piece, no
//         register staging), publishes "segments 0..j of this stream are loaded", and then
//         writes the pieces to their destination with bulk stores.
//
// With partly kept sentences (skipkv_compact_fill: keep == 2, survivors flagged per token) the plan first packs
// the surviving rows of such a sentence to the front of the sentence's own rows, so that it becomes a shorter
// contiguous sentence and the move proceeds unchanged; a third, tiny launch then corrects the index-map
// entries of those sentences.
//
// Why this is safe in place: rows only move down (dst <= src), so a store into segment j can
// only overwrite source rows of segments <= j.  A segment therefore stores only after every
// lower segment of its stream has finished loading (the per-stream `loaded` counter advances
// strictly in segment order) and after its own loads have landed.  Tickets are issued in
// ascending segment order, so whatever a CTA waits for is already held by a running CTA whose
// loads never wait: the wait cannot deadlock, and it is bounded anyway (on expiry the status
// word is flagged and the stores of that segment are skipped).
#include "common.cuh"

namespace skipkv {

constexpr int kSegRows = 256;                       // rows per segment (64 KB of shared memory)
constexpr int kSegBytes = kSegRows * kRowBytes;
constexpr int kMoveThreads = 128;
constexpr int kPlanThreads = 1024;

// exclusive block scan of three ints at once; returns the block totals through tot[]
__device__ __forceinline__ void block_scan3(int v0, int v1, int v2, int& e0, int& e1, int& e2, int tot[3],
                                            int (*wsum)[3]) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    int i0 = v0, i1 = v1, i2 = v2;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int a0 = __shfl_up_sync(0xffffffffu, i0, d), a1 = __shfl_up_sync(0xffffffffu, i1, d),
                  a2 = __shfl_up_sync(0xffffffffu, i2, d);
        if (lane >= d) { i0 += a0; i1 += a1; i2 += a2; }
    }
    if (lane == 31) { wsum[warp][0] = i0; wsum[warp][1] = i1; wsum[warp][2] = i2; }
    __syncthreads();
    int b0 = 0, b1 = 0, b2 = 0, t0 = 0, t1 = 0, t2 = 0;
    for (int w = 0; w < nw; ++w) {
        if (w == warp) { b0 = t0; b1 = t1; b2 = t2; }
        t0 += wsum[w][0]; t1 += wsum[w][1]; t2 += wsum[w][2];
    }
    e0 = b0 + i0 - v0; e1 = b1 + i1 - v1; e2 = b2 + i2 - v2;
    tot[0] = t0; tot[1] = t1; tot[2] = t2;
    __syncthreads();
}

// Rows of tokens [pb, pe) of a slab whose flag is set move, in order, to rows pb, pb+1, ... of the same slab.
// K and V together, 64 rows per pass: every thread holds one 16-byte piece of each; all pieces of a pass are read before any is written,
// and destinations never lie above sources.
__device__ __forceinline__ void pack_rows(uint4* kbase, uint4* vbase, const uint8_t* tk, int pb, int pe, int* s_pos,
                                          int* s_wcnt) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int r = tid >> 4, col = tid & 15;
    int done = 0;
    for (int cb = pb; cb < pe; cb += 64) {
        if (tid < 64) {
            const int f = (cb + tid < pe) ? (tk[cb + tid] != 0) : 0;
            const unsigned m = __ballot_sync(0xffffffffu, f);
            s_pos[tid] = __popc(m & ((1u << lane) - 1u));
            if (lane == 0) s_wcnt[warp] = __popc(m);
        }
        __syncthreads();
        const int t = cb + r;
        const bool f = t < pe && tk[t] != 0;
        const int dst = pb + done + s_pos[r] + (r >= 32 ? s_wcnt[0] : 0);
        uint4 kval = make_uint4(0u, 0u, 0u, 0u), vval = kval;
        if (f) { kval = kbase[size_t(t) * 16 + col]; vval = vbase[size_t(t) * 16 + col]; }
        done += s_wcnt[0] + s_wcnt[1];
        __syncthreads();
        if (f && dst != t) { kbase[size_t(dst) * 16 + col] = kval; vbase[size_t(dst) * 16 + col] = vval; }
        __syncthreads();
    }
}

template <bool kFill>
__global__ void __launch_bounds__(kPlanThreads)
compact_plan_kernel(int Hk, int max_sent, const int64_t* slab_off, const int32_t* cap, const uint8_t* keep,
                    const uint8_t* tok_keep, uint4* K, uint4* V, int32_t* sent_off, int32_t* sent_id, int32_t* n_sent,
                    int32_t* kv_len, Header* hdr, int32_t* cp_nseg, uint32_t* cp_loaded, int32_t* cp_nruns,
                    int32_t* cp_run_src, int32_t* cp_run_dst, int32_t* cp_part) {
    __shared__ int wsum[kPlanThreads / 32][3];
    __shared__ int s_bad;
    __shared__ int s_npart, s_part[kMaxPartial][3], s_pos[64], s_wcnt[2];
    __shared__ int s_next_begin[2];                      // old sent_off[base] of the next chunk of sentences (by chunk parity)
    // the move kernel is launched as a programmatic dependent: let its CTAs set themselves up while this grid runs
    pdl_trigger();
    pdl_wait();                                          // inputs may come from the kernel before
    const int slab = blockIdx.x;
    const int b = slab / Hk;
    const int tid = threadIdx.x;
    const uint8_t* kp = keep + size_t(slab) * max_sent;
    int32_t* so = sent_off + size_t(slab) * (max_sent + 1);
    int32_t* sid = sent_id + size_t(slab) * max_sent;
    int32_t* run_src = cp_run_src + size_t(slab) * max_sent;
    int32_t* run_dst = cp_run_dst + size_t(slab) * (max_sent + 1);
    const int S = n_sent[slab];
    const int capb = cap[b];
    const size_t row0 = slab_row0(slab_off, cap, Hk, b, slab % Hk);
    const uint8_t* tk = kFill ? tok_keep + row0 : nullptr;
    int32_t* part = cp_part + size_t(slab) * (1 + 3 * kMaxPartial);
    if (tid == 0) {
        s_npart = 0;
        if (kFill) part[0] = 0;
        s_bad = (S < 0 || S > max_sent) ? 1 : 0;
        cp_loaded[2 * slab] = 0u;
        cp_loaded[2 * slab + 1] = 0u;
        if (slab == 0) hdr->compact_ticket = 0u;
    }
    __syncthreads();
    if (s_bad) {
        if (tid == 0) { atomicOr(&hdr->status, SKIPKV_STATUS_BAD_TABLE); cp_nseg[slab] = 0; cp_nruns[slab] = 0; }
        return;
    }
    int c_len = 0, c_cnt = 0, c_run = 0;     // carries: kept tokens, kept sentences, runs so far
    int prev_alive_carry = 0;
    for (int base = 0; base < S; base += kPlanThreads) {
        const int i = base + tid;
        int b_i = 0, e_i = 0, id_i = -1, alive = 0, klen = 0;
        if (i < S) {
            // the table is rewritten in place, and the chunk before may already have overwritten so[base]: its
            // last thread parked the old value
            b_i = (tid == 0 && base > 0) ? s_next_begin[((base / kPlanThreads) & 1) ^ 1] : so[i];
            e_i = so[i + 1]; id_i = sid[i];
            if (tid == kPlanThreads - 1) s_next_begin[(base / kPlanThreads) & 1] = e_i;   // for thread 0 of the next chunk
            if (b_i < 0 || e_i < b_i || e_i > capb || (i == 0 && b_i != 0)) atomicOr(&s_bad, 1);
            else if (kp[i] != 0 && e_i > b_i) {
                klen = e_i - b_i;
                if (kFill && kp[i] == 2) {               // partly kept: count its survivors
                    klen = 0;
                    for (int t = b_i; t < e_i; ++t) klen += tk[t] != 0 ? 1 : 0;
                }
                alive = klen > 0 ? (klen < e_i - b_i ? 3 : 1) : 0;   // bit 1: rows are missing behind this sentence
            }
        }
        // does the previous sentence also survive, whole?  (adjacent whole survivors form one run; a partly
        // kept sentence can end a run but nothing can follow it in the same run)
        int prev_alive = __shfl_up_sync(0xffffffffu, alive, 1);
        __shared__ int s_last[kPlanThreads / 32];
        if ((tid & 31) == 31) s_last[tid >> 5] = alive;
        __syncthreads();
        if ((tid & 31) == 0) prev_alive = (tid == 0) ? prev_alive_carry : s_last[(tid >> 5) - 1];
        const int last_alive = s_last[kPlanThreads / 32 - 1];
        const int start = (alive && prev_alive != 1) ? 1 : 0;
        const int partial = alive == 3;
        alive = alive ? 1 : 0;
        int x_len, x_cnt, x_run, tot[3];
        block_scan3(klen, alive, start, x_len, x_cnt, x_run, tot, wsum);   // syncs: old values are all read
        if (alive) {
            so[c_cnt + x_cnt + 1] = c_len + x_len + klen;
            sid[c_cnt + x_cnt] = id_i;
            if (start) {
                run_src[c_run + x_run] = b_i;
                run_dst[c_run + x_run] = c_len + x_len;
            }
            if (kFill && partial) {
                const int q = atomicAdd(&s_npart, 1);
                if (q < kMaxPartial) { s_part[q][0] = b_i; s_part[q][1] = e_i; s_part[q][2] = c_len + x_len; }
                else atomicOr(&s_bad, 1);
            }
        }
        c_len += tot[0]; c_cnt += tot[1]; c_run += tot[2];
        prev_alive_carry = last_alive;
        __syncthreads();
    }
    if (s_bad) {
        // tables may be half rewritten; flag it and move nothing
        if (tid == 0) { atomicOr(&hdr->status, SKIPKV_STATUS_BAD_TABLE); cp_nseg[slab] = 0; cp_nruns[slab] = 0; }
        return;
    }
    for (int i = c_cnt + 1 + tid; i <= max_sent; i += kPlanThreads) so[i] = c_len;
    for (int i = c_cnt + tid; i < max_sent; i += kPlanThreads) sid[i] = -1;
    if (tid == 0) {
        so[0] = 0;
        run_dst[c_run] = c_len;
        n_sent[slab] = c_cnt;
        kv_len[slab] = c_len;
        cp_nruns[slab] = c_run;
        cp_nseg[slab] = (c_len + kSegRows - 1) / kSegRows;
    }
    if (kFill) {
        __syncthreads();
        const int np = s_npart;
        if (tid < np * 3) part[1 + tid] = s_part[tid / 3][tid % 3];
        if (tid == 0) part[0] = np;
        for (int q = 0; q < np; ++q) {                     // uniform over the CTA
            pack_rows(K + row0 * 16, V + row0 * 16, tk, s_part[q][0], s_part[q][1], s_pos, s_wcnt);
        }
    }
}

// index_map entries of the partly kept sentences: destination token dst + k came from the k-th flagged token.
__global__ void __launch_bounds__(64)
compact_fill_index_kernel(int Hk, const int64_t* slab_off, const int32_t* cap, const uint8_t* tok_keep,
                          int32_t* index_map, const int32_t* cp_part) {
    __shared__ int s_wcnt[2];
    const int slab = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pdl_trigger();
    pdl_wait();                                          // after the move kernel, which wrote the run-based entries
    const int32_t* part = cp_part + size_t(slab) * (1 + 3 * kMaxPartial);
    const int np = min(part[0], kMaxPartial);
    const size_t row0 = slab_row0(slab_off, cap, Hk, slab / Hk, slab % Hk);
    for (int q = 0; q < np; ++q) {
        const int pb = part[1 + 3 * q], pe = part[2 + 3 * q], dst = part[3 + 3 * q];
        int done = 0;
        for (int cb = pb; cb < pe; cb += 64) {
            const int t = cb + tid;
            const int f = (t < pe) ? (tok_keep[row0 + t] != 0) : 0;
            const unsigned m = __ballot_sync(0xffffffffu, f);
            if (lane == 0) s_wcnt[warp] = __popc(m);
            __syncthreads();
            const int pos = done + __popc(m & ((1u << lane) - 1u)) + (warp ? s_wcnt[0] : 0);
            if (f) index_map[row0 + dst + pos] = t;
            done += s_wcnt[0] + s_wcnt[1];
            __syncthreads();
        }
    }
}

__global__ void __launch_bounds__(kMoveThreads)
compact_move_kernel(int n_slabs, int Hk, int max_sent, const int64_t* slab_off, const int32_t* cap,
                    __nv_bfloat16* K, __nv_bfloat16* V, int32_t* index_map, Header* hdr, const int32_t* cp_nseg,
                    uint32_t* cp_loaded, const int32_t* cp_nruns, const int32_t* cp_run_src,
                    const int32_t* cp_run_dst, const int32_t* block_table, int max_pages) {
    extern __shared__ __align__(1024) uint8_t smem[];
    __shared__ __align__(8) uint64_t bar;
    __shared__ int s_red[kMoveThreads / 32];
    __shared__ uint32_t s_ticket;
    __shared__ int s_abort;                            // a wait of this CTA ran out: it takes no further segment
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    if (tid == 0) { mbar_init(&bar, 1); mbar_fence_init(); s_abort = 0; }
    // everything below reads what the plan kernel wrote: wait until that grid has completed and its writes are visible
    pdl_wait();
    // every CTA derives the scheduler bound: the largest segment count of any slab
    int mx = 0;
    for (int i = tid; i < n_slabs; i += kMoveThreads) mx = max(mx, cp_nseg[i]);
#pragma unroll
    for (int d = 16; d; d >>= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, d));
    if (lane == 0) s_red[warp] = mx;
    __syncthreads();
    int max_nseg = 0;
    for (int w = 0; w < kMoveThreads / 32; ++w) max_nseg = max(max_nseg, s_red[w]);
    const uint32_t n_streams = 2u * n_slabs;
    const uint32_t n_tickets = n_streams * uint32_t(max_nseg);
    const uint32_t limit = load_wait_limit(hdr);       // polls a wait makes before it gives up
    uint32_t phase = 0;

    for (;;) {
        __syncthreads();                               // s_ticket / smem free for the next round
        if (s_abort) break;                            // (read by every thread after the barrier: a uniform exit)
        if (tid == 0) s_ticket = atomicAdd(&hdr->compact_ticket, 1u);
        __syncthreads();
        const uint32_t T = s_ticket;
        if (T >= n_tickets) break;
        const int stream = int(T % n_streams), j = int(T / n_streams);
        const int slab = stream >> 1;
        if (j >= cp_nseg[slab]) continue;
        const int b = slab / Hk, h = slab % Hk;
        // contiguous slabs: token t of the slab is row row0 + t; paged cache (128-row pages): row table[t / 128] * 128 + t % 128,
        // and a copy is cut where its source or its destination crosses a page
        const int32_t* table = block_table ? block_table + size_t(slab) * max_pages : nullptr;
        const size_t row0 = table ? size_t(slab) * max_pages * 128 : slab_row0(slab_off, cap, Hk, b, h);   // (paged: index_map rows)
        uint8_t* tensor = reinterpret_cast<uint8_t*>((stream & 1) ? V : K);
        uint8_t* base = tensor + (table ? 0 : row0 * kRowBytes);
        auto row_ptr = [&](int t) {
            return table ? tensor + (size_t(max(table[t >> 7], 0)) * 128 + (t & 127)) * kRowBytes : base + size_t(t) * kRowBytes;
        };
        auto piece_rows = [&](int src, int dst, int left) {      // rows of a copy that stay inside one page on both sides
            return table ? min(left, min(128 - (src & 127), 128 - (dst & 127))) : left;
        };
        const int32_t* run_src = cp_run_src + size_t(slab) * max_sent;
        const int32_t* run_dst = cp_run_dst + size_t(slab) * (max_sent + 1);
        const int nruns = cp_nruns[slab];
        const int new_len = run_dst[nruns];
        const int d0 = j * kSegRows, d1 = min(d0 + kSegRows, new_len);
        // first run that reaches into [d0, d1): largest r with run_dst[r] <= d0
        int lo = 0, hi = nruns - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (run_dst[mid] <= d0) lo = mid; else hi = mid - 1;
        }
        const int r0 = lo;

        if (warp == 0) {
            // pass 1: bytes this segment will receive; pass 2: issue the copies
            uint32_t bytes = 0;
            for (int r = r0 + lane; r < nruns && run_dst[r] < d1; r += 32) {
                const int ps = max(run_dst[r], d0), pe = min(run_dst[r + 1], d1);
                const int src = run_src[r] + (ps - run_dst[r]);
                if (src != ps) bytes += uint32_t(pe - ps) * kRowBytes;
            }
#pragma unroll
            for (int d = 16; d; d >>= 1) bytes += __shfl_xor_sync(0xffffffffu, bytes, d);
            if (lane == 0) {
                if (bytes) mbar_expect_tx(&bar, bytes); else mbar_arrive(&bar);
            }
            __syncwarp();
            for (int r = r0 + lane; r < nruns && run_dst[r] < d1; r += 32) {
                const int ps = max(run_dst[r], d0), pe = min(run_dst[r + 1], d1);
                const int src = run_src[r] + (ps - run_dst[r]);
                if (src != ps)
                    for (int o = 0; o < pe - ps;) {
                        const int nr = piece_rows(src + o, ps + o, pe - ps - o);
                        bulk_g2s(smem + size_t(ps + o - d0) * kRowBytes, row_ptr(src + o), uint32_t(nr) * kRowBytes, &bar);
                        o += nr;
                    }
            }
        } else if (index_map != nullptr && (stream & 1) == 0) {
            // dest token k of this segment came from token run_src[r] + (k - run_dst[r])
            int32_t* im = index_map + row0;
            for (int r = r0; r < nruns && run_dst[r] < d1; ++r) {
                const int ps = max(run_dst[r], d0), pe = min(run_dst[r + 1], d1);
                const int delta = run_src[r] - run_dst[r];
                for (int k = ps + (tid - 32); k < pe; k += kMoveThreads - 32) im[k] = k + delta;
            }
        }
        if (warp == 0) {
            // every lane observes the landing of the loads it is about to forward
            int ok = mbar_wait(&bar, phase, limit) ? 1 : 0;
            if (lane == 0) {
                if (!ok) atomicOr(&hdr->status, SKIPKV_STATUS_COPY_TIMEOUT);
                // hand-off: wait until segments 0..j-1 of this stream are loaded, then publish j
                volatile uint32_t* ld = cp_loaded + stream;
                uint32_t spins = 0;
                while (*ld < uint32_t(j)) {
                    if (++spins > limit) {
                        ok = 0;
                        atomicOr(&hdr->status, SKIPKV_STATUS_COMPACT_TIMEOUT);
                        break;
                    }
                    __nanosleep(32);
                }
                __threadfence();
                atomicMax(cp_loaded + stream, uint32_t(j) + 1u);
            }
            ok = __shfl_sync(0xffffffffu, ok, 0) & __all_sync(0xffffffffu, ok);
            if (ok) {
                for (int r = r0 + lane; r < nruns && run_dst[r] < d1; r += 32) {
                    const int ps = max(run_dst[r], d0), pe = min(run_dst[r + 1], d1);
                    const int src = run_src[r] + (ps - run_dst[r]);
                    if (src != ps)
                        for (int o = 0; o < pe - ps;) {
                            const int nr = piece_rows(src + o, ps + o, pe - ps - o);
                            bulk_s2g(row_ptr(ps + o), smem + size_t(ps + o - d0) * kRowBytes, uint32_t(nr) * kRowBytes);
                            o += nr;
                        }
                }
                bulk_commit();
            } else {
                // A wait ran out (flagged above): the stores of this segment are skipped and this CTA stops.  Its own
                // loads may still be in flight towards its shared memory, and they must land before it retires.
                mbar_wait(&bar, phase, 1u << 20);
                if (lane == 0) s_abort = 1;
            }
            bulk_wait_read_all();                      // shared memory may be refilled
        }
        phase ^= 1u;
    }
    if (warp == 0) bulk_wait_all();                    // all stores performed before exit
}

}  // namespace skipkv

using namespace skipkv;

static int compact_impl(const skipkv_shape* shape, void* K, void* V, const uint8_t* keep, const uint8_t* tok_keep,
                        int32_t* sent_off, int32_t* sent_id, int32_t* n_sent, int32_t* kv_len, int32_t* index_map,
                        void* ws, void* stream, const int32_t* block_table = nullptr, int max_pages = 0) {
    if (int rc = check_shape(shape)) return rc;
    if (!K || !V || !keep || !sent_off || !sent_id || !n_sent || !kv_len) return SKIPKV_ERR_INVALID_ARG;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255)) return SKIPKV_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(K) & 15) || (reinterpret_cast<uintptr_t>(V) & 15)) return SKIPKV_ERR_INVALID_ARG;
    const WsLayout L = make_layout(*shape);
    uint8_t* w = static_cast<uint8_t*>(ws);
    Header* hdr = reinterpret_cast<Header*>(w + L.header);
    int32_t* nseg = reinterpret_cast<int32_t*>(w + L.cp_nseg);
    uint32_t* loaded = reinterpret_cast<uint32_t*>(w + L.cp_loaded);
    int32_t* nruns = reinterpret_cast<int32_t*>(w + L.cp_nruns);
    int32_t* run_src = reinterpret_cast<int32_t*>(w + L.cp_run_src);
    int32_t* run_dst = reinterpret_cast<int32_t*>(w + L.cp_run_dst);
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    int32_t* part = reinterpret_cast<int32_t*>(w + L.cp_part);
    auto plan = tok_keep ? compact_plan_kernel<true> : compact_plan_kernel<false>;
    SKIPKV_CUDA(launch_dependent(plan, dim3(L.slabs), dim3(kPlanThreads), 0, st, int(shape->n_kv_heads),
                                 int(shape->max_sent), shape->slab_off, shape->cap, keep, tok_keep, static_cast<uint4*>(K),
                                 static_cast<uint4*>(V), sent_off, sent_id, n_sent, kv_len, hdr, nseg, loaded, nruns,
                                 run_src, run_dst, part));

    // set on every call: the attribute belongs to the current device's context, which a cached flag would not track
    SKIPKV_CUDA(cudaFuncSetAttribute(compact_move_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSegBytes));
    SKIPKV_CUDA(launch_dependent(compact_move_kernel, dim3(unsigned(num_sms() * 3)), dim3(kMoveThreads), kSegBytes, st,
                                 int(L.slabs), int(shape->n_kv_heads), int(shape->max_sent), shape->slab_off, shape->cap,
                                 static_cast<__nv_bfloat16*>(K), static_cast<__nv_bfloat16*>(V), index_map, hdr, nseg, loaded,
                                 nruns, run_src, run_dst, block_table, max_pages));
    if (tok_keep && index_map)
        SKIPKV_CUDA(launch_dependent(compact_fill_index_kernel, dim3(L.slabs), dim3(64), 0, st, int(shape->n_kv_heads),
                                     shape->slab_off, shape->cap, tok_keep, index_map, static_cast<const int32_t*>(part)));
    return SKIPKV_OK;
}

extern "C" int skipkv_compact(const skipkv_shape* shape, void* K, void* V, const uint8_t* keep,
                              int32_t* sent_off, int32_t* sent_id, int32_t* n_sent, int32_t* kv_len,
                              int32_t* index_map, void* ws, void* stream) {
    return compact_impl(shape, K, V, keep, nullptr, sent_off, sent_id, n_sent, kv_len, index_map, ws, stream);
}

extern "C" int skipkv_compact_fill(const skipkv_shape* shape, void* K, void* V, const uint8_t* keep,
                                   const uint8_t* tok_keep, int32_t* sent_off, int32_t* sent_id, int32_t* n_sent,
                                   int32_t* kv_len, int32_t* index_map, void* ws, void* stream) {
    if (!tok_keep) return SKIPKV_ERR_INVALID_ARG;
    return compact_impl(shape, K, V, keep, tok_keep, sent_off, sent_id, n_sent, kv_len, index_map, ws, stream);
}

extern "C" int skipkv_compact_paged(const skipkv_shape* shape, void* K_pages, void* V_pages, const int32_t* block_table,
                                    int32_t max_pages, const uint8_t* keep, int32_t* sent_off, int32_t* sent_id,
                                    int32_t* n_sent, int32_t* kv_len, int32_t* index_map, void* ws, void* stream) {
    if (!block_table || max_pages <= 0) return SKIPKV_ERR_INVALID_ARG;
    return compact_impl(shape, K_pages, V_pages, keep, nullptr, sent_off, sent_id, n_sent, kv_len, index_map, ws, stream,
                        block_table, max_pages);
}
