// skipkv_decode_attn: GQA decode attention over the ragged, compacted cache (the attention
// equation of paper Section 4.1 with one query per head), with the steering add of Section 4.2
// performed by the tail of the same launch.
//
// The step is HBM bound: every live K and V row is read exactly once.  Design:
//  * Work = 128-row tiles enumerated over all (sequence, head) slabs.  The tile list is cut into
//    equal contiguous ranges, one per persistent CTA, so CTAs are balanced whatever the ragged
//    lengths are; a CTA's range may cross slab boundaries, each (CTA, slab) intersection gives
//    one partial result (running max, sum, 128-wide accumulator per head).
//  * K and V tiles are streamed into a shared-memory ring with bulk asynchronous copies (each
//    tile is one contiguous block of the slab) signalled through mbarriers, issued two tiles
//    ahead by one elected lane; sixteen warps work on 8 rows of a tile each.  (512 threads in one
//    CTA per SM leave 128 registers per thread, which the mapping below needs; the ring of
//    3 x 64 KB keeps 128 KB of loads in flight per SM.)
//  * Consumer mapping: a half-warp per row, 8 channels (16 bytes) per lane.  The four heads of
//    the group share every K/V load.  fp32 arithmetic with packed two-wide FMAs; the 16 partial
//    dot products a lane holds for 4 rows x 4 heads are reduced with a 15-shuffle butterfly
//    that leaves one finished logit per lane.
//  * Softmax is online in base 2 (the log2(e)/sqrt(d) factor is folded into q).
//  * The last CTA to deliver a partial for a slab (self-resetting counter in the workspace)
//    merges that slab's partials and writes the bf16 output.
//  * Every wait is bounded; on expiry the status word is flagged and the kernel drains.
#include <cstdio>
#include <mutex>

#include "common.cuh"
#include "steer.cuh"

namespace skipkv {

// Measured on the headline workload (166 MB of live rows, calls back to back): one CTA of 512 threads per SM with
// 128-row tiles takes 45.8 us per call, two CTAs of 256 threads with 64-row tiles 46.9 us (178.7 against 174.3 us over
// the un-evicted cache): the second CTA does not hide the fixed part of a call, because both CTAs of an SM reach their
// set-up and their merge at the same time.
constexpr int kTileRows = 128;
constexpr int kTileBytes = kTileRows * kRowBytes;         // 32 KB for K, same for V
constexpr int kPageRows = 128;                            // paged cache: rows per page
constexpr int kPageBytes = kPageRows * kRowBytes;
constexpr int kTilesPerPage = kPageRows / kTileRows;
constexpr int kStages = 3;
constexpr int kConsWarps = 16;
constexpr int kDecThreads = kConsWarps * 32;
constexpr int kCtasPerSm = 1;
constexpr int kPartStride = 130;                          // global record: 128 accumulators + max + sum
constexpr int kWpStride = 132;                            // same record in shared memory, 16-byte aligned rows
constexpr int kMaxDecSlabs = 8192;

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Optional fusion of the per-step bookkeeping into the decode launch (k_new == nullptr: plain decode attention).
// The tile schedule covers the rows already cached; the CTA that owns a slab's last tile writes the new K/V row into
// the cache, folds it into the attention as a one-row tile after the last streamed tile, and updates the slab's range
// list and length when it flushes the segment.  A slab that was empty is handled with the zero-length slabs.  Lengths are read from kv_len and written to kv_len_out (a different buffer), so CTAs that
// start late still derive the same tile schedule.
struct StepArgs {
    const uint4* k_new;          // [batch][Hk][16]
    const uint4* v_new;
    int32_t* kv_len_out;         // [batch][Hk]
    int32_t* sent_off;           // range list, updated in place
    int32_t* sent_id;
    int32_t* n_sent;
    const uint8_t* new_sent;     // [batch]
    const int32_t* gen_id;       // [batch]
    uint4* q_win;                // nullable: [batch][Hq][window][16]
    int window, slot, max_sent;
};

struct DecSmem {
    uint64_t full[kStages];
    uint64_t empty[kStages];
    int abort_flag;
    int is_last;
    uint32_t wsum[kDecThreads / 32];
    int step_n_sent, step_starts;          // fused step: range-list inputs of the slab whose tail this CTA holds
};

__device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, %0;" ::"n"(kConsWarps * 32) : "memory"); }

// One consumer warp, 8 rows [row_base, row_base+8) of a tile, the kH (1..4) heads of the warp's head group: the
// multiply-adds are done for those heads only, the reduction always runs over four head slots.
template <bool kGuard, int kH>
__device__ __forceinline__ void tile_rows_h(const uint8_t* Ks, const uint8_t* Vs, int row_base, int rows, int lane,
                                          const float2 (&q2)[4][4], float2 (&acc)[4][4], float& m_run,
                                          float& l_run) {
    const int half = lane >> 4, l16 = lane & 15;
    const uint4* Kp = reinterpret_cast<const uint4*>(Ks + size_t(row_base + half) * kRowBytes) + l16;
    const uint4* Vp = reinterpret_cast<const uint4*>(Vs + size_t(row_base + half) * kRowBytes) + l16;
    float part[16];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint4 kk = Kp[i * 32];                     // row_base + 2i + half
        const float2 k0 = bf16x2_to_f2(kk.x), k1 = bf16x2_to_f2(kk.y), k2 = bf16x2_to_f2(kk.z),
                     k3 = bf16x2_to_f2(kk.w);
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            if (h < kH) {
                float2 a = __fmul2_rn(q2[h][0], k0);
                a = __ffma2_rn(q2[h][1], k1, a);
                a = __ffma2_rn(q2[h][2], k2, a);
                a = __ffma2_rn(q2[h][3], k3, a);
                part[i * 4 + h] = a.x + a.y;
            } else {
                part[i * 4 + h] = 0.f;
            }
        }
    }
    // butterfly over the 16 lanes of a half-warp: lane l16 ends with the full sum of part[l16]
    const bool u8 = lane & 8, u4 = lane & 4, u2 = lane & 2, u1 = lane & 1;
    float r8[8], r4[4], r2[2];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const float mine = u8 ? part[k + 8] : part[k], send = u8 ? part[k] : part[k + 8];
        r8[k] = mine + __shfl_xor_sync(0xffffffffu, send, 8);
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float mine = u4 ? r8[k + 4] : r8[k], send = u4 ? r8[k] : r8[k + 4];
        r4[k] = mine + __shfl_xor_sync(0xffffffffu, send, 4);
    }
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const float mine = u2 ? r4[k + 2] : r4[k], send = u2 ? r4[k] : r4[k + 2];
        r2[k] = mine + __shfl_xor_sync(0xffffffffu, send, 2);
    }
    float s;
    {
        const float mine = u1 ? r2[1] : r2[0], send = u1 ? r2[0] : r2[1];
        s = mine + __shfl_xor_sync(0xffffffffu, send, 1);
    }
    // this lane's logit: row row_base + 2*(l16>>2) + half, head l16 & 3
    if (kGuard) {
        if (row_base + 2 * (l16 >> 2) + half >= rows) s = -INFINITY;
    }
    float bm = s;
    bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 4));
    bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 8));
    bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 16));
    const float m_new = fmaxf(m_run, bm);
    if (__any_sync(0xffffffffu, m_new > m_run)) {
        const float sc = ex2(m_run - m_new);             // first block: 2^(-inf) = 0
        l_run *= sc;
#pragma unroll
        for (int h = 0; h < kH; ++h) {
            const float sh = __shfl_sync(0xffffffffu, sc, h);
            const float2 s2 = make_float2(sh, sh);
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[h][c] = __fmul2_rn(acc[h][c], s2);
        }
        m_run = m_new;
    }
    const float p = ex2(s - m_run);
    l_run += p;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        uint4 vv = Vp[i * 32];
        if (kGuard) {
            if (row_base + 2 * i + half >= rows) vv = make_uint4(0u, 0u, 0u, 0u);   // stale shared memory
        }
        const float2 v0 = bf16x2_to_f2(vv.x), v1 = bf16x2_to_f2(vv.y), v2 = bf16x2_to_f2(vv.z),
                     v3 = bf16x2_to_f2(vv.w);
#pragma unroll
        for (int h = 0; h < kH; ++h) {
            const float ph = __shfl_sync(0xffffffffu, p, (lane & 16) | (i * 4 + h));
            const float2 pp = make_float2(ph, ph);
            acc[h][0] = __ffma2_rn(pp, v0, acc[h][0]);
            acc[h][1] = __ffma2_rn(pp, v1, acc[h][1]);
            acc[h][2] = __ffma2_rn(pp, v2, acc[h][2]);
            acc[h][3] = __ffma2_rn(pp, v3, acc[h][3]);
        }
    }
}

template <bool kGuard, bool kExact>
__device__ __forceinline__ void tile_rows(int heads, const uint8_t* Ks, const uint8_t* Vs, int row_base, int rows, int lane,
                                          const float2 (&q2)[4][4], float2 (&acc)[4][4], float& m_run, float& l_run) {
    if (!kExact) {
        tile_rows_h<kGuard, 4>(Ks, Vs, row_base, rows, lane, q2, acc, m_run, l_run);
        return;
    }
    switch (heads) {                                         // the same for every thread of a warp
        case 4: tile_rows_h<kGuard, 4>(Ks, Vs, row_base, rows, lane, q2, acc, m_run, l_run); break;
        case 3: tile_rows_h<kGuard, 3>(Ks, Vs, row_base, rows, lane, q2, acc, m_run, l_run); break;
        case 2: tile_rows_h<kGuard, 2>(Ks, Vs, row_base, rows, lane, q2, acc, m_run, l_run); break;
        default: tile_rows_h<kGuard, 1>(Ks, Vs, row_base, rows, lane, q2, acc, m_run, l_run); break;
    }
}

// kExact: head groups of equal size with the multiply-adds of a warp limited to its group's heads (for group sizes
// that are not a multiple of four; a separate instance, so that the common four-heads-per-group kernel carries one
// copy of the row code, not four).
// kStep: the launch also performs the per-step bookkeeping described at StepArgs (a separate instance, so that
// plain decode attention carries none of it).
template <bool kStep, bool kExact>
__global__ void __launch_bounds__(kDecThreads, kCtasPerSm)
decode_attn_kernel(int batch, int Hq, int Hk, int n_slabs, const int64_t* slab_off, const int32_t* cap,
                   const __nv_bfloat16* q, const uint8_t* K, const uint8_t* V, const int32_t* kv_len,
                   __nv_bfloat16* out, uint32_t* status, uint32_t* dec_cnt, float* dec_part, int d_model,
                   __nv_bfloat16* hidden, const __nv_bfloat16* steer_vec, const float* alpha, const uint8_t* flag,
                   const int32_t* block_table, int max_pages, StepArgs step, const uint32_t* wait_limit) {
    extern __shared__ __align__(1024) uint8_t dsm[];
    uint8_t* ring = dsm;                                                     // kStages x (K tile, V tile)
    float* wpart = reinterpret_cast<float*>(dsm + kStages * 2 * kTileBytes);  // [warps][4 heads][132]
    DecSmem* sm = reinterpret_cast<DecSmem*>(wpart + kConsWarps * 4 * kWpStride);
    int* pref = reinterpret_cast<int*>(sm + 1);                              // [n_slabs + 1] tile prefix

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pdl_trigger();
    // live rows of slab s; with a block table (paged cache) a slab cannot exceed its max_pages pages of kPageRows rows
    auto room = [&](int s) { return block_table ? min(cap[s / Hk], max_pages * kPageRows) : cap[s / Hk]; };
    auto old_len = [&](int s) { return min(max(kv_len[s], 0), room(s)); };     // rows before this launch
    // cache row of token t of slab s (contiguous slabs, or through the block table)
    auto phys_row = [&](int s, int t) {
        return block_table ? size_t(max(block_table[size_t(s) * max_pages + t / kPageRows], 0)) * kPageRows + size_t(t % kPageRows)
                           : slab_row0(slab_off, cap, Hk, s / Hk, s % Hk) + size_t(t);
    };
    // rows streamed through the tile ring; with the fused step the row being appended is folded in separately
    auto live = [&](int s) { return old_len(s); };
    const int n = Hq / Hk;                     // heads per group
    const int NG = (n + 3) / 4;                // head groups (1 or 2) of H0 heads each, the last one possibly smaller:
    const int H0 = kExact ? (n + NG - 1) / NG : 4;   // exact: 5 heads are 3 + 2, not 4 + 1, and no warp multiplies for absent heads
    const int G = gridDim.x, cta = blockIdx.x;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&sm->full[s], 1); mbar_init(&sm->empty[s], kConsWarps); }
        sm->abort_flag = 0;
        sm->is_last = 0;
        mbar_fence_init();
    }
    if (kStep) {
        // the step's small inputs are read in the middle of the stream: start them towards L2 now (L2 is the point of
        // coherence, so this is safe before the wait below)
        const size_t row_bytes = size_t(n_slabs) * kRowBytes;
        for (size_t o = size_t(cta * kDecThreads + tid) * 128; o < row_bytes; o += size_t(G) * kDecThreads * 128) {
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(step.k_new) + o));
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(step.v_new) + o));
        }
        if (tid * 32 < n_slabs) asm volatile("prefetch.global.L2 [%0];" ::"l"(step.n_sent + tid * 32));
    }
    pdl_wait();                                          // inputs (and the workspace) may come from the kernel before
    // polls a wait makes before it gives up: the workspace's setting, or the default without a workspace
    uint32_t limit = kDefaultWaitLimit;
    if (wait_limit) { const uint32_t v = *reinterpret_cast<const volatile uint32_t*>(wait_limit); if (v) limit = v; }
    // tile prefix over slabs (its first barrier also publishes the barrier inits)
    cta_prefix<kDecThreads>(n_slabs, [&](int s) { return (live(s) + kTileRows - 1) / kTileRows; }, pref, sm->wsum);
    const int Ttot = pref[n_slabs];
    const int per_cta = max(1, (Ttot + G - 1) / G);
    const int t_begin = min(cta * per_cta, Ttot), t_end = min(t_begin + per_cta, Ttot);

    // slab holding tile t_begin: largest s with pref[s] <= t_begin and a non-empty slab
    int slab0 = 0;
    if (t_begin < t_end) {
        int lo = 0, hi = n_slabs - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (pref[mid] <= t_begin) lo = mid; else hi = mid - 1;
        }
        slab0 = lo;
    }

    {
        const int hg = warp % NG;                       // head group of this warp
        const int Hg = min(H0, n - hg * H0);            // its heads
        const int rb = warp / NG;                       // row block: rows [rb*NG*8, (rb+1)*NG*8) of each tile
        const int half = lane >> 4, l16 = lane & 15;
        const float qscale = 1.4426950408889634f * rsqrtf(float(kHeadDim));
        float2 q2[4][4], acc[4][4];
        float m_run = -INFINITY, l_run = 0.f;
        bool aborted = false;

        // ---- copy issue (thread 0 only): the CTA's k-th tile goes to stage k % kStages.  The cursor
        // walks the slab parts of this CTA's tile range; divisions and table reads happen once per part.
        const bool is_producer = (tid == 0);
        int p_slab = slab0, p_t = t_begin, p_rows_left = 0, p_stage = 0, p_j = 0;
        uint32_t p_phase = 0;                           // parity of the previous use of p_stage (first lap: no wait)
        bool p_first_lap = true;
        const uint8_t *p_K = K, *p_V = V;
        auto issue_next = [&]() {
            if (p_t >= t_end) return;
            if (p_rows_left <= 0) {
                while (pref[p_slab + 1] <= p_t) ++p_slab;
                const int j = p_t - pref[p_slab];
                if (!block_table) {
                    const size_t off =
                        (slab_row0(slab_off, cap, Hk, p_slab / Hk, p_slab % Hk) + size_t(j) * kTileRows) * kRowBytes;
                    p_K = K + off;
                    p_V = V + off;
                }
                p_j = j;
                p_rows_left = live(p_slab) - j * kTileRows;
            }
            if (block_table) {                          // paged cache: tile j of the slab lies in page block_table[slab][j / tiles per page]
                const size_t off = size_t(max(block_table[size_t(p_slab) * max_pages + p_j / kTilesPerPage], 0)) * kPageBytes +
                                   size_t(p_j % kTilesPerPage) * kTileBytes;
                p_K = K + off;
                p_V = V + off;
            }
            if (!p_first_lap) {
                if (sm->abort_flag || !mbar_wait(&sm->empty[p_stage], p_phase, limit)) {
                    if (!sm->abort_flag) atomicOr(status, SKIPKV_STATUS_COPY_TIMEOUT);
                    sm->abort_flag = 1;
                    return;
                }
            }
            const uint32_t bytes = uint32_t(min(kTileRows, p_rows_left)) * kRowBytes;
            uint8_t* dstK = ring + size_t(p_stage) * 2 * kTileBytes;
            mbar_expect_tx(&sm->full[p_stage], 2 * bytes);
            bulk_g2s(dstK, p_K, bytes, &sm->full[p_stage]);
            bulk_g2s(dstK + kTileBytes, p_V, bytes, &sm->full[p_stage]);
            p_K += kTileBytes;
            p_V += kTileBytes;
            p_rows_left -= kTileRows;
            ++p_t;
            ++p_j;
            if (++p_stage == kStages) {
                p_stage = 0;
                if (p_first_lap) p_first_lap = false; else p_phase ^= 1u;
            }
        };
        if (is_producer)
            for (int k = 0; k < kStages - 1; ++k) issue_next();
        // ------------------------------------------------------------------ steering add
        // Independent of the attention (its own tensor), so it runs here, behind the wait for the first tiles
        // whose copies were just issued, instead of lengthening the tail of the launch.
        if (hidden != nullptr) {
            const int vec_per_row = d_model / 8, total = batch * vec_per_row;
            for (int i = cta * kDecThreads + tid; i < total; i += G * kDecThreads)
                steer_vec8(i, vec_per_row, hidden, steer_vec, alpha, flag);
        }
        // fused step: this step's queries take their slot of the observation window
        if (kStep && step.q_win != nullptr) {
            const int total = batch * Hq * 16;
            for (int i = cta * kDecThreads + tid; i < total; i += G * kDecThreads)
                step.q_win[(size_t(i >> 4) * step.window + step.slot) * 16 + (i & 15)] = reinterpret_cast<const uint4*>(q)[i];
        }
        // fused step: new length and range list of a slab after the append (all consumer threads call this together)
        auto step_tables = [&](int slab_, int b_, bool appended, int S0, int starts_sentence) {
            const int len = old_len(slab_);
            const int new_len = appended ? len + 1 : len;
            int32_t* so = step.sent_off + size_t(slab_) * (step.max_sent + 1);
            const bool table_ok = S0 >= 0 && S0 <= step.max_sent;
            int S = S0;
            bool full_list = false;
            if (appended && table_ok && (S0 == 0 || starts_sentence)) {
                if (S0 < step.max_sent) S = S0 + 1; else full_list = true;   // full list: the token joins the last sentence
            }
            if (tid == 0) {
                step.kv_len_out[slab_] = new_len;
                if (appended && table_ok && S != S0) {
                    if (S0 == 0) so[0] = 0;
                    step.sent_id[size_t(slab_) * step.max_sent + S0] = step.gen_id[b_];
                    step.n_sent[slab_] = S;
                }
                if (!appended || !table_ok || full_list) atomicOr(status, SKIPKV_STATUS_BAD_TABLE);
            }
            if (appended && table_ok)
                for (int i = S + tid; i <= step.max_sent; i += kConsWarps * 32) so[i] = new_len;
        };

        int slab = slab0, t = t_begin, c_stage = 0;
        uint32_t c_phase = 0;
        while (t < t_end) {
            // ---------------------------------------------------------- one (CTA, slab) segment
            while (pref[slab + 1] <= t) ++slab;
            const int seg_end = min(t_end, pref[slab + 1]);
            const int b = slab / Hk, h = slab % Hk;
            int rows_left = live(slab) - (t - pref[slab]) * kTileRows;
            const bool seg_append = kStep && old_len(slab) < room(slab);   // fused step: a row joins this slab
            // fused step, this CTA holds the slab's last tile: fetch what the tail of the segment will need now, so
            // that the loads are long complete when they are used
            const bool own_tail = kStep && seg_end == pref[slab + 1];
            if (own_tail) {
                // the row being appended: into the cache, and staged as a one-row tile (K at byte 0, V at byte 2048 of
                // the merge buffer, which is idle until the flush) for the fold-in after the last streamed tile
                if (seg_append && warp == kConsWarps - 1) {
                    const int part = lane >> 4, c = lane & 15;
                    const uint4 val = (part ? step.v_new : step.k_new)[size_t(slab) * 16 + c];
                    reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(wpart) + part * 2048)[c] = val;
                    const size_t row = phys_row(slab, old_len(slab));
                    reinterpret_cast<uint4*>(const_cast<uint8_t*>(part ? V : K))[row * 16 + c] = val;
                }
                if (tid == kDecThreads - 33) { sm->step_n_sent = step.n_sent[slab]; sm->step_starts = step.new_sent[b]; }
            }
#pragma unroll
            for (int hh = 0; hh < 4; ++hh) {
                const int hl = hg * H0 + hh;
                uint4 qq = make_uint4(0u, 0u, 0u, 0u);
                if (hh < Hg)
                    qq = reinterpret_cast<const uint4*>(q + (size_t(b) * Hq + size_t(h) * n + hl) * kHeadDim)[l16];
                const float2 s2 = make_float2(qscale, qscale);
                q2[hh][0] = __fmul2_rn(bf16x2_to_f2(qq.x), s2);
                q2[hh][1] = __fmul2_rn(bf16x2_to_f2(qq.y), s2);
                q2[hh][2] = __fmul2_rn(bf16x2_to_f2(qq.z), s2);
                q2[hh][3] = __fmul2_rn(bf16x2_to_f2(qq.w), s2);
#pragma unroll
                for (int c = 0; c < 4; ++c) acc[hh][c] = make_float2(0.f, 0.f);
            }
            m_run = -INFINITY;
            l_run = 0.f;
            for (; t < seg_end; ++t, rows_left -= kTileRows) {
                if (is_producer) issue_next();                  // keeps kStages-1 tiles in flight
                if (!aborted) {
                    if (!mbar_wait(&sm->full[c_stage], c_phase, limit) || sm->abort_flag) {
                        if (!sm->abort_flag) atomicOr(status, SKIPKV_STATUS_COPY_TIMEOUT);
                        sm->abort_flag = 1;
                        aborted = true;
                    }
                }
                if (!aborted) {
                    const uint8_t* Ks = ring + size_t(c_stage) * 2 * kTileBytes;
                    const uint8_t* Vs = Ks + kTileBytes;
                    if (rows_left >= kTileRows) {
                        for (int sub = 0; sub < NG; ++sub)
                            tile_rows<false, kExact>(Hg, Ks, Vs, (rb * NG + sub) * 8, kTileRows, lane, q2, acc, m_run, l_run);
                    } else {
                        for (int sub = 0; sub < NG; ++sub) {
                            const int row_base = (rb * NG + sub) * 8;
                            if (row_base >= rows_left) break;
                            tile_rows<true, kExact>(Hg, Ks, Vs, row_base, rows_left, lane, q2, acc, m_run, l_run);
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sm->empty[c_stage]);
                }
                if (++c_stage == kStages) { c_stage = 0; c_phase ^= 1u; }
            }

            // ---------------------------------------------------------- fused step: this CTA held the slab's last tile
            if (own_tail && seg_append) {
                consumer_bar();                            // the staged row is visible
                if (warp < NG && !aborted)                 // one warp per head group folds the row into its running state
                    tile_rows<true, kExact>(Hg, reinterpret_cast<const uint8_t*>(wpart), reinterpret_cast<const uint8_t*>(wpart) + 2048, 0, 1,
                                    lane, q2, acc, m_run, l_run);
                consumer_bar();                            // before the flush reuses the buffer
            }
            if (own_tail) {
                consumer_bar();                            // the values parked at the start of the segment are visible
                step_tables(slab, b, seg_append, sm->step_n_sent, sm->step_starts);
            }
            // ---------------------------------------------------------- flush this (CTA, slab) segment
            // halves of the warp hold different rows: add them; finish the sum of p
#pragma unroll
            for (int hh = 0; hh < 4; ++hh)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    acc[hh][c].x += __shfl_xor_sync(0xffffffffu, acc[hh][c].x, 16);
                    acc[hh][c].y += __shfl_xor_sync(0xffffffffu, acc[hh][c].y, 16);
                }
            l_run += __shfl_xor_sync(0xffffffffu, l_run, 4);
            l_run += __shfl_xor_sync(0xffffffffu, l_run, 8);
            l_run += __shfl_xor_sync(0xffffffffu, l_run, 16);
            float* wp = wpart + size_t(warp) * 4 * kWpStride;
            if (half == 0) {
#pragma unroll
                for (int hh = 0; hh < 4; ++hh) {
                    float4* dst = reinterpret_cast<float4*>(wp + hh * kWpStride + l16 * 8);
                    dst[0] = make_float4(acc[hh][0].x, acc[hh][0].y, acc[hh][1].x, acc[hh][1].y);
                    dst[1] = make_float4(acc[hh][2].x, acc[hh][2].y, acc[hh][3].x, acc[hh][3].y);
                }
            }
            if (lane < 4) {
                wp[lane * kWpStride + 128] = m_run;
                wp[lane * kWpStride + 129] = l_run;
            }
            consumer_bar();
            // merge the warps of each head group; thread -> (head, channel) pairs
            const int fc = pref[slab] / per_cta, lc = (pref[slab + 1] - 1) / per_cta;
            const int n_part = lc - fc + 1;
            __nv_bfloat16* o = out + (size_t(b) * Hq + size_t(h) * n) * kHeadDim;
            float* rec = dec_part + size_t(cta + slab) * n * kPartStride;
            for (int idx = tid; idx < n * kHeadDim; idx += kConsWarps * 32) {
                const int hl = idx / kHeadDim, c = idx % kHeadDim;
                const int g2 = hl / H0, hh = hl % H0;
                float M = -INFINITY;
                for (int w = g2; w < kConsWarps; w += NG) M = fmaxf(M, wpart[(w * 4 + hh) * kWpStride + 128]);
                float L = 0.f, A = 0.f;
                for (int w = g2; w < kConsWarps; w += NG) {
                    const float* p = wpart + (w * 4 + hh) * kWpStride;
                    const float e = ex2(p[128] - M);
                    L += p[129] * e;
                    A += p[c] * e;
                }
                if (n_part == 1) {
                    o[idx] = __float2bfloat16_rn(L > 0.f ? A / L : 0.f);
                } else {
                    rec[hl * kPartStride + c] = A;
                    if (c == 0) { rec[hl * kPartStride + 128] = M; rec[hl * kPartStride + 129] = L; }
                }
            }
            if (n_part > 1) {
                consumer_bar();                            // every thread's record stores are ordered before ...
                if (tid == 0) {
                    __threadfence();                       // ... this fence, which publishes them with the arrival below
                    const uint32_t old = atomicAdd(dec_cnt + slab, 1u);
                    const int last = (old == uint32_t(n_part - 1)) ? 1 : 0;
                    if (last) dec_cnt[slab] = 0u;          // self-resetting for the next launch
                    sm->is_last = last;
                }
                consumer_bar();
                if (sm->is_last) {
                    __threadfence();
                    const float* r0 = dec_part + size_t(fc + slab) * n * kPartStride;
                    for (int idx = tid; idx < n * kHeadDim; idx += kConsWarps * 32) {
                        const int hl = idx / kHeadDim, c = idx % kHeadDim;
                        // four records per round: their loads are all in flight before the first is used
                        float M = -INFINITY, L = 0.f, A = 0.f;
                        for (int p0 = 0; p0 < n_part; p0 += 4) {
                            float mm[4], ll[4], aa[4];
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                const float* rp = r0 + (size_t(min(p0 + k, n_part - 1)) * n + hl) * kPartStride;
                                mm[k] = (p0 + k < n_part) ? __ldcg(rp + 128) : -INFINITY;
                                ll[k] = __ldcg(rp + 129);
                                aa[k] = __ldcg(rp + c);
                            }
                            float Mn = M;
#pragma unroll
                            for (int k = 0; k < 4; ++k) Mn = fmaxf(Mn, mm[k]);
                            const float keep = ex2(M - Mn);              // first round: 2^(-inf) = 0
                            L *= keep; A *= keep;
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                const float e = ex2(mm[k] - Mn);         // absent records: 2^(-inf) = 0
                                L = fmaf(ll[k], e, L);
                                A = fmaf(aa[k], e, A);
                            }
                            M = Mn;
                        }
                        o[idx] = __float2bfloat16_rn(L > 0.f ? A / L : 0.f);
                    }
                }
            }
            consumer_bar();                                // wpart and is_last reusable
        }
        // after an abort copies may still be in flight: they must land before the CTA retires
        if (is_producer && sm->abort_flag)
            for (int st = 0; st < kStages; ++st) { mbar_wait(&sm->full[st], 0u, 1u << 16); mbar_wait(&sm->full[st], 1u, 1u << 16); }
        // slabs with no live row: zeros (owned round-robin)
        for (int s = cta; s < n_slabs; s += G) {
            if (live(s) > 0) continue;
            const int b = s / Hk, h = s % Hk;
            __nv_bfloat16* o = out + (size_t(b) * Hq + size_t(h) * n) * kHeadDim;
            if (kStep && room(s) > 0) {
                // fused step on an empty slab: the appended row is its only row, so every head's output is that value row
                const __nv_bfloat16* vrow = reinterpret_cast<const __nv_bfloat16*>(step.v_new) + size_t(s) * kHeadDim;
                for (int idx = tid; idx < n * kHeadDim; idx += kConsWarps * 32) o[idx] = vrow[idx % kHeadDim];
                if (tid < 32) {
                    const int part = tid >> 4, c = tid & 15;
                    const size_t row = phys_row(s, 0);
                    reinterpret_cast<uint4*>(const_cast<uint8_t*>(part ? V : K))[row * 16 + c] =
                        (part ? step.v_new : step.k_new)[size_t(s) * 16 + c];
                }
                const int S0 = step.n_sent[s], starts = step.new_sent[b];
                consumer_bar();                            // every thread has read n_sent before it changes
                step_tables(s, b, true, S0, starts);
            } else {
                for (int idx = tid; idx < n * kHeadDim; idx += kConsWarps * 32) o[idx] = __float2bfloat16_rn(0.f);
                if (kStep) step_tables(s, b, false, 0, 0);  // no room: unchanged, reported
            }
        }
    }
}

}  // namespace skipkv

using namespace skipkv;

static int decode_impl(const skipkv_shape* shape, const void* q, const void* K, const void* V, const int32_t* kv_len,
                       void* out, void* hidden, const void* steer_vec, const float* alpha, const uint8_t* flag,
                       const int32_t* block_table, int max_pages, const StepArgs& step, void* ws, void* stream) {
    if (int rc = check_shape(shape)) return rc;
    if (!q || !K || !V || !kv_len || !out) return SKIPKV_ERR_INVALID_ARG;
    if (hidden && (!steer_vec || !alpha || !flag || shape->d_model <= 0)) return SKIPKV_ERR_INVALID_ARG;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255)) return SKIPKV_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(K) & 15) || (reinterpret_cast<uintptr_t>(V) & 15) ||
        (reinterpret_cast<uintptr_t>(q) & 15))
        return SKIPKV_ERR_INVALID_ARG;
    const WsLayout L = make_layout(*shape);
    if (L.slabs > kMaxDecSlabs) return SKIPKV_ERR_UNSUPPORTED;
    uint8_t* w = static_cast<uint8_t*>(ws);
    const size_t smem = size_t(kStages) * 2 * kTileBytes + size_t(kConsWarps) * 4 * kWpStride * 4 + sizeof(DecSmem) +
                        size_t(L.slabs + 1) * 4;
    if (smem > 227 * 1024) {                         // the per-slab tile table no longer fits beside the tile ring
        set_error_text("skipkv_decode_attn: batch * n_kv_heads too large for the shared-memory tile table");
        return SKIPKV_ERR_UNSUPPORTED;
    }
    // set on every call: the attribute belongs to the current device's context, which a cached value would not track
    const bool exact = (shape->n_q_heads / shape->n_kv_heads) % 4 != 0;
    auto kern = step.k_new ? (exact ? decode_attn_kernel<true, true> : decode_attn_kernel<true, false>)
                           : (exact ? decode_attn_kernel<false, true> : decode_attn_kernel<false, false>);
    SKIPKV_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
    int grid = num_sms() * kCtasPerSm;
    if (grid > L.dec_max_ctas) grid = L.dec_max_ctas;
    SKIPKV_CUDA(launch_dependent(
        kern, dim3(grid), dim3(kDecThreads), smem, static_cast<cudaStream_t>(stream), int(shape->batch),
        int(shape->n_q_heads), int(shape->n_kv_heads), int(L.slabs), shape->slab_off, shape->cap,
        static_cast<const __nv_bfloat16*>(q), static_cast<const uint8_t*>(K), static_cast<const uint8_t*>(V), kv_len,
        static_cast<__nv_bfloat16*>(out), &reinterpret_cast<Header*>(w + L.header)->status,
        reinterpret_cast<uint32_t*>(w + L.dec_cnt), reinterpret_cast<float*>(w + L.dec_part), int(shape->d_model),
        static_cast<__nv_bfloat16*>(hidden), static_cast<const __nv_bfloat16*>(steer_vec), alpha, flag, block_table,
        max_pages, step, static_cast<const uint32_t*>(&reinterpret_cast<Header*>(w + L.header)->wait_limit)));
    return SKIPKV_OK;
}

extern "C" int skipkv_decode_attn(const skipkv_shape* shape, const void* q, const void* K, const void* V,
                                  const int32_t* kv_len, void* out, void* hidden, const void* steer_vec,
                                  const float* alpha, const uint8_t* flag, void* ws, void* stream) {
    return decode_impl(shape, q, K, V, kv_len, out, hidden, steer_vec, alpha, flag, nullptr, 0, StepArgs{}, ws, stream);
}

extern "C" int skipkv_decode_attn_paged(const skipkv_shape* shape, const void* q, const void* K_pages,
                                        const void* V_pages, const int32_t* block_table, int32_t max_pages,
                                        const int32_t* kv_len, void* out, void* hidden, const void* steer_vec,
                                        const float* alpha, const uint8_t* flag, void* ws, void* stream) {
    if (!block_table || max_pages <= 0) return SKIPKV_ERR_INVALID_ARG;
    return decode_impl(shape, q, K_pages, V_pages, kv_len, out, hidden, steer_vec, alpha, flag, block_table, max_pages,
                       StepArgs{}, ws, stream);
}

extern "C" int skipkv_decode_step(const skipkv_shape* shape, const void* q, const void* k_new, const void* v_new, void* K,
                                  void* V, const int32_t* kv_len_in, int32_t* kv_len_out, int32_t* sent_off,
                                  int32_t* sent_id, int32_t* n_sent, const uint8_t* new_sent, const int32_t* gen_id,
                                  void* q_win, int32_t slot, void* out, void* hidden, const void* steer_vec,
                                  const float* alpha, const uint8_t* flag, void* ws, void* stream) {
    if (!k_new || !v_new || !kv_len_in || !kv_len_out || kv_len_in == kv_len_out || !sent_off || !sent_id || !n_sent ||
        !new_sent || !gen_id)
        return SKIPKV_ERR_INVALID_ARG;
    if (int rc = check_shape(shape)) return rc;
    if (shape->max_sent <= 0) return SKIPKV_ERR_INVALID_ARG;
    if (q_win && (slot < 0 || slot >= shape->window)) return SKIPKV_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(k_new) | reinterpret_cast<uintptr_t>(v_new) | reinterpret_cast<uintptr_t>(q_win)) & 15)
        return SKIPKV_ERR_INVALID_ARG;
    StepArgs step{};
    step.k_new = static_cast<const uint4*>(k_new); step.v_new = static_cast<const uint4*>(v_new);
    step.kv_len_out = kv_len_out; step.sent_off = sent_off; step.sent_id = sent_id; step.n_sent = n_sent;
    step.new_sent = new_sent; step.gen_id = gen_id; step.q_win = static_cast<uint4*>(q_win);
    step.window = shape->window; step.slot = slot; step.max_sent = shape->max_sent;
    return decode_impl(shape, q, K, V, kv_len_in, out, hidden, steer_vec, alpha, flag, nullptr, 0, step, ws, stream);
}

extern "C" int skipkv_decode_step_paged(const skipkv_shape* shape, const void* q, const void* k_new, const void* v_new,
                                        void* K_pages, void* V_pages, const int32_t* block_table, int32_t max_pages,
                                        const int32_t* kv_len_in, int32_t* kv_len_out, int32_t* sent_off, int32_t* sent_id,
                                        int32_t* n_sent, const uint8_t* new_sent, const int32_t* gen_id, void* q_win,
                                        int32_t slot, void* out, void* hidden, const void* steer_vec, const float* alpha,
                                        const uint8_t* flag, void* ws, void* stream) {
    if (!block_table || max_pages <= 0) return SKIPKV_ERR_INVALID_ARG;
    if (!k_new || !v_new || !kv_len_in || !kv_len_out || kv_len_in == kv_len_out || !sent_off || !sent_id || !n_sent ||
        !new_sent || !gen_id)
        return SKIPKV_ERR_INVALID_ARG;
    if (int rc = check_shape(shape)) return rc;
    if (shape->max_sent <= 0) return SKIPKV_ERR_INVALID_ARG;
    if (q_win && (slot < 0 || slot >= shape->window)) return SKIPKV_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(k_new) | reinterpret_cast<uintptr_t>(v_new) | reinterpret_cast<uintptr_t>(q_win)) & 15)
        return SKIPKV_ERR_INVALID_ARG;
    StepArgs step{};
    step.k_new = static_cast<const uint4*>(k_new); step.v_new = static_cast<const uint4*>(v_new);
    step.kv_len_out = kv_len_out; step.sent_off = sent_off; step.sent_id = sent_id; step.n_sent = n_sent;
    step.new_sent = new_sent; step.gen_id = gen_id; step.q_win = static_cast<uint4*>(q_win);
    step.window = shape->window; step.slot = slot; step.max_sent = shape->max_sent;
    return decode_impl(shape, q, K_pages, V_pages, kv_len_in, out, hidden, steer_vec, alpha, flag, block_table, max_pages, step,
                       ws, stream);
}

// ---------------------------------------------------------------------------------------------
// Decode attention for callers that cannot provide a workspace.
//
// Some callers have no device allocator to draw scratch from: a serving process that handed every
// free byte of HBM to its KV-cache pool at start-up (so a later cudaMalloc would fail), or a
// plug-in that is forbidden to allocate because cudaMalloc synchronises the whole device and would
// stall the other streams of the process.  For them the partial results and arrival counters of
// the kernel live in the fixed array below, which every GPU that loads this library holds until
// the process exits (about 2 MB).  Sizes are therefore capped: at most SKIPKV_STATIC_MAX_SLABS
// (sequence, head) slabs and a decode grid of at most kStaticMaxCtas CTAs.
//
// The array's name is only a host-side handle in host code; the device address is looked up once
// per device with cudaGetSymbolAddress (with that device current) and handed to the kernel.
// ---------------------------------------------------------------------------------------------
namespace skipkv {

constexpr int kStaticMaxSlabs = SKIPKV_STATIC_MAX_SLABS;
constexpr int kStaticMaxCtas = 256;
constexpr size_t kStaticCntOff = 256;                                      // after the status word
constexpr size_t kStaticPartOff = kStaticCntOff + size_t(kStaticMaxSlabs) * 4;
constexpr size_t kStaticBytes =
    kStaticPartOff + size_t(kStaticMaxCtas + kStaticMaxSlabs) * kMaxGroup * kPartStride * 4;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
static unsigned char* g_static_addr[kMaxDevices];      // device address of the array, per device
static bool g_static_ready[kMaxDevices];
static std::mutex g_static_mutex;

// First call on a device: resolve the array's device address.  Later calls only read the cached pointer.
static int static_setup(int dev, unsigned char** base) {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ready[dev]) {
        void* p = nullptr;
        SKIPKV_CUDA(cudaGetSymbolAddress(&p, g_static_scratch));
        if (!p) return SKIPKV_ERR_CUDA;
        g_static_addr[dev] = static_cast<unsigned char*>(p);
        g_static_ready[dev] = true;
    }
    *base = g_static_addr[dev];
    return SKIPKV_OK;
}

}  // namespace skipkv

extern "C" int skipkv_decode_attn_static(const skipkv_shape* shape, const void* q, const void* K, const void* V,
                                         const int32_t* kv_len, void* out, void* hidden, const void* steer_vec,
                                         const float* alpha, const uint8_t* flag, uint32_t* status, void* stream) {
    if (int rc = check_shape(shape)) return rc;
    if (!q || !K || !V || !kv_len || !out) return SKIPKV_ERR_INVALID_ARG;
    if (hidden && (!steer_vec || !alpha || !flag || shape->d_model <= 0)) return SKIPKV_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(K) & 15) || (reinterpret_cast<uintptr_t>(V) & 15) ||
        (reinterpret_cast<uintptr_t>(q) & 15))
        return SKIPKV_ERR_INVALID_ARG;
    const int slabs = shape->batch * shape->n_kv_heads;
    if (slabs > kStaticMaxSlabs) {
        char msg[160];
        std::snprintf(msg, sizeof(msg),
                      "skipkv_decode_attn_static: batch*n_kv_heads = %d exceeds SKIPKV_STATIC_MAX_SLABS = %d; "
                      "use skipkv_decode_attn with a workspace",
                      slabs, kStaticMaxSlabs);
        set_error_text(msg);
        return SKIPKV_ERR_UNSUPPORTED;
    }
    int dev = 0;
    SKIPKV_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) {
        set_error_text("skipkv_decode_attn_static: device ordinal beyond 63");
        return SKIPKV_ERR_UNSUPPORTED;
    }
    const size_t smem = size_t(kStages) * 2 * kTileBytes + size_t(kConsWarps) * 4 * kWpStride * 4 + sizeof(DecSmem) +
                        size_t(slabs + 1) * 4;
    unsigned char* base = nullptr;
    if (int rc = static_setup(dev, &base)) return rc;
    SKIPKV_CUDA(cudaFuncSetAttribute(decode_attn_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // The array keeps whatever the previous call left: the status word and the arrival counters
    // must start at zero (the partial records are fully written before they are read).
    SKIPKV_CUDA(cudaMemsetAsync(base, 0, kStaticPartOff, st));
    int grid = num_sms() * kCtasPerSm;
    if (grid > kStaticMaxCtas) grid = kStaticMaxCtas;
    uint32_t* status_word = status ? status : reinterpret_cast<uint32_t*>(base);
    decode_attn_kernel<false, false><<<grid, kDecThreads, smem, st>>>(
        shape->batch, shape->n_q_heads, shape->n_kv_heads, slabs, shape->slab_off, shape->cap,
        static_cast<const __nv_bfloat16*>(q), static_cast<const uint8_t*>(K), static_cast<const uint8_t*>(V), kv_len,
        static_cast<__nv_bfloat16*>(out), status_word, reinterpret_cast<uint32_t*>(base + kStaticCntOff),
        reinterpret_cast<float*>(base + kStaticPartOff), shape->d_model, static_cast<__nv_bfloat16*>(hidden),
        static_cast<const __nv_bfloat16*>(steer_vec), alpha, flag, static_cast<const int32_t*>(nullptr), 0, StepArgs{},
        static_cast<const uint32_t*>(nullptr));
    SKIPKV_CUDA(cudaGetLastError());
    return SKIPKV_OK;
}
