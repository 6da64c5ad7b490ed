// skipkv_score: sentence scores per (sequence, KV head) slab (paper Section 4.1).
//
//   sweep 1   log-sum-exp of every window-query row over the slab's tokens
//             (tensor cores: logits = Q_group x K_tile^T, one thread per query row)
//   sweep 2   tok_imp[t] = (1/alpha) sum_w max_q 2^(s_q[w][t] - lse_q[w])   (max before exp: exp is monotone)
//             (tensor cores: logits = K_tile x Q_group^T, one thread per token), and in the same pass
//             the per-sentence sums of the key rows as a second product on the tile already in shared
//             memory: K_tile^T x (0/1 matrix token -> sentence slot)
//   pool      per sentence: mean tok_imp, mean key, normalisation, split into bf16 high and low parts
//   gram x2   pairwise cosine G on the tensor cores (three bf16 products: hi.hi + hi.lo + lo.hi);
//             pass 1: Z_i = sum_{j!=i} e^{G_ij} and lam_i = max_{j>i} G_ij;
//             pass 2: red_i = (1/S) sum_{j!=i} e^{G_ij} / Z_j (G symmetric) and the final score.
//
// Logits are kept in base 2: s = (q.k) * log2(e)/sqrt(d).  |G| <= 1 so the row softmax of G
// needs no max subtraction.
//
// Both sweeps are persistent, warp-specialised kernels, one CTA per SM: a TMA warp streams
// 128-token key tiles (and the group's query block) into shared memory, one thread issues
// tcgen05.mma into a ring of tensor-memory accumulators (four in sweep 1, three in sweep 2), several
// warpgroups of epilogue warps take the tiles round-robin, and (sweep 2) one more warpgroup writes the 0/1
// matrices of the pooling product and reads out the pooled sums while one thread of a further warp issues
// that product.  Work is the list of 128-token tiles over all slabs cut into equal contiguous ranges, so
// ragged slabs balance.
//
// Query rows of a group are staged as blocks of WB = floor(128/n) window positions x n heads
// (row q*WB + w of a block), so that the n heads of a window position sit at a fixed column
// stride for the max over heads.
#include <cstddef>

#include "common.cuh"
#include "tc.cuh"

namespace skipkv {

constexpr int kAccBufs = 4;             // tensor-memory accumulators of 128 columns
constexpr int kMaxRB = 4;               // query blocks per group
constexpr int kSwMaxStages = 6;
constexpr int kSw1Groups = 4;           // epilogue warpgroups of sweep 1
constexpr int kSw2Groups = 2;           // epilogue warpgroups of sweep 2
constexpr int kSw2Bufs = 3;             // sweep 2: accumulators of the logits (the columns after them hold the pooled sums)
constexpr int kPoolWarps = 4;           // sweep 2: the warpgroup that writes the indicator matrices and drains the pooled sums
constexpr int kIndRing = 2;             // indicator matrices in flight (the pooled sums have two accumulators of their own)
constexpr int kIndSlots = 16;           // sentence slots of one indicator matrix
constexpr int kIndBytes = kIndSlots * 128 * 2;   // [16 slots][128 tokens] bf16 as two 64-token halves, 128-byte swizzle
constexpr uint32_t kPoolCol = kSw2Bufs * 128;    // tensor-memory column of the first pooled-sum accumulator (16 columns each)
constexpr int kSw1Threads = (2 + 4 * kSw1Groups) * 32;        // TMA warp, MMA warp, epilogue warps
constexpr int kSw2Threads = (2 + 4 * kSw2Groups + kPoolWarps + 1) * 32;   // + the thread that issues the pooling products
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

struct SweepCtl {                       // barriers and small shared state, after the tile buffers
    uint64_t full[kSwMaxStages], empty[kSwMaxStages];
    uint64_t qfull, qempty;
    // "accumulator ready" barriers are per epilogue warpgroup (a ring of 4 per group, indexed by the group's own item
    // count), so every barrier has one consumer that sees its phases in order; a barrier per accumulator would be
    // waited on by different groups in turn, and a group polling for a later phase could pass on an earlier one.
    uint64_t tfull[4][4], tempty[kAccBufs];
    uint32_t tmem_base;
    int abort_flag;
    // sweep 2, ring of indicator matrices: written by the four pooling warps -> multiplied by the MMA thread -> drained by
    // the pooling warps
    uint64_t ifull[kIndRing], iempty[kIndRing];
    uint64_t pfull[2];                  // the last product of a run of tiles into accumulator i has completed
    uint64_t issued_done[2];            // after a failed wait: every product of the MMA thread (0) / the pooling issuer (1) has retired
    int ind_flags[kIndRing];            // 1: the tile has another matrix after this one, 2: joins the open run, 4: closes a run
    uint32_t wsum[32];
    alignas(16) float neg_lse[kSw2Groups][kMaxRB * 128];   // sweep 2: one copy per epilogue warpgroup (read as float4)
};
static_assert(offsetof(SweepCtl, neg_lse) % 16 == 0, "neg_lse is read with 16-byte loads");

struct SweepArgs {
    int Hq, Hk, window, n_slabs, max_cap, max_sent, RB, WB, stages;
    const int64_t* slab_off;
    const int32_t* cap;
    const int32_t* kv_len;
    const int32_t* sent_off;
    const int32_t* n_sent;
    float2* sc_part;                    // [(cta + slab) * kSw1Groups + warpgroup][RB * 128] (max, sum)
    float* tok_imp_user;
    float* tok_imp_ws;
    float* vsum;                        // [slabs][max_sent][128] sums of key rows
    uint32_t* status;
    const Header* hdr;
    const int32_t* block_table;         // nullable: paged cache, tile j of slab s is page block_table[s * max_pages + j]
    int max_pages;
};

// ---- sweep 1 epilogue: one accumulator (128 tokens) folded into the running (max, sum) of a row
// (The loop over the four 32-column pieces is kept rolled, here and in imp_fold for four heads per group: the epilogue
// code is fetched again for every tile, and unrolled it stalls on instruction fetch more than the loop costs.)
template <bool kMasked>
__device__ __forceinline__ void lse_fold(uint32_t taddr, int valid, float scale, float& m, float& l) {
    const int nch = kMasked ? (valid + 31) >> 5 : 4;
#pragma unroll 1
    for (int ch = 0; ch < nch; ++ch) {
        float v[32];
        tmem_ld32(taddr + ch * 32, v);
        if (kMasked && ch * 32 + 32 > valid) {
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (ch * 32 + j >= valid) v[j] = -INFINITY;
        }
        float c0 = fmaxf(v[0], v[1]), c1 = fmaxf(v[2], v[3]);
#pragma unroll
        for (int j = 4; j < 32; j += 2) { c0 = fmaxf(c0, v[j]); c1 = fmaxf(c1, v[j + 1]); }
        const float m_new = fmaxf(m, fmaxf(c0, c1) * scale);
        const float neg = -m_new;
        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
            s0 += ex2f(fmaf(v[j + 0], scale, neg));
            s1 += ex2f(fmaf(v[j + 1], scale, neg));
            s2 += ex2f(fmaf(v[j + 2], scale, neg));
            s3 += ex2f(fmaf(v[j + 3], scale, neg));
        }
        l = l * ex2f(m - m_new) + ((s0 + s1) + (s2 + s3));      // first chunk: 2^(-inf) = 0
        m = m_new;
    }
}

// ---- sweep 2 epilogue: one accumulator (this thread's token x one query block) added to the token's total
template <int kN>
__device__ __forceinline__ float imp_fold(uint32_t taddr, const float* neg_lse, int wvalid, float scale) {
    constexpr int WB = 128 / kN;
    if constexpr (kN == 4) {
        float b4[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) b4[j] = -INFINITY;
#pragma unroll 1
        for (int q = 0; q < 4; ++q) {
            float v[32];
            tmem_ld32(taddr + q * 32, v);
#pragma unroll
            for (int j4 = 0; j4 < 32; j4 += 4) {
                const float4 nl = *reinterpret_cast<const float4*>(neg_lse + q * 32 + j4);
                b4[j4 + 0] = fmaxf(b4[j4 + 0], fmaf(v[j4 + 0], scale, nl.x));
                b4[j4 + 1] = fmaxf(b4[j4 + 1], fmaf(v[j4 + 1], scale, nl.y));
                b4[j4 + 2] = fmaxf(b4[j4 + 2], fmaf(v[j4 + 2], scale, nl.z));
                b4[j4 + 3] = fmaxf(b4[j4 + 3], fmaf(v[j4 + 3], scale, nl.w));
            }
        }
        float t0 = 0.f, t1 = 0.f;
#pragma unroll
        for (int j = 0; j < 32; j += 2) {
            t0 += (j < wvalid) ? ex2f(b4[j]) : 0.f;
            t1 += (j + 1 < wvalid) ? ex2f(b4[j + 1]) : 0.f;
        }
        return t0 + t1;
    }
    if constexpr (kN > 4) {
        // WB <= 25 window positions per head: one load of 32 columns per head, starting at the head's first column
        // (the columns read past its last position are not used), in a rolled loop like the four-head case
        float best[WB];
#pragma unroll
        for (int w = 0; w < WB; ++w) best[w] = -INFINITY;
#pragma unroll 1
        for (int q = 0; q < kN; ++q) {
            float v[32];
            tmem_ld32(taddr + q * WB, v);
            const float* nl = neg_lse + q * WB;
#pragma unroll
            for (int w = 0; w < WB; ++w) best[w] = fmaxf(best[w], fmaf(v[w], scale, nl[w]));
        }
        float t0 = 0.f, t1 = 0.f;
#pragma unroll
        for (int w = 0; w < WB; w += 2) {
            t0 += (w < wvalid) ? ex2f(best[w]) : 0.f;
            if (w + 1 < WB) t1 += (w + 1 < wvalid) ? ex2f(best[w + 1]) : 0.f;
        }
        return t0 + t1;
    }
    float best[WB];
    float total = 0.f;
#pragma unroll
    for (int ch = 0; ch < 4; ++ch) {
        if (ch * 32 >= kN * WB) break;
        float v[32];
        tmem_ld32(taddr + ch * 32, v);
#pragma unroll
        for (int j4 = 0; j4 < 32; j4 += 4) {
            const float4 nl = *reinterpret_cast<const float4*>(neg_lse + ch * 32 + j4);
            const float nls[4] = {nl.x, nl.y, nl.z, nl.w};
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                const int c = ch * 32 + j4 + jj;
                if (c < kN * WB) {
                    const int q = c / WB, w = c % WB;
                    const float x = fmaf(v[j4 + jj], scale, nls[jj]);
                    best[w] = (q == 0) ? x : fmaxf(best[w], x);
                    if (q == kN - 1) total += (w < wvalid) ? ex2f(best[w]) : 0.f;
                }
            }
        }
    }
    return total;
}

// ---- sweep 2: pooled key sums on the tensor cores
// Pooling product of one staged tile: D[128 channels x 16 slots] = K_tile^T x Ind^T.  A = the tile as the TMA load
// wrote it ([token][channel], two 64-channel halves, 128-byte swizzle) read as an MN-major operand: 64 channels x 8
// tokens per swizzle atom, atoms 1024 bytes apart along the tokens and a half (16 KB) apart along the channels.
// B = the indicator matrix [slot][token], K-major like every other operand here.
constexpr uint32_t kIdescPool = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | ((uint32_t(kIndSlots) >> 3) << 17) |
                                ((128u >> 4) << 24);
__device__ __forceinline__ void umma_pool(uint32_t tmem_d, uint32_t tile_smem, uint32_t ind_smem, bool accumulate) {
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {                     // 16 tokens per step
        const uint32_t a_addr = tile_smem + ks * 2048;
        const uint64_t da = uint64_t((a_addr >> 4) & 0x3fffu) | (uint64_t(kOpHalfBytes >> 4) << 16) |
                            (uint64_t(1024 >> 4) << 32) | (uint64_t(1) << 46) | (uint64_t(2) << 61);
        const uint64_t db = umma_desc_sw128(ind_smem + (ks >> 2) * (kIndBytes / 2) + (ks & 3) * 32);
        umma_bf16(tmem_d, da, db, kIdescPool, (accumulate || ks) ? 1u : 0u);
    }
}
// 16 consecutive fp32 columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
// One 16-byte piece of an indicator matrix: tokens 8c .. 8c + 7 of slot row j; ones (bf16 1.0) for the tokens
// [lo, hi), zeros elsewhere.
__device__ __forceinline__ void indicator_piece(uint8_t* ind, int j, int c, int lo, int hi) {
    const int b0 = min(max(lo - 8 * c, 0), 8), b1 = min(max(hi - 8 * c, 0), 8);
    const uint32_t m8 = b1 > b0 ? (((1u << b1) - 1u) & ~((1u << b0) - 1u)) : 0u;
    uint4 val;
    val.x = (m8 & 1u) * 0x3F80u + ((m8 >> 1) & 1u) * 0x3F800000u;
    val.y = ((m8 >> 2) & 1u) * 0x3F80u + ((m8 >> 3) & 1u) * 0x3F800000u;
    val.z = ((m8 >> 4) & 1u) * 0x3F80u + ((m8 >> 5) & 1u) * 0x3F800000u;
    val.w = ((m8 >> 6) & 1u) * 0x3F80u + ((m8 >> 7) & 1u) * 0x3F800000u;
    *reinterpret_cast<uint4*>(ind + (c >> 3) * (kIndBytes / 2) + j * 128 + (((c & 7) ^ (j & 7)) << 4)) = val;
}

template <int kSweep, int kN>
__global__ void __launch_bounds__(kSweep == 1 ? kSw1Threads : kSw2Threads, 1)
score_sweep_kernel(const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapQ,
                   const SweepArgs a) {
    extern __shared__ uint8_t sweep_smem_raw[];
    constexpr int kThreads = kSweep == 1 ? kSw1Threads : kSw2Threads;
    constexpr int kGroups = kSweep == 1 ? kSw1Groups : kSw2Groups;
    const uint32_t raw = smem_u32(sweep_smem_raw);
    uint8_t* tiles = sweep_smem_raw + (((raw + 1023u) & ~1023u) - raw);          // 1024-byte aligned
    uint8_t* qbuf = tiles + size_t(a.stages) * kOpBytes;
    uint8_t* indb = qbuf + size_t(a.RB) * kOpBytes;                              // sweep 2: the indicator matrices
    SweepCtl* ctl = reinterpret_cast<SweepCtl*>(indb + (kSweep == 2 ? kIndRing * kIndBytes : 0));
    int* pref = reinterpret_cast<int*>(ctl + 1);                                 // [n_slabs + 1] tile prefix

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int G = gridDim.x, cta = blockIdx.x;
    const int n_slabs = a.n_slabs, Hk = a.Hk, RB = a.RB;
    pdl_trigger();
    auto live = [&](int s) {
        const int room = a.block_table ? min(a.cap[s / Hk], a.max_pages * 128) : a.cap[s / Hk];
        return min(max(a.kv_len[s], 0), room);
    };

    if (tid == 0) {
        for (int s = 0; s < kSwMaxStages; ++s) {
            mbar_init(&ctl->full[s], 1);
            mbar_init(&ctl->empty[s], kSweep == 1 ? 1 : 2);      // commit of the logits (+ commit of the tile's last pooling product)
        }
        mbar_init(&ctl->qfull, 1);
        mbar_init(&ctl->qempty, 1);
        for (int b = 0; b < kAccBufs; ++b) mbar_init(&ctl->tempty[b], 4);
        for (int g = 0; g < 4; ++g)
            for (int j = 0; j < 4; ++j) mbar_init(&ctl->tfull[g][j], 1);
        for (int i = 0; i < kIndRing; ++i) { mbar_init(&ctl->ifull[i], kPoolWarps); mbar_init(&ctl->iempty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&ctl->pfull[i], 1); mbar_init(&ctl->issued_done[i], 1); }
        ctl->abort_flag = 0;
        mbar_fence_init();
        tmap_prefetch(&mapK);
        tmap_prefetch(&mapQ);
    }
    if (warp == 1) tmem_alloc(&ctl->tmem_base, 512);
    // the lengths may come from the kernel before this call (and, in sweep 2, the records from sweep 1): the set-up
    // above touched nothing that another kernel writes
    pdl_wait();
    const uint32_t limit = load_wait_limit(a.hdr);
    tc_fence_before();
    cta_prefix<kThreads>(n_slabs, [&](int s) { return (live(s) + 127) >> 7; }, pref, ctl->wsum);   // also publishes the set-up
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    const int Ttot = pref[n_slabs];
    const int per_cta = max(1, (Ttot + G - 1) / G);
    const int t_begin = min(cta * per_cta, Ttot), t_end = min(t_begin + per_cta, Ttot);
    const int ntl = t_end - t_begin;
    int slab0 = 0;
    if (ntl > 0) {
        int lo = 0, hi = n_slabs - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (pref[mid] <= t_begin) lo = mid; else hi = mid - 1;
        }
        slab0 = lo;
    }
    const float scale = kLog2e * rsqrtf(float(kHeadDim));
    const int n = a.Hq / Hk;

    if (kSweep == 1 && warp < 2 && lane != 0) {
        // the 62 otherwise idle lanes of the TMA and MMA warps clear the per-sentence key sums that sweep 2 accumulates
        const size_t total = size_t(n_slabs) * a.max_sent * (kHeadDim / 4);        // float4 words
        const size_t per = (total + G - 1) / G, w0 = min(size_t(cta) * per, total), w1 = min(w0 + per, total);
        float4* v4 = reinterpret_cast<float4*>(a.vsum);
        for (size_t i = w0 + size_t(warp * 31 + lane - 1); i < w1; i += 62) v4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0 && ntl > 0) {
            // what depends on the slab only is kept in registers: between "stage free" and the next copy's issue nothing
            // waits on shared or global memory
            int slab = slab0, stage = 0, issued = 0, slab_begin = 0, slab_end = 0;
            long long row0 = 0;
            uint32_t lap = 0, qlap = 0;
            bool ok = true;
            for (int t = t_begin; t < t_end && ok; ++t) {
                if (t == t_begin || slab_end <= t) {
                    while (pref[slab + 1] <= t) ++slab;
                    slab_begin = pref[slab]; slab_end = pref[slab + 1];
                    row0 = a.block_table ? 0 : (long long)slab_row0(a.slab_off, a.cap, Hk, slab / Hk, slab % Hk);
                    if (qlap > 0) ok = role_wait(&ctl->qempty, (qlap - 1) & 1u, limit, &ctl->abort_flag, a.status);
                    if (!ok) break;
                    const int b = slab / Hk, h = slab % Hk;
                    mbar_expect_tx(&ctl->qfull, uint32_t(RB) * 2u * 128u * uint32_t(a.WB * n));
                    for (int k = 0; k < RB; ++k) {
                        tma_load_3d(qbuf + size_t(k) * kOpBytes, &mapQ, 0, k * a.WB, b * a.Hq + h * n, &ctl->qfull);
                        tma_load_3d(qbuf + size_t(k) * kOpBytes + kOpHalfBytes, &mapQ, 64, k * a.WB, b * a.Hq + h * n,
                                    &ctl->qfull);
                    }
                    ++qlap;
                }
                const long long row =
                    a.block_table ? (long long)max(a.block_table[size_t(slab) * a.max_pages + (t - slab_begin)], 0) * 128
                                  : row0 + (long long)(t - slab_begin) * 128;
                if (lap > 0) ok = role_wait(&ctl->empty[stage], (lap - 1) & 1u, limit, &ctl->abort_flag, a.status);
                if (!ok) break;
                uint8_t* dst = tiles + size_t(stage) * kOpBytes;
                mbar_expect_tx(&ctl->full[stage], kOpBytes);
                tma_load_2d(dst, &mapK, 0, int(row), &ctl->full[stage]);
                tma_load_2d(dst + kOpHalfBytes, &mapK, 64, int(row), &ctl->full[stage]);
                ++issued;
                if (++stage == a.stages) { stage = 0; ++lap; }
            }
            if (!ok) {
                // copies already issued must land before the CTA retires
                for (int s = 0; s < a.stages; ++s) { mbar_wait(&ctl->full[s], 0u, 1u << 16); mbar_wait(&ctl->full[s], 1u, 1u << 16); }
                mbar_wait(&ctl->qfull, 0u, 1u << 16);
                mbar_wait(&ctl->qfull, 1u, 1u << 16);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0 && ntl > 0) {
            int slab = slab0, stage = 0, it = 0, slab_end = 0;
            uint32_t lap = 0, qlap = 0;
            bool ok = true;
            for (int t = t_begin; t < t_end && ok; ++t) {
                if (t == t_begin || slab_end <= t) {
                    while (pref[slab + 1] <= t) ++slab;
                    slab_end = pref[slab + 1];
                    ok = role_wait(&ctl->qfull, qlap & 1u, limit, &ctl->abort_flag, a.status);
                    if (!ok) break;
                    ++qlap;
                }
                ok = role_wait(&ctl->full[stage], lap & 1u, limit, &ctl->abort_flag, a.status);
                if (!ok) break;
                const uint32_t k_smem = smem_u32(tiles + size_t(stage) * kOpBytes);
                for (int k = 0; k < RB && ok; ++k, ++it) {
                    constexpr int kBufs = kSweep == 1 ? kAccBufs : kSw2Bufs;
                    const int buf = it % kBufs, use = it / kBufs;
                    if (use > 0) ok = role_wait(&ctl->tempty[buf], uint32_t(use - 1) & 1u, limit, &ctl->abort_flag, a.status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t q_smem = smem_u32(qbuf + size_t(k) * kOpBytes);
                    if (kSweep == 1) umma_tile_128x128x128(tmem_base + buf * 128, q_smem, k_smem, false);
                    else             umma_tile_128x128x128(tmem_base + buf * 128, k_smem, q_smem, false);
                    {
                        const int ti = t - t_begin, gj = (ti / kGroups) * RB + k;     // the owning group's item count
                        umma_commit(&ctl->tfull[ti % kGroups][gj & 3]);
                    }
                }
                if (t + 1 == t_end || slab_end <= t + 1) umma_commit(&ctl->qempty);
                umma_commit(&ctl->empty[stage]);
                if (++stage == a.stages) { stage = 0; ++lap; }
            }
            if (!ok) {
                // nobody will wait for the products still in flight: let them retire before the tensor memory is released
                umma_commit(&ctl->issued_done[0]);
                mbar_wait(&ctl->issued_done[0], 0u, 1u << 18);
            }
        }
    } else if (warp < 2 + 4 * kGroups) {
        // ------------------------------------------------------------------ epilogue warpgroups
        const int g = (warp - 2) >> 2;                       // warpgroup: tiles t_begin + g, + g + kGroups, ...
        const int quarter = warp & 3;                        // tensor-memory lanes this warp may read
        const int row = quarter * 32 + lane;
        const uint32_t lane_addr = tmem_base + (uint32_t(quarter * 32) << 16);
        bool ok = true;
        int slab = slab0, tl = g;
        if (kSweep == 1) {
            for (int seg_t = t_begin; seg_t < t_end;) {
                while (pref[slab + 1] <= seg_t) ++slab;
                const int seg_end = min(t_end, pref[slab + 1]);
                const int N = live(slab);
                float m[kMaxRB], l[kMaxRB];
#pragma unroll
                for (int k = 0; k < kMaxRB; ++k) { m[k] = -INFINITY; l[k] = 0.f; }
                for (; t_begin + tl < seg_end; tl += kGroups) {
                    const int t = t_begin + tl;
                    const int valid = min(128, N - (t - pref[slab]) * 128);
#pragma unroll
                    for (int k = 0; k < kMaxRB; ++k) {
                        if (k < RB && ok) {
                            const int it = tl * RB + k, buf = it & (kAccBufs - 1);
                            const int gj = (tl / kGroups) * RB + k;
                            ok = role_wait(&ctl->tfull[g][gj & 3], uint32_t(gj >> 2) & 1u, limit, &ctl->abort_flag, a.status);
                            ok = __all_sync(0xffffffffu, ok);
                            if (ok) {
                                tc_fence_after();
                                if (valid == 128) lse_fold<false>(lane_addr + buf * 128, valid, scale, m[k], l[k]);
                                else              lse_fold<true>(lane_addr + buf * 128, valid, scale, m[k], l[k]);
                                tc_fence_before();
                                __syncwarp();
                                if (lane == 0) mbar_arrive(&ctl->tempty[buf]);
                            }
                        }
                    }
                }
                float2* rec = a.sc_part + (size_t(cta + slab) * kSw1Groups + g) * (size_t(RB) * 128);
#pragma unroll
                for (int k = 0; k < kMaxRB; ++k)
                    if (k < RB) rec[k * 128 + row] = make_float2(m[k], l[k]);
                seg_t = seg_end;
            }
        } else {
            float* nl = ctl->neg_lse[g];
            const int wt = tid - 64 - g * 128;              // thread index inside the warpgroup
            int N = 0;
            size_t row0 = 0;
            bool have = false;
            for (; tl < ntl; tl += kGroups) {
                const int t = t_begin + tl;
                if (!have || pref[slab + 1] <= t) {
                    while (pref[slab + 1] <= t) ++slab;
                    have = true;
                    N = live(slab);
                    row0 = a.block_table ? size_t(slab) * a.max_pages * 128 : slab_row0(a.slab_off, a.cap, Hk, slab / Hk, slab % Hk);
                    // log-sum-exp of every query row of this slab from the sweep-1 records
                    const int fc = pref[slab] / per_cta, lc = (pref[slab + 1] - 1) / per_cta;
                    const float2* r0 = a.sc_part + size_t(fc + slab) * kSw1Groups * (size_t(RB) * 128);
                    const int n_part = (lc - fc + 1) * kSw1Groups;
                    named_bar_sync(2 + g, 128);              // previous readers of nl are done
                    for (int k = 0; k < RB; ++k) {
                        float M = -INFINITY;
                        for (int p = 0; p < n_part; ++p) M = fmaxf(M, r0[size_t(p) * RB * 128 + k * 128 + wt].x);
                        float L = 0.f;
                        for (int p = 0; p < n_part; ++p) {
                            const float2 pr = r0[size_t(p) * RB * 128 + k * 128 + wt];
                            if (pr.y > 0.f) L += pr.y * ex2f(pr.x - M);
                        }
                        nl[k * 128 + wt] = (L > 0.f) ? -(M + log2f(L)) : 0.f;
                    }
                    named_bar_sync(2 + g, 128);
                }
                float total = 0.f;
#pragma unroll
                for (int k = 0; k < kMaxRB; ++k) {
                    if (k < RB && ok) {
                        const int it = tl * RB + k, buf = it % kSw2Bufs;
                        const int gj = (tl / kGroups) * RB + k;
                        ok = role_wait(&ctl->tfull[g][gj & 3], uint32_t(gj >> 2) & 1u, limit, &ctl->abort_flag, a.status);
                        ok = __all_sync(0xffffffffu, ok);
                        if (ok) {
                            tc_fence_after();
                            total += imp_fold<kN>(lane_addr + buf * 128, nl + k * 128,
                                                  min(128 / kN, a.window - k * (128 / kN)), scale);
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(&ctl->tempty[buf]);
                        }
                    }
                }
                const int tok = (t - pref[slab]) * 128 + row;
                if (ok && tok < N) {
                    const float v = total / float(a.window);
                    a.tok_imp_ws[size_t(slab) * a.max_cap + tok] = v;
                    if (a.tok_imp_user) a.tok_imp_user[row0 + tok] = v;
                }
            }
        }
    } else if (kSweep == 2 && warp < 2 + 4 * kGroups + kPoolWarps) {
        // ------------------------------------------------------------------ per-sentence sums of the key rows
        // The sums are a product on the tensor cores: (tile^T: channel x token) x (indicator: token x sentence slot).
        // A run of consecutive tiles whose sentences all fall among the 16 sentences B .. B + 15 shares one accumulator
        // (slot j = sentence B + j; the products of the run accumulate), so the sums are read out and added to global
        // memory once per run, about every fifth tile.  Each of the four warps writes a quarter of a tile's matrix and
        // arrives; one thread of a fifth warp issues the product; when a tile opens a new run the four warps read out the
        // run before it (a thread owns one channel) while the new one is being multiplied.  A tile that touches more
        // than 16 sentences (empty ones count) gets several matrices, each a run of its own.
        // Every warp keeps, one entry per lane, the sentence offsets B .. B + 31 of the current run (entries past the
        // table read as "never starts"), fetched from global memory when a run opens: loads from shared memory wait
        // several hundred cycles here (the tensor core streams its operands from it), so the per-tile work touches
        // shared memory only to write the matrix.
        constexpr int kNever = 0x7fffffff;
        const int gw = warp - (2 + 4 * kGroups);                // warp of the group: slots 4 gw .. 4 gw + 3 of a matrix
        const int gtid = tid - (2 + 4 * kGroups) * 32;
        const int quarter = warp & 3;                           // tensor-memory lanes this warp may read
        const int ch = quarter * 32 + lane;
        const uint32_t lane_addr = tmem_base + (uint32_t(quarter * 32) << 16) + kPoolCol;
        int slab = slab0, S = 0, N = 0, first = 0;
        int ic = 0;                                             // indicator matrices written so far
        int run = -1, B = 0, w = kNever;                        // current run: index, sentence of slot 0, offsets B + lane
        uint32_t run_held = 0;                                  // its slots that hold tokens so far
        int run_slab = 0;
        const int32_t* so = a.sent_off;
        bool ok = true, have = false;
        // 32-way search for the last sentence that starts at or before token `tok`, one probe per lane
        auto holder = [&](int tok) {
            int lo = 0, len = S;
            while (len > 32) {
                const int stride = (len + 31) >> 5;
                const int pidx = lo + lane * stride;
                const bool le = pidx < lo + len && so[pidx] <= tok;
                const int adv = max(__popc(__ballot_sync(0xffffffffu, le)) - 1, 0) * stride;
                len = min(stride, len - adv);
                lo += adv;
            }
            const bool le = lane < len && so[lo + lane] <= tok;
            return lo + max(__popc(__ballot_sync(0xffffffffu, le)) - 1, 0);
        };
        // read out run r (accumulator r & 1) and add it to the sums
        auto drain = [&](int r, int r_slab, int r_B, uint32_t r_held) {
            ok = role_wait(&ctl->pfull[r & 1], uint32_t(r >> 1) & 1u, limit, &ctl->abort_flag, a.status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) return;
            tc_fence_after();
            float v[kIndSlots];
            tmem_ld16(lane_addr + uint32_t(r & 1) * kIndSlots, v);
            tc_fence_before();
            float* dst = a.vsum + (size_t(r_slab) * a.max_sent + r_B) * kHeadDim + ch;
#pragma unroll
            for (int j = 0; j < kIndSlots; ++j)
                if (r_held & (1u << j)) atomicAdd(dst + size_t(j) * kHeadDim, v[j]);
        };
        for (int tl = 0; tl < ntl && ok; ++tl) {
            const int t = t_begin + tl;
            const bool fresh = !have || pref[slab + 1] <= t;
            if (fresh) {
                while (pref[slab + 1] <= t) ++slab;
                have = true;
                so = a.sent_off + size_t(slab) * (a.max_sent + 1);
                S = min(max(a.n_sent[slab], 0), a.max_sent);
                N = live(slab);
            }
            const int tok0 = (t - pref[slab]) * 128, valid = min(128, N - tok0), tok_end = tok0 + valid;
            const int stage = tl % a.stages;
            if (fresh) first = tok0 > 0 ? holder(tok0) : 0;     // (a slab that opens with empty sentences: they get slots)
            // every warp follows every tile's arrival (in order, so it sees each phase of the stage's barrier)
            ok = role_wait(&ctl->full[stage], uint32_t(tl / a.stages) & 1u, limit, &ctl->abort_flag, a.status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (valid < 128) {
                // a zero in the indicator does not silence a NaN or an infinity in a dead row: clear the rows past the
                // slab's end in the staged tile (the logits of those rows are never read)
                uint8_t* tile = tiles + size_t(stage) * kOpBytes;
                for (int u = valid * 8 + gtid; u < 128 * 8; u += kPoolWarps * 32) {
                    *reinterpret_cast<uint4*>(tile + u * 16) = make_uint4(0u, 0u, 0u, 0u);
                    *reinterpret_cast<uint4*>(tile + kOpHalfBytes + u * 16) = make_uint4(0u, 0u, 0u, 0u);
                }
            }
            int cur = first;                                    // first sentence of the tile not yet in a matrix
            int more = 0;
            do {
                // can the tile (from sentence cur on) join the open run?  its last sentence must be below B + 16
                bool join = false;
                if (run >= 0 && !fresh && cur >= B && cur - B < kIndSlots) {
                    const int touching = __popc(__ballot_sync(0xffffffffu, lane > cur - B && B + lane < S && w < tok_end));
                    join = cur + touching - B < kIndSlots;
                }
                const int r_prev = run, p_slab = run_slab, p_B = B;
                const uint32_t p_held = run_held;
                if (!join) {                                    // open a run at sentence cur
                    ++run; B = cur; run_slab = slab; run_held = 0;
                    w = (B + lane <= S) ? so[B + lane] : kNever;
                }
                // tile-relative start of the sentences B + lane, clamped to the tile; slot j holds [cl(j), cl(j + 1))
                const int cl = min(max(min(w, tok_end) - tok0, 0), valid);
                const int cl_next = __shfl_down_sync(0xffffffffu, cl, 1);
                const uint32_t held = __ballot_sync(0xffffffffu, lane < kIndSlots && B + lane < S && cl_next > cl);
                const int s_next = __shfl_sync(0xffffffffu, w, kIndSlots);           // start of the sentence after slot 15
                more = (B + kIndSlots < S && s_next < tok_end) ? 1 : 0;
                const int is = ic & (kIndRing - 1);
                if (ic >= kIndRing) {                           // the product that read this buffer last has completed
                    ok = role_wait(&ctl->iempty[is], uint32_t(ic / kIndRing - 1) & 1u, limit, &ctl->abort_flag, a.status);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                }
                {
                    const int j = 4 * gw + (lane >> 3);         // this thread's slot row and its two pieces
                    const int lo = __shfl_sync(0xffffffffu, cl, j), hi = __shfl_sync(0xffffffffu, cl, j + 1);
                    const bool is_sent = (held >> j) & 1u;
                    indicator_piece(indb + size_t(is) * kIndBytes, j, (lane & 7) * 2, is_sent ? lo : 0, is_sent ? hi : 0);
                    indicator_piece(indb + size_t(is) * kIndBytes, j, (lane & 7) * 2 + 1, is_sent ? lo : 0, is_sent ? hi : 0);
                }
                fence_proxy_async_smem();                       // the matrix (and cleared rows) are read by the tensor core
                tc_fence_before();                              // and this warp's reads of the accumulators came first
                __syncwarp();
                if (lane == 0) {
                    if (gw == 0) ctl->ind_flags[is] = more | (join ? 2 : 0) | ((!join && r_prev >= 0) ? 4 : 0);
                    mbar_arrive(&ctl->ifull[is]);
                }
                run_held |= held;
                ++ic;
                if (!join && r_prev >= 0) {                     // the run before, while the new one is being multiplied
                    drain(r_prev, p_slab, p_B, p_held);
                    if (!ok) break;
                }
                cur = B + kIndSlots;
            } while (more);
            // the next tile starts in the last sentence of the run's window that starts at or before its first token
            const int n_le = __popc(__ballot_sync(0xffffffffu, B + lane < S && w <= tok0 + 128));
            first = (n_le == 32 && B + 32 < S) ? holder(tok0 + 128) : B + max(n_le - 1, 0);
        }
        if (ok && run >= 0) drain(run, run_slab, B, run_held);  // the issuer closes the last run when its tiles are done
    } else if (kSweep == 2) {
        // ------------------------------------------------------------------ issuer of the pooling products
        // (its own thread: an issue blocks for the length of the product, and every look at shared memory costs the
        // thread that issues the logits a few hundred cycles)
        if (lane == 0 && ntl > 0) {
            const uint32_t indb_u32 = smem_u32(indb);
            bool ok = true;
            int pc = 0, run = -1;
            for (int tl = 0; tl < ntl && ok; ++tl) {
                const int stage = tl % a.stages;
                int flags = 0;
                do {
                    const int is = pc & (kIndRing - 1);
                    ok = role_wait(&ctl->ifull[is], uint32_t(pc / kIndRing) & 1u, limit, &ctl->abort_flag, a.status);
                    if (!ok) break;
                    flags = *reinterpret_cast<volatile int*>(&ctl->ind_flags[is]);       // 1: more, 2: joins the run, 4: closes one
                    tc_fence_after();
                    if (flags & 4) umma_commit(&ctl->pfull[run & 1]);                    // everything of the run before is issued
                    if (!(flags & 2)) ++run;
                    umma_pool(tmem_base + kPoolCol + uint32_t(run & 1) * kIndSlots, smem_u32(tiles + size_t(stage) * kOpBytes),
                              indb_u32 + uint32_t(is) * kIndBytes, (flags & 2) != 0);
                    umma_commit(&ctl->iempty[is]);
                    ++pc;
                } while (flags & 1);
                if (ok) umma_commit(&ctl->empty[stage]);
            }
            if (ok && run >= 0) umma_commit(&ctl->pfull[run & 1]);
            if (!ok) {
                umma_commit(&ctl->issued_done[1]);
                mbar_wait(&ctl->issued_done[1], 0u, 1u << 18);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// ---------------------------------------------------------------------------------------
// pooling: one warp per sentence, 4 channels per lane; writes the normalised mean key as bf16 hi + lo
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
score_pool_kernel(int Hk, int max_sent, int max_cap, const int32_t* cap, const int32_t* kv_len,
                  const int32_t* sent_off, const int32_t* n_sent, float eps, const float* tok_imp_ws,
                  const float* vsum, float* sent_imp, __nv_bfloat16* vbar_hi, __nv_bfloat16* vbar_lo) {
    pdl_trigger();
    pdl_wait();
    const int slab = blockIdx.y;
    const int lane = threadIdx.x & 31;
    const int i = blockIdx.x * 8 + (threadIdx.x >> 5);
    const int S = min(n_sent[slab], max_sent);
    if (i >= S) return;
    const int N = min(max(kv_len[slab], 0), cap[slab / Hk]);
    const int32_t* so = sent_off + size_t(slab) * (max_sent + 1);
    const int b = max(so[i], 0), e = min(so[i + 1], N);
    float ti = 0.f;
    for (int t = b + lane; t < e; t += 32) ti += tok_imp_ws[size_t(slab) * max_cap + t];
    const float len = float(max(e - b, 1));
    const size_t o = (size_t(slab) * max_sent + i) * kHeadDim;
    float4 v = reinterpret_cast<const float4*>(vsum + o)[lane];
    if (e <= b) v = make_float4(0.f, 0.f, 0.f, 0.f);
    v.x /= len; v.y /= len; v.z /= len; v.w /= len;
    float nn = v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
#pragma unroll
    for (int d = 16; d; d >>= 1) {
        nn += __shfl_xor_sync(0xffffffffu, nn, d);
        ti += __shfl_xor_sync(0xffffffffu, ti, d);
    }
    const float inv = 1.f / (sqrtf(nn) + eps);
    const float x[4] = {v.x * inv, v.y * inv, v.z * inv, v.w * inv};
    uint32_t hi[4], lo[4];                                   // bf16 bit patterns
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const __nv_bfloat16 h = __float2bfloat16_rn(x[c]);
        const __nv_bfloat16 r = __float2bfloat16_rn(x[c] - __bfloat162float(h));
        hi[c] = __bfloat16_as_ushort(h);
        lo[c] = __bfloat16_as_ushort(r);
    }
    reinterpret_cast<uint2*>(vbar_hi + o)[lane] = make_uint2(hi[0] | (hi[1] << 16), hi[2] | (hi[3] << 16));
    reinterpret_cast<uint2*>(vbar_lo + o)[lane] = make_uint2(lo[0] | (lo[1] << 16), lo[2] | (lo[3] << 16));
    if (lane == 0) sent_imp[size_t(slab) * max_sent + i] = (e > b) ? ti / len : 0.f;
}

// ---------------------------------------------------------------------------------------
// Gram passes on the tensor cores.  Work item = 128 sentences i of one slab against all j in blocks of 128;
// persistent CTAs take the items round-robin, so barriers, tensor memory and descriptors are set up once and
// the j-block ring keeps streaming from one item into the next.
// ---------------------------------------------------------------------------------------
constexpr int kGramGroups = 4;          // epilogue warpgroups = tensor-memory accumulators: one group's tensor-memory
                                       // reads hide behind the arithmetic of the others
struct GramCtl {
    uint64_t afull, aempty, bfull[2], bempty[2], tfull[kGramGroups], tempty[kGramGroups];
    uint32_t tmem_base;
    int abort_flag;
    uint32_t wsum[32];
    alignas(16) float invz[kGramGroups][2][128];   // by the parity of the group's block count: a warp that runs ahead
                                                   // fills the other half while its siblings still read this one
    float part[2][kGramGroups - 1][2][128];   // by item parity: the other groups' (sum, max) shares of a row
};
constexpr int kGramThreads = (2 + 4 * kGramGroups) * 32;
static size_t gram_smem_bytes(int slabs) { return 1024 + 6 * size_t(kOpBytes) + sizeof(GramCtl) + size_t(slabs + 1) * 4; }

// Optional source of the sentence penalty: the lookup table T of one value per generation-space sentence,
// [batch][table_len], read through the cache-space sentence's generation-space index (Phi).  table == nullptr:
// the penalty comes from the pooled keys of the slab.
struct LamTable {
    const float* table;
    const int32_t* sent_id;
    int table_len;
    int Hk;
};

template <int kPass>
__global__ void __launch_bounds__(kGramThreads, 1)
score_gram_kernel(const __grid_constant__ CUtensorMap mapHi, const __grid_constant__ CUtensorMap mapLo, int n_slabs,
                  int max_sent, const int32_t* n_sent, float sigma, float tau, float* sc_z, const float* sent_imp,
                  float* sent_red, float* sent_lam, float* sent_score, LamTable ext, const Header* hdr) {
    extern __shared__ uint8_t gram_smem_raw[];
    const uint32_t raw = smem_u32(gram_smem_raw);
    uint8_t* At = gram_smem_raw + (((raw + 1023u) & ~1023u) - raw);              // hi, lo of the i block
    uint8_t* Bt = At + 2 * kOpBytes;                                             // 2 stages x (hi, lo) of a j block
    GramCtl* ctl = reinterpret_cast<GramCtl*>(Bt + 4 * kOpBytes);
    int* ipref = reinterpret_cast<int*>(ctl + 1);                                // [n_slabs + 1] prefix of i blocks
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int G = gridDim.x, cta = blockIdx.x;
    auto sent_of = [&](int s) { return min(max(n_sent[s], 0), max_sent); };
    pdl_trigger();

    if (tid == 0) {
        mbar_init(&ctl->afull, 1);
        mbar_init(&ctl->aempty, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&ctl->bfull[s], 1);
            mbar_init(&ctl->bempty[s], 1);
        }
        for (int s = 0; s < kGramGroups; ++s) {
            mbar_init(&ctl->tfull[s], 1);
            mbar_init(&ctl->tempty[s], 4);
        }
        ctl->abort_flag = 0;
        mbar_fence_init();
        tmap_prefetch(&mapHi);
        tmap_prefetch(&mapLo);
    }
    if (warp == 1) tmem_alloc(&ctl->tmem_base, 128 * kGramGroups);
    pdl_wait();                                          // n_sent, the pooled keys and the row sums may come from the kernel before
    uint32_t* status = const_cast<uint32_t*>(&hdr->status);
    const uint32_t limit = load_wait_limit(hdr);
    tc_fence_before();
    cta_prefix<kGramThreads>(n_slabs, [&](int s) { return (sent_of(s) + 127) >> 7; }, ipref, ctl->wsum);   // i blocks per slab
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    const int n_items = ipref[n_slabs];

    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            int slab = 0;
            uint32_t bc = 0, ic = 0;                                // j blocks and items issued so far
            for (int item = cta; item < n_items && ok; item += G, ++ic) {
                while (ipref[slab + 1] <= item) ++slab;
                const int S = sent_of(slab), NJ = (S + 127) >> 7, rowbase = slab * max_sent;
                const int i0 = (item - ipref[slab]) * 128;
                if (ic > 0) ok = role_wait(&ctl->aempty, (ic - 1) & 1u, limit, &ctl->abort_flag, status);
                if (!ok) break;
                mbar_expect_tx(&ctl->afull, 2 * kOpBytes);
                tma_load_2d(At, &mapHi, 0, rowbase + i0, &ctl->afull);
                tma_load_2d(At + kOpHalfBytes, &mapHi, 64, rowbase + i0, &ctl->afull);
                tma_load_2d(At + kOpBytes, &mapLo, 0, rowbase + i0, &ctl->afull);
                tma_load_2d(At + kOpBytes + kOpHalfBytes, &mapLo, 64, rowbase + i0, &ctl->afull);
                for (int jb = 0; jb < NJ && ok; ++jb, ++bc) {
                    const int s = bc & 1;
                    if (bc >= 2) ok = role_wait(&ctl->bempty[s], ((bc >> 1) - 1) & 1u, limit, &ctl->abort_flag, status);
                    if (!ok) break;
                    uint8_t* dst = Bt + size_t(s) * 2 * kOpBytes;
                    mbar_expect_tx(&ctl->bfull[s], 2 * kOpBytes);
                    tma_load_2d(dst, &mapHi, 0, rowbase + jb * 128, &ctl->bfull[s]);
                    tma_load_2d(dst + kOpHalfBytes, &mapHi, 64, rowbase + jb * 128, &ctl->bfull[s]);
                    tma_load_2d(dst + kOpBytes, &mapLo, 0, rowbase + jb * 128, &ctl->bfull[s]);
                    tma_load_2d(dst + kOpBytes + kOpHalfBytes, &mapLo, 64, rowbase + jb * 128, &ctl->bfull[s]);
                }
            }
            if (!ok) {
                mbar_wait(&ctl->afull, 0u, 1u << 16); mbar_wait(&ctl->afull, 1u, 1u << 16);
                for (int s = 0; s < 2; ++s) { mbar_wait(&ctl->bfull[s], 0u, 1u << 16); mbar_wait(&ctl->bfull[s], 1u, 1u << 16); }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            bool ok = true;
            int slab = 0;
            uint32_t bc = 0, ic = 0;
            const uint32_t a_hi = smem_u32(At), a_lo = smem_u32(At + kOpBytes);
            for (int item = cta; item < n_items && ok; item += G, ++ic) {
                while (ipref[slab + 1] <= item) ++slab;
                const int NJ = (sent_of(slab) + 127) >> 7;
                ok = role_wait(&ctl->afull, ic & 1u, limit, &ctl->abort_flag, status);
                for (int jb = 0; jb < NJ && ok; ++jb, ++bc) {
                    const int s = bc & 1, acc = bc % kGramGroups;
                    ok = role_wait(&ctl->bfull[s], (bc >> 1) & 1u, limit, &ctl->abort_flag, status);
                    if (ok && bc >= kGramGroups) ok = role_wait(&ctl->tempty[acc], ((bc / kGramGroups) - 1) & 1u, limit, &ctl->abort_flag, status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t b_hi = smem_u32(Bt + size_t(s) * 2 * kOpBytes), b_lo = b_hi + kOpBytes;
                    const uint32_t d = tmem_base + acc * 128;
                    umma_tile_128x128x128(d, a_hi, b_hi, false);
                    umma_tile_128x128x128(d, a_hi, b_lo, true);
                    umma_tile_128x128x128(d, a_lo, b_hi, true);
                    umma_commit(&ctl->tfull[acc]);
                    umma_commit(&ctl->bempty[s]);
                }
                if (ok) umma_commit(&ctl->aempty);                   // every MMA that reads this i block has completed
            }
        }
    } else {
        const int grp = (warp - 2) >> 2;                           // the accumulator this warpgroup drains
        const int quarter = warp & 3, wt = (tid - 64) & 127;
        const uint32_t lane_addr = tmem_base + (uint32_t(quarter * 32) << 16) + grp * 128;
        bool ok = true;
        int slab = 0;
        uint32_t bc = 0, ic = 0;
        for (int item = cta; item < n_items; item += G, ++ic) {
            while (ipref[slab + 1] <= item) ++slab;
            const int S = sent_of(slab), NJ = (S + 127) >> 7, rowbase = slab * max_sent;
            const int i0 = (item - ipref[slab]) * 128;
            const int row = quarter * 32 + lane;
            const int i = i0 + row;
            float accum = 0.f, mx = -INFINITY;
            for (int jb = 0; jb < NJ; ++jb, ++bc) {
                if (int(bc % kGramGroups) != grp) continue;        // another warpgroup's block
                const int j0 = jb * 128;
                float* invz_s = ctl->invz[grp][(bc / kGramGroups) & 1u];
                if (kPass == 2) {
                    const int j = j0 + wt;
                    const float z = (j < S) ? sc_z[size_t(rowbase) + j] : 1.f;
                    invz_s[wt] = (z > 0.f) ? 1.f / z : 0.f;
                    named_bar_sync(1 + grp, 128);
                }
                if (ok) {
                    ok = role_wait(&ctl->tfull[grp], (bc / kGramGroups) & 1u, limit, &ctl->abort_flag, status);
                    ok = __all_sync(0xffffffffu, ok);
                }
                if (!ok) continue;                               // keeps the barrier pattern uniform
                tc_fence_after();
                const bool interior = (j0 + 128 <= S) && (j0 != i0);
#pragma unroll 1
                for (int ch = 0; ch < 4; ++ch) {
                    float v[32];
                    tmem_ld32(lane_addr + ch * 32, v);
                    const float* iz = invz_s + ch * 32;
                    if (interior) {
                        float e0 = 0.f, e1 = 0.f;
#pragma unroll
                        for (int jj = 0; jj < 32; jj += 2) {
                            if (kPass == 1) {
                                e0 += ex2f(v[jj] * kLog2e);
                                e1 += ex2f(v[jj + 1] * kLog2e);
                            } else {
                                e0 = fmaf(ex2f(v[jj] * kLog2e), iz[jj], e0);
                                e1 = fmaf(ex2f(v[jj + 1] * kLog2e), iz[jj + 1], e1);
                            }
                        }
                        accum += e0 + e1;
                        if (kPass == 1 && j0 > i0) {
#pragma unroll
                            for (int jj = 0; jj < 32; ++jj) mx = fmaxf(mx, v[jj]);
                        }
                    } else {
#pragma unroll
                        for (int jj = 0; jj < 32; ++jj) {
                            const int j = j0 + ch * 32 + jj;
                            if (j < S && j != i) {
                                const float e = ex2f(v[jj] * kLog2e);
                                if (kPass == 1) {
                                    accum += e;
                                    if (j > i) mx = fmaxf(mx, v[jj]);
                                } else {
                                    accum = fmaf(e, iz[jj], accum);
                                }
                            }
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctl->tempty[grp]);
            }
            // the warpgroups hold the sums (and maxima) over interleaved j blocks: the others hand theirs to the first
            if (grp > 0) {
                ctl->part[ic & 1][grp - 1][0][row] = accum;
                if (kPass == 1) ctl->part[ic & 1][grp - 1][1][row] = mx;
            }
            named_bar_sync(1 + kGramGroups, 128 * kGramGroups);
            if (grp == 0 && ok && i < S) {
#pragma unroll
                for (int g = 0; g < kGramGroups - 1; ++g) {
                    accum += ctl->part[ic & 1][g][0][row];
                    if (kPass == 1) mx = fmaxf(mx, ctl->part[ic & 1][g][1][row]);
                }
                const size_t o = size_t(rowbase) + i;
                if (kPass == 1) {
                    sc_z[o] = accum;
                    if (ext.table) {                             // penalty from the generation-space table through Phi
                        const int g = ext.sent_id[o];
                        sent_lam[o] = (g >= 0 && g < ext.table_len) ? ext.table[size_t(slab / ext.Hk) * ext.table_len + g] : 0.f;
                    } else {
                        sent_lam[o] = (mx > tau) ? mx : 0.f;
                    }
                } else {
                    const float red = accum / float(S);
                    sent_red[o] = red;
                    sent_score[o] = sigma * sent_imp[o] - (1.f - sigma) * red - sent_lam[o];
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 128 * kGramGroups);
    }
}

template <int kSweep, int kN>
static int launch_sweep(const CUtensorMap& mapK, const CUtensorMap& mapQ, const SweepArgs& a, int grid, size_t smem,
                        cudaStream_t st) {
    auto kern = score_sweep_kernel<kSweep, kN>;
    SKIPKV_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
    SKIPKV_CUDA(launch_dependent(kern, dim3(grid), dim3(kSweep == 1 ? kSw1Threads : kSw2Threads), smem, st, mapK, mapQ, a));
    return SKIPKV_OK;
}

}  // namespace skipkv

using namespace skipkv;

static int score_impl(const skipkv_shape* shape, const skipkv_params* params, const void* K, const void* q_win,
                      const int32_t* kv_len, const int32_t* sent_off, const int32_t* n_sent, float* tok_imp,
                      float* sent_imp, float* sent_red, float* sent_lam, float* sent_score, LamTable ext, void* ws,
                      void* stream, const int32_t* block_table = nullptr, int max_pages = 0) {
    if (int rc = check_shape(shape)) return rc;
    if (!params || !K || !q_win || !kv_len || !sent_off || !n_sent || !sent_imp || !sent_red || !sent_lam || !sent_score)
        return SKIPKV_ERR_INVALID_ARG;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255)) return SKIPKV_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(K) & 15) || (reinterpret_cast<uintptr_t>(q_win) & 15)) return SKIPKV_ERR_INVALID_ARG;
    if (shape->max_sent <= 0) return SKIPKV_OK;
    const WsLayout L = make_layout(*shape);
    uint8_t* w = static_cast<uint8_t*>(ws);
    uint32_t* status = &reinterpret_cast<Header*>(w + L.header)->status;
    float* sc_tok = reinterpret_cast<float*>(w + L.sc_tokimp);
    float* vsum = reinterpret_cast<float*>(w + L.sc_vsum);
    __nv_bfloat16* vbar_hi = reinterpret_cast<__nv_bfloat16*>(w + L.sc_vbar_hi);
    __nv_bfloat16* vbar_lo = reinterpret_cast<__nv_bfloat16*>(w + L.sc_vbar_lo);
    float* sc_z = reinterpret_cast<float*>(w + L.sc_z);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int Hq = shape->n_q_heads, Hk = shape->n_kv_heads, n = L.group;

    CUtensorMap mapK, mapQ, mapHi, mapLo;
    if (int rc = tmap_rows(&mapK, K, uint64_t(shape->total_rows), 128)) return rc;
    if (int rc = tmap_qwin(&mapQ, q_win, uint64_t(shape->batch) * Hq, uint32_t(shape->window), uint32_t(L.sc_wb), uint32_t(n)))
        return rc;
    const uint64_t vrows = uint64_t(L.slabs) * uint64_t(shape->max_sent);
    if (int rc = tmap_rows(&mapHi, vbar_hi, vrows, 128)) return rc;
    if (int rc = tmap_rows(&mapLo, vbar_lo, vrows, 128)) return rc;

    SweepArgs a{};
    a.Hq = Hq; a.Hk = Hk; a.window = shape->window; a.n_slabs = L.slabs; a.max_cap = shape->max_cap;
    a.max_sent = shape->max_sent; a.RB = L.sc_rb; a.WB = L.sc_wb;
    a.slab_off = shape->slab_off; a.cap = shape->cap; a.kv_len = kv_len; a.sent_off = sent_off; a.n_sent = n_sent;
    a.sc_part = reinterpret_cast<float2*>(w + L.sc_part);
    a.tok_imp_user = tok_imp; a.tok_imp_ws = sc_tok; a.vsum = vsum; a.status = status;
    a.hdr = reinterpret_cast<const Header*>(w + L.header);
    a.block_table = block_table; a.max_pages = max_pages;
    const size_t max_smem = 227 * 1024;
    const size_t fixed1 = 1024 + size_t(a.RB) * kOpBytes + sizeof(SweepCtl) + size_t(L.slabs + 1) * 4;
    if (fixed1 + kOpBytes > max_smem) return SKIPKV_ERR_UNSUPPORTED;
    SweepArgs a1 = a, a2 = a;
    a1.stages = int((max_smem - fixed1) / kOpBytes);
    if (a1.stages > kSwMaxStages) a1.stages = kSwMaxStages;
    // sweep 2 also holds the indicator matrices of its pooling product
    const size_t fixed2 = fixed1 + size_t(kIndRing) * kIndBytes;
    if (fixed2 + kOpBytes > max_smem) return SKIPKV_ERR_UNSUPPORTED;
    a2.stages = int((max_smem - fixed2) / kOpBytes);
    if (a2.stages > kSwMaxStages) a2.stages = kSwMaxStages;
    const size_t smem1 = fixed1 + size_t(a1.stages) * kOpBytes, smem2 = fixed2 + size_t(a2.stages) * kOpBytes;
    int grid = num_sms();
    if (grid > L.dec_max_ctas) grid = L.dec_max_ctas;

    if (int rc = launch_sweep<1, 1>(mapK, mapQ, a1, grid, smem1, st)) return rc;
    int rc = SKIPKV_ERR_UNSUPPORTED;
    switch (n) {
        case 1: rc = launch_sweep<2, 1>(mapK, mapQ, a2, grid, smem2, st); break;
        case 2: rc = launch_sweep<2, 2>(mapK, mapQ, a2, grid, smem2, st); break;
        case 3: rc = launch_sweep<2, 3>(mapK, mapQ, a2, grid, smem2, st); break;
        case 4: rc = launch_sweep<2, 4>(mapK, mapQ, a2, grid, smem2, st); break;
        case 5: rc = launch_sweep<2, 5>(mapK, mapQ, a2, grid, smem2, st); break;
        case 6: rc = launch_sweep<2, 6>(mapK, mapQ, a2, grid, smem2, st); break;
        case 7: rc = launch_sweep<2, 7>(mapK, mapQ, a2, grid, smem2, st); break;
        case 8: rc = launch_sweep<2, 8>(mapK, mapQ, a2, grid, smem2, st); break;
        default: break;
    }
    if (rc) return rc;
    {
        dim3 pgrid((shape->max_sent + 7) / 8, L.slabs);
        SKIPKV_CUDA(launch_dependent(score_pool_kernel, pgrid, dim3(256), 0, st, Hk, shape->max_sent, shape->max_cap,
                                     shape->cap, kv_len, sent_off, n_sent, params->eps, sc_tok, vsum, sent_imp, vbar_hi,
                                     vbar_lo));
    }
    {
        const size_t gsmem = gram_smem_bytes(L.slabs);
        if (gsmem > 227 * 1024) return SKIPKV_ERR_UNSUPPORTED;
        const long long max_items = (long long)L.slabs * ((shape->max_sent + 127) / 128);
        const int ggrid = int(max_items < (long long)grid ? max_items : (long long)grid);
        SKIPKV_CUDA(cudaFuncSetAttribute(score_gram_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(gsmem)));
        SKIPKV_CUDA(cudaFuncSetAttribute(score_gram_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(gsmem)));
        SKIPKV_CUDA(launch_dependent(score_gram_kernel<1>, dim3(ggrid), dim3(kGramThreads), gsmem, st, mapHi, mapLo, L.slabs,
                                     shape->max_sent, n_sent, params->sigma, params->tau, sc_z, sent_imp, sent_red, sent_lam,
                                     sent_score, ext, reinterpret_cast<const Header*>(w + L.header)));
        SKIPKV_CUDA(launch_dependent(score_gram_kernel<2>, dim3(ggrid), dim3(kGramThreads), gsmem, st, mapHi, mapLo, L.slabs,
                                     shape->max_sent, n_sent, params->sigma, params->tau, sc_z, sent_imp, sent_red, sent_lam,
                                     sent_score, ext, reinterpret_cast<const Header*>(w + L.header)));
    }
    return SKIPKV_OK;
}

extern "C" int skipkv_score(const skipkv_shape* shape, const skipkv_params* params, const void* K, const void* q_win,
                            const int32_t* kv_len, const int32_t* sent_off, const int32_t* n_sent, float* tok_imp,
                            float* sent_imp, float* sent_red, float* sent_lam, float* sent_score, void* ws,
                            void* stream) {
    return score_impl(shape, params, K, q_win, kv_len, sent_off, n_sent, tok_imp, sent_imp, sent_red, sent_lam,
                      sent_score, LamTable{nullptr, nullptr, 0, 1}, ws, stream);
}

extern "C" int skipkv_score_table(const skipkv_shape* shape, const skipkv_params* params, const void* K,
                                  const void* q_win, const int32_t* kv_len, const int32_t* sent_off,
                                  const int32_t* sent_id, const int32_t* n_sent, const float* lam_table,
                                  int32_t table_len, float* tok_imp, float* sent_imp, float* sent_red, float* sent_lam,
                                  float* sent_score, void* ws, void* stream) {
    if (!sent_id || !lam_table || table_len <= 0) return SKIPKV_ERR_INVALID_ARG;
    if (int rc = check_shape(shape)) return rc;
    return score_impl(shape, params, K, q_win, kv_len, sent_off, n_sent, tok_imp, sent_imp, sent_red, sent_lam,
                      sent_score, LamTable{lam_table, sent_id, table_len, shape->n_kv_heads}, ws, stream);
}

extern "C" int skipkv_score_paged(const skipkv_shape* shape, const skipkv_params* params, const void* K_pages,
                                  const int32_t* block_table, int32_t max_pages, const void* q_win, const int32_t* kv_len,
                                  const int32_t* sent_off, const int32_t* n_sent, float* tok_imp, float* sent_imp,
                                  float* sent_red, float* sent_lam, float* sent_score, void* ws, void* stream) {
    if (!block_table || max_pages <= 0) return SKIPKV_ERR_INVALID_ARG;
    if (int rc = check_shape(shape)) return rc;
    if (int64_t(max_pages) * 128 > int64_t(shape->max_cap) + 127) return SKIPKV_ERR_INVALID_ARG;   // the workspace is sized by max_cap
    return score_impl(shape, params, K_pages, q_win, kv_len, sent_off, n_sent, tok_imp, sent_imp, sent_red, sent_lam,
                      sent_score, LamTable{nullptr, nullptr, 0, 1}, ws, stream, block_table, max_pages);
}
