// skipkv_select: which sentences survive under the KV budget (paper Section 4.1: evict in
// increasing order of the final score until the cache meets budget B), at sentence granularity.
//
// One CTA per (sequence, head) slab.  Each sentence becomes a 64-bit key
//     [ 1 bit: not protected | 32 bits: ~orderable(score) | 31 bits: sentence index ]
// so an ascending sort yields: protected-tail sentences in index order, then the rest by score
// descending with ties broken by the lower index (exact fp32 comparison, -0 == +0).  The keys
// are sorted with a block-wide bitonic network in shared memory, the sentence lengths are
// prefix-summed in rank order, and a sentence survives iff its inclusive running total is
// within the budget.  Because lengths are non-negative the running total is monotone, so this
// is exactly "the longest rank prefix that fits; stop at the first sentence that does not".
// skipkv_select_fill then lets that first sentence keep its most important tokens, so that exactly B survive.
#include "common.cuh"

namespace skipkv {

constexpr int kSelThreads = 512;

__device__ __forceinline__ uint32_t orderable(float f) {
    uint32_t u = __float_as_uint(f);
    if ((u << 1) == 0u) u = 0u;                        // -0 -> +0
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u); // ascending in f
}

// exclusive scan over P = blockDim.x * per values held per thread as a running block; generic helper:
// each thread passes its local total, gets the exclusive offset of its first element.
__device__ __forceinline__ uint32_t block_excl(uint32_t v, uint32_t* wsum, uint32_t& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t a = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= d) inc += a;
    }
    if (lane == 31) wsum[warp] = inc;
    __syncthreads();
    uint32_t base = 0, t = 0;
    for (int w = 0; w < nw; ++w) {
        if (w == warp) base = t;
        t += wsum[w];
    }
    total = t;
    __syncthreads();
    return base + inc - v;
}

// Exactly-B retention: where tok_keep is non-null the first sentence that does not fit keeps its `slack` tokens of
// largest importance (equal values: the earlier token), flagged in tok_keep (one byte per cache row), and gets
// keep = 2.  tok_imp is indexed by cache row when from_rows is set, else [slab][max_cap].
struct FillArgs {
    const float* tok_imp;
    const float* tok_red;      // nullable, one value per cache row: the cut sentence's tokens are then ordered by
    float sigma;               // sigma * tok_imp - (1 - sigma) * tok_red (each operation rounded to fp32)
    uint8_t* tok_keep;
    const int64_t* slab_off;
    const int32_t* cap;
    int Hk, max_cap, from_rows;
};

__global__ void __launch_bounds__(kSelThreads)
select_kernel(int max_sent, int P, int budget, int protect_tail, const float* sent_score, const int32_t* sent_off,
              const int32_t* n_sent, uint8_t* keep, int32_t* kept_idx, int32_t* n_kept, int32_t* new_len,
              FillArgs fill, uint32_t* status) {
    extern __shared__ __align__(16) uint8_t sel_smem[];
    uint64_t* keys = reinterpret_cast<uint64_t*>(sel_smem);             // [P]
    uint8_t* flags = reinterpret_cast<uint8_t*>(keys + P);             // [P] keep flag by sentence index
    __shared__ uint32_t wsum[kSelThreads / 32];
    __shared__ int s_cut, s_slack;
    pdl_trigger();
    pdl_wait();                                          // inputs may come from the kernel before
    const int slab = blockIdx.x, tid = threadIdx.x;
    const float* score = sent_score + size_t(slab) * max_sent;
    const int32_t* so = sent_off + size_t(slab) * (max_sent + 1);
    uint8_t* kp = keep + size_t(slab) * max_sent;
    int32_t* ki = kept_idx ? kept_idx + size_t(slab) * max_sent : nullptr;
    int S = n_sent[slab];
    if (S < 0 || S > max_sent || S > P) {
        if (tid == 0) atomicOr(status, SKIPKV_STATUS_BAD_TABLE);
        S = 0;
    }
    const int total = (S > 0) ? so[S] : 0;

    if (total <= budget) {                              // already fits: identity
        for (int i = tid; i < max_sent; i += kSelThreads) {
            kp[i] = (i < S) ? 1 : 0;
            if (ki) ki[i] = (i < S) ? i : -1;
        }
        if (tid == 0) {
            if (n_kept) n_kept[slab] = S;
            if (new_len) new_len[slab] = total;
        }
        return;
    }

    for (int i = tid; i < P; i += kSelThreads) {
        uint64_t k = ~0ull;
        if (i < S) {
            const int b = so[i], e = so[i + 1];
            const bool forced = protect_tail > 0 && e > total - protect_tail && e > b;
            const uint64_t hi = forced ? 0ull : (0x100000000ull | uint64_t(~orderable(score[i])));
            k = (hi << 31) | uint64_t(uint32_t(i));
        }
        keys[i] = k;
        flags[i] = 0;
    }
    if (tid == 0) { s_cut = -1; s_slack = 0; }
    __syncthreads();
    // bitonic sort, ascending.  Thread p of a pass owns the compare-exchange pair (i, i | j) with
    // i = ((p & ~(j-1)) << 1) | (p & (j-1)).  For j <= 32 the 32 pairs of a warp stay inside the warp's own
    // 64-key block, so those steps only need a warp barrier; a block barrier separates them from the wider steps.
    for (int k = 2; k <= P; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int p = tid; p < (P >> 1); p += kSelThreads) {
                const int i = ((p & ~(j - 1)) << 1) | (p & (j - 1)), l = i | j;
                const uint64_t a = keys[i], c = keys[l];
                const bool up = (i & k) == 0;
                if ((a > c) == up) { keys[i] = c; keys[l] = a; }
            }
            if (j > 32 || j == 1) __syncthreads(); else __syncwarp();
        }
    }
    // running total of lengths in rank order; each thread owns a contiguous block of ranks
    const int per = (P + kSelThreads - 1) / kSelThreads;
    const int r0 = tid * per, r1 = min(r0 + per, S);
    uint32_t local = 0;
    for (int r = r0; r < r1; ++r) {
        const int i = int(keys[r] & 0x7fffffffu);
        local += uint32_t(so[i + 1] - so[i]);
    }
    uint32_t tot;
    uint32_t run = block_excl(local, wsum, tot);
    uint32_t kept_tokens = 0;
    for (int r = r0; r < r1; ++r) {
        const int i = int(keys[r] & 0x7fffffffu);
        const uint32_t before = run;
        run += uint32_t(so[i + 1] - so[i]);
        if (run <= uint32_t(budget)) { flags[i] = 1; kept_tokens = run; }
        else if (fill.tok_keep && before < uint32_t(budget)) { s_cut = i; s_slack = budget - int(before); }  // one rank only
    }
    __syncthreads();
    if (fill.tok_keep && s_cut >= 0) {
        const int c = s_cut, slack = s_slack;
        const int cb = so[c], len = so[c + 1] - cb;
        const int b = slab / fill.Hk, h = slab % fill.Hk;
        const size_t row0 = slab_row0(fill.slab_off, fill.cap, fill.Hk, b, h);
        const float* imp = fill.from_rows ? fill.tok_imp + row0 + cb : fill.tok_imp + size_t(slab) * fill.max_cap + cb;
        uint8_t* tk = fill.tok_keep + row0 + cb;
        const float* red = fill.tok_red ? fill.tok_red + row0 + cb : nullptr;
        const float w_red = __fsub_rn(1.f, fill.sigma);
        auto key = [&](int u) {
            const float i = __ldg(imp + u);
            return red ? __fsub_rn(__fmul_rn(fill.sigma, i), __fmul_rn(w_red, __ldg(red + u))) : i;
        };
        for (int t = tid; t < len; t += kSelThreads) {   // rank by counting: tokens that come before t in the order
            const float mine = key(t);
            int rank = 0;
            for (int u = 0; u < len; ++u) {
                const float other = key(u);
                rank += (other > mine || (other == mine && u < t)) ? 1 : 0;
            }
            tk[t] = rank < slack ? 1 : 0;
        }
        if (tid == 0) flags[c] = 2;
        __syncthreads();
    }
    const bool filled = fill.tok_keep && s_cut >= 0;
    // outputs in sentence-index order
    const int per_i = (max(S, 1) + kSelThreads - 1) / kSelThreads;
    const int i0 = tid * per_i, i1 = min(i0 + per_i, S);
    uint32_t cnt = 0;
    for (int i = i0; i < i1; ++i) cnt += flags[i] ? 1u : 0u;
    uint32_t nk;
    uint32_t pos = block_excl(cnt, wsum, nk);
    for (int i = i0; i < i1; ++i) {
        kp[i] = flags[i];
        if (flags[i] && ki) ki[pos] = i;
        pos += flags[i] ? 1u : 0u;
    }
    for (int i = S + tid; i < max_sent; i += kSelThreads) kp[i] = 0;
    if (ki) for (int i = int(nk) + tid; i < max_sent; i += kSelThreads) ki[i] = -1;
    // the largest kept running total is the new length
    uint32_t m = kept_tokens;
#pragma unroll
    for (int d = 16; d; d >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, d));
    __syncthreads();
    if ((tid & 31) == 0) wsum[tid >> 5] = m;
    __syncthreads();
    if (tid == 0) {
        uint32_t mm = 0;
        for (int w = 0; w < kSelThreads / 32; ++w) mm = max(mm, wsum[w]);
        if (n_kept) n_kept[slab] = int(nk);
        if (new_len) new_len[slab] = filled ? budget : int(mm);
    }
}

}  // namespace skipkv

using namespace skipkv;

static int select_impl(const skipkv_shape* shape, const skipkv_params* params, const float* sent_score,
                       const int32_t* sent_off, const int32_t* n_sent, uint8_t* keep, int32_t* kept_idx,
                       int32_t* n_kept, int32_t* new_len, FillArgs fill, void* ws, void* stream) {
    if (int rc = check_shape(shape)) return rc;
    if (!params || !sent_score || !sent_off || !n_sent || !keep) return SKIPKV_ERR_INVALID_ARG;
    if (params->budget < 0 || params->protect_tail < 0) return SKIPKV_ERR_INVALID_ARG;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255)) return SKIPKV_ERR_WORKSPACE;
    int P = 32;
    while (P < shape->max_sent) P <<= 1;
    const size_t smem = size_t(P) * 9;
    if (smem > 200 * 1024) return SKIPKV_ERR_UNSUPPORTED;     // max_sent beyond ~22k sentences per slab
    if (smem > 48 * 1024)   // set on every call: the attribute belongs to the current device's context
        SKIPKV_CUDA(cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
    const int slabs = shape->batch * shape->n_kv_heads;
    SKIPKV_CUDA(launch_dependent(select_kernel, dim3(slabs), dim3(kSelThreads), smem, static_cast<cudaStream_t>(stream),
                                 shape->max_sent, P, params->budget, params->protect_tail, sent_score, sent_off, n_sent, keep,
                                 kept_idx, n_kept, new_len, fill, &static_cast<Header*>(ws)->status));
    return SKIPKV_OK;
}

extern "C" int skipkv_select(const skipkv_shape* shape, const skipkv_params* params, const float* sent_score,
                             const int32_t* sent_off, const int32_t* n_sent, uint8_t* keep, int32_t* kept_idx,
                             int32_t* n_kept, int32_t* new_len, void* ws, void* stream) {
    return select_impl(shape, params, sent_score, sent_off, n_sent, keep, kept_idx, n_kept, new_len, FillArgs{}, ws,
                       stream);
}

static int select_fill_impl(const skipkv_shape* shape, const skipkv_params* params, const float* sent_score,
                            const float* tok_imp, const float* tok_red, const int32_t* sent_off, const int32_t* n_sent,
                            uint8_t* keep, uint8_t* tok_keep, int32_t* kept_idx, int32_t* n_kept, int32_t* new_len, void* ws,
                            void* stream) {
    if (!tok_keep || !params) return SKIPKV_ERR_INVALID_ARG;
    if (int rc = check_shape(shape)) return rc;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255)) return SKIPKV_ERR_WORKSPACE;
    FillArgs fill{};
    fill.tok_keep = tok_keep;
    fill.tok_red = tok_red;
    fill.sigma = params->sigma;
    fill.slab_off = shape->slab_off; fill.cap = shape->cap; fill.Hk = shape->n_kv_heads; fill.max_cap = shape->max_cap;
    if (tok_imp) { fill.tok_imp = tok_imp; fill.from_rows = 1; }
    else { fill.tok_imp = reinterpret_cast<const float*>(static_cast<uint8_t*>(ws) + make_layout(*shape).sc_tokimp); }
    return select_impl(shape, params, sent_score, sent_off, n_sent, keep, kept_idx, n_kept, new_len, fill, ws, stream);
}

extern "C" int skipkv_select_fill(const skipkv_shape* shape, const skipkv_params* params, const float* sent_score,
                                  const float* tok_imp, const int32_t* sent_off, const int32_t* n_sent, uint8_t* keep,
                                  uint8_t* tok_keep, int32_t* kept_idx, int32_t* n_kept, int32_t* new_len, void* ws,
                                  void* stream) {
    return select_fill_impl(shape, params, sent_score, tok_imp, nullptr, sent_off, n_sent, keep, tok_keep, kept_idx, n_kept,
                            new_len, ws, stream);
}

extern "C" int skipkv_select_fill_red(const skipkv_shape* shape, const skipkv_params* params, const float* sent_score,
                                      const float* tok_imp, const float* tok_red, const int32_t* sent_off,
                                      const int32_t* n_sent, uint8_t* keep, uint8_t* tok_keep, int32_t* kept_idx,
                                      int32_t* n_kept, int32_t* new_len, void* ws, void* stream) {
    if (!tok_red) return SKIPKV_ERR_INVALID_ARG;
    return select_fill_impl(shape, params, sent_score, tok_imp, tok_red, sent_off, n_sent, keep, tok_keep, kept_idx, n_kept,
                            new_len, ws, stream);
}
