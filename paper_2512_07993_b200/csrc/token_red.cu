// skipkv_token_redundancy: the token-redundancy term at TOKEN granularity (paper Section 4.1,
// token-redundancy equation: R = mean(softmax(Kbar Kbar^T)) with Kbar = K / (||K||_2 + eps)), an
// N' x N' Gram matrix per (sequence, KV head) slab over the slab's own key rows:
//     G_ij  = K_i . K_j / ((|K_i| + eps)(|K_j| + eps))
//     Z_j   = sum_{k != j} exp(G_jk)
//     R_i   = (1/N') sum_{j != i} exp(G_ji) / Z_j
// Three launches:
//   token_norm_kernel      1 / (|K_t| + eps) of every live row (a warp per row); clears Z and R;
//   token_red_kernel<1>    row sums Z;
//   token_red_kernel<2>    R.
// G is symmetric, so every pair of 128-row blocks {I, J} is multiplied and exponentiated once: the tile gives the
// rows of I their sums over the columns (a thread owns a row) and the rows of J theirs as column sums (a butterfly
// over the lanes of each warp, then shared-memory and global reductions).  A work item is block I of a slab
// against I itself and the blocks after it, cyclically, half-way round: every pair once, all items of a slab
// equally long.  Z and R are accumulated with floating-point reductions: sums agree to rounding, not to the bit,
// from run to run.
// The Gram kernels are persistent and warp-specialised.  Warp 0 streams the bf16 key tiles straight from the cache
// with tiled TMA loads (the i tile once per item, the j tiles through a ring), warp 1 issues one
// 128 x 128 x 128 tcgen05.mma group per (i, j) block into one of four tensor-memory accumulators, and four
// warpgroups (one per accumulator, so that one's tensor-memory reads hide behind the others' arithmetic)
// read the accumulators back, scale by the two inverse norms and exponentiate.  The products of bf16
// keys are exact in fp32, so no operand is rounded: normalisation happens after the contraction.
// One exponential per matrix element makes the special-function unit, not the tensor pipe, the limit.
#include "tc.cuh"

namespace skipkv {

constexpr int kTrGroups = 4;                 // epilogue warpgroups = tensor-memory accumulators of 128 columns
constexpr int kTrThreads = (2 + 4 * kTrGroups) * 32;   // TMA warp, MMA warp, epilogue warpgroups
constexpr int kTrStages = 4;                 // j tiles in flight
constexpr float kTrLog2e = 1.4426950408889634f;

struct TrCtl {
    uint64_t afull, aempty, bfull[kTrStages], bempty[kTrStages], tfull[kTrGroups], tempty[kTrGroups];
    uint32_t tmem_base;
    int abort_flag;
    uint32_t wsum[32];
    // per warpgroup, by the parity of its block count: a warp that runs ahead fills the other half while its
    // siblings still read this one (the barrier of the block after orders the reuse)
    alignas(16) float jn[kTrGroups][2][128]; // log2(e) / (|K_j| + eps) of the j block under an accumulator
    alignas(16) float jz[kTrGroups][2][128]; // pass 2: 1 / Z_j
    float part[2][kTrGroups - 1][128];       // the other warpgroups' shares of an item's row sums (by item parity)
    float colsum[kTrGroups][2][128];         // column sums of the tile under an accumulator (by the same parity as jn)
};
static size_t tr_smem_bytes(int slabs) { return 1024 + (1 + kTrStages) * size_t(kOpBytes) + sizeof(TrCtl) + size_t(slabs + 1) * 4; }

// Blocks that item (slab of NB blocks, block I) multiplies block I with: I itself and the next ones, cyclically.
__device__ __forceinline__ int tr_count(int NB, int I) {
    const int half = NB >> 1;
    return (NB & 1) ? 1 + half : half + (I < half ? 1 : 0);
}
// Sum over the 32 lanes of x[c] for every c: lane c returns the sum of column c (31 exchanges).
__device__ __forceinline__ float tr_col_reduce(const float (&x)[32], int lane) {
    float a[16], b[8], c[4], d[2];
    const bool u16 = lane & 16, u8 = lane & 8, u4 = lane & 4, u2 = lane & 2, u1 = lane & 1;
#pragma unroll
    for (int k = 0; k < 16; ++k) a[k] = (u16 ? x[k + 16] : x[k]) + __shfl_xor_sync(0xffffffffu, u16 ? x[k] : x[k + 16], 16);
#pragma unroll
    for (int k = 0; k < 8; ++k) b[k] = (u8 ? a[k + 8] : a[k]) + __shfl_xor_sync(0xffffffffu, u8 ? a[k] : a[k + 8], 8);
#pragma unroll
    for (int k = 0; k < 4; ++k) c[k] = (u4 ? b[k + 4] : b[k]) + __shfl_xor_sync(0xffffffffu, u4 ? b[k] : b[k + 4], 4);
#pragma unroll
    for (int k = 0; k < 2; ++k) d[k] = (u2 ? c[k + 2] : c[k]) + __shfl_xor_sync(0xffffffffu, u2 ? c[k] : c[k + 2], 2);
    return (u1 ? d[1] : d[0]) + __shfl_xor_sync(0xffffffffu, u1 ? d[0] : d[1], 1);
}

__device__ __forceinline__ float tr_ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__global__ void __launch_bounds__(256)
token_norm_kernel(int Hk, int max_cap, const int64_t* slab_off, const int32_t* cap, const __nv_bfloat16* K,
                  const int32_t* kv_len, float eps, float* inv_norm, float* z, float* tok_red) {
    const int slab = blockIdx.y, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    pdl_trigger();
    pdl_wait();
    const int len = min(max(kv_len[slab], 0), min(cap[slab / Hk], max_cap));
    const int t0 = blockIdx.x * 64 + warp * 8;
    if (t0 >= len) return;
    const size_t row0 = slab_row0(slab_off, cap, Hk, slab / Hk, slab % Hk);
    uint2 x[8];
#pragma unroll
    for (int r = 0; r < 8; ++r)
        x[r] = (t0 + r < len) ? reinterpret_cast<const uint2*>(K + (row0 + t0 + r) * kHeadDim)[lane] : make_uint2(0u, 0u);
#pragma unroll
    for (int r = 0; r < 8; ++r) {
        const float a = bf16lo(x[r].x), b = bf16hi(x[r].x), c = bf16lo(x[r].y), d = bf16hi(x[r].y);
        float ss = a * a + b * b + c * c + d * d;
#pragma unroll
        for (int s = 16; s; s >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, s);
        if (lane == 0 && t0 + r < len) {
            inv_norm[size_t(slab) * max_cap + t0 + r] = 1.f / (sqrtf(ss) + eps);
            z[size_t(slab) * max_cap + t0 + r] = 0.f;            // both are accumulated by the passes that follow
            tok_red[row0 + t0 + r] = 0.f;
        }
    }
}

template <int kPass>
__global__ void __launch_bounds__(kTrThreads, 1)
token_red_kernel(const __grid_constant__ CUtensorMap mapK, int n_slabs, int Hk, int max_cap, const int64_t* slab_off,
                 const int32_t* cap, const int32_t* kv_len, const float* inv_norm, float* z, float* tok_red,
                 const Header* hdr) {
    extern __shared__ uint8_t tr_smem_raw[];
    const uint32_t raw = smem_u32(tr_smem_raw);
    uint8_t* At = tr_smem_raw + (((raw + 1023u) & ~1023u) - raw);
    uint8_t* Bt = At + kOpBytes;
    TrCtl* ctl = reinterpret_cast<TrCtl*>(Bt + kTrStages * kOpBytes);
    int* ipref = reinterpret_cast<int*>(ctl + 1);                                // [n_slabs + 1] prefix of i blocks
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int G = gridDim.x, cta = blockIdx.x;
    auto len_of = [&](int s) { return min(max(kv_len[s], 0), min(cap[s / Hk], max_cap)); };
    pdl_trigger();

    if (tid == 0) {
        mbar_init(&ctl->afull, 1);
        mbar_init(&ctl->aempty, 1);
        for (int s = 0; s < kTrStages; ++s) { mbar_init(&ctl->bfull[s], 1); mbar_init(&ctl->bempty[s], 1); }
        for (int s = 0; s < kTrGroups; ++s) { mbar_init(&ctl->tfull[s], 1); mbar_init(&ctl->tempty[s], 4); }
        ctl->abort_flag = 0;
        mbar_fence_init();
        tmap_prefetch(&mapK);
    }
    if (warp == 1) tmem_alloc(&ctl->tmem_base, 128 * kTrGroups);
    pdl_wait();                                          // kv_len and the norms may come from the kernels before
    uint32_t* status = const_cast<uint32_t*>(&hdr->status);
    const uint32_t limit = load_wait_limit(hdr);
    tc_fence_before();
    cta_prefix<kTrThreads>(n_slabs, [&](int s) { return (len_of(s) + 127) >> 7; }, ipref, ctl->wsum);   // i blocks per slab
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    const int n_items = ipref[n_slabs];
    auto row0_of = [&](int s) { return int(slab_row0(slab_off, cap, Hk, s / Hk, s % Hk)); };

    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            int slab = 0;
            uint32_t bc = 0, ic = 0;                                // j blocks and items issued so far
            for (int item = cta; item < n_items && ok; item += G, ++ic) {
                while (ipref[slab + 1] <= item) ++slab;
                const int NB = (len_of(slab) + 127) >> 7, row0 = row0_of(slab);
                const int I = item - ipref[slab], NJ = tr_count(NB, I);
                const int i0 = I * 128;
                if (ic > 0) ok = role_wait(&ctl->aempty, (ic - 1) & 1u, limit, &ctl->abort_flag, status);
                if (!ok) break;
                mbar_expect_tx(&ctl->afull, kOpBytes);
                tma_load_2d(At, &mapK, 0, row0 + i0, &ctl->afull);
                tma_load_2d(At + kOpHalfBytes, &mapK, 64, row0 + i0, &ctl->afull);
                for (int jb = 0; jb < NJ && ok; ++jb, ++bc) {
                    const int s = bc % kTrStages;
                    if (bc >= kTrStages) ok = role_wait(&ctl->bempty[s], ((bc / kTrStages) - 1) & 1u, limit, &ctl->abort_flag, status);
                    if (!ok) break;
                    uint8_t* dst = Bt + size_t(s) * kOpBytes;
                    mbar_expect_tx(&ctl->bfull[s], kOpBytes);
                    const int J = (I + jb) % NB;
                    tma_load_2d(dst, &mapK, 0, row0 + J * 128, &ctl->bfull[s]);
                    tma_load_2d(dst + kOpHalfBytes, &mapK, 64, row0 + J * 128, &ctl->bfull[s]);
                }
            }
            if (!ok) {                                   // let the copies in flight land before the CTA exits
                mbar_wait(&ctl->afull, 0u, 1u << 16); mbar_wait(&ctl->afull, 1u, 1u << 16);
                for (int s = 0; s < kTrStages; ++s) { mbar_wait(&ctl->bfull[s], 0u, 1u << 16); mbar_wait(&ctl->bfull[s], 1u, 1u << 16); }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            bool ok = true;
            int slab = 0;
            uint32_t bc = 0, ic = 0;
            const uint32_t a = smem_u32(At);
            for (int item = cta; item < n_items && ok; item += G, ++ic) {
                while (ipref[slab + 1] <= item) ++slab;
                const int NJ = tr_count((len_of(slab) + 127) >> 7, item - ipref[slab]);
                ok = role_wait(&ctl->afull, ic & 1u, limit, &ctl->abort_flag, status);
                for (int jb = 0; jb < NJ && ok; ++jb, ++bc) {
                    const int st = bc % kTrStages, s = bc % kTrGroups;
                    ok = role_wait(&ctl->bfull[st], (bc / kTrStages) & 1u, limit, &ctl->abort_flag, status);
                    if (ok && bc >= kTrGroups) ok = role_wait(&ctl->tempty[s], ((bc / kTrGroups) - 1) & 1u, limit, &ctl->abort_flag, status);
                    if (!ok) break;
                    tc_fence_after();
                    umma_tile_128x128x128(tmem_base + s * 128, a, smem_u32(Bt + size_t(st) * kOpBytes), false);
                    umma_commit(&ctl->tfull[s]);
                    umma_commit(&ctl->bempty[st]);
                }
                if (ok) umma_commit(&ctl->aempty);                   // every MMA that reads this i tile has completed
            }
        }
    } else {
        const int grp = (warp - 2) >> 2;                           // the accumulator this warpgroup drains
        const int quarter = warp & 3, wt = (tid - 64) & 127;
        const uint32_t lane_addr = tmem_base + (uint32_t(quarter * 32) << 16) + grp * 128;
        bool ok = true;
        int slab = 0;
        uint32_t bc = 0, ic = 0;
        ctl->colsum[grp][0][wt] = 0.f;
        ctl->colsum[grp][1][wt] = 0.f;
        named_bar_sync(1 + grp, 128);
        for (int item = cta; item < n_items; item += G, ++ic) {
            while (ipref[slab + 1] <= item) ++slab;
            const int S = len_of(slab), NB = (S + 127) >> 7;
            const int I = item - ipref[slab], NJ = tr_count(NB, I);
            const size_t sbase = size_t(slab) * max_cap;
            const int i0 = I * 128;
            const int row = quarter * 32 + lane;
            const int i = i0 + row;
            const float inv_i = (i < S) ? inv_norm[sbase + i] : 0.f;
            float invz_i = 0.f;                                    // pass 2: 1 / Z_i, the weight of this row in column sums
            if (kPass == 2 && i < S) { const float zz = z[sbase + i]; invz_i = (zz > 0.f) ? 1.f / zz : 0.f; }
            const float inv_S = 1.f / float(max(S, 1));
            float accum = 0.f;
            for (int jb = 0; jb < NJ; ++jb, ++bc) {
                if (int(bc % kTrGroups) != grp) continue;          // another warpgroup's block
                const int J = (I + jb) % NB, j0 = J * 128;
                const bool diag = jb == 0;                         // the block against itself: row sums only
                const uint32_t par = (bc / kTrGroups) & 1u;
                float* jn_s = ctl->jn[grp][par];
                float* jz_s = ctl->jz[grp][par];
                float* cs = ctl->colsum[grp][par];
                {
                    const int j = j0 + wt;
                    jn_s[wt] = (j < S) ? inv_norm[sbase + j] * kTrLog2e : 0.f;
                    if (kPass == 2) {
                        const float zz = (j < S) ? z[sbase + j] : 1.f;
                        jz_s[wt] = (zz > 0.f) ? 1.f / zz : 0.f;
                    }
                    named_bar_sync(1 + grp, 128);
                }
                if (ok) {
                    ok = role_wait(&ctl->tfull[grp], par, limit, &ctl->abort_flag, status);
                    ok = __all_sync(0xffffffffu, ok);
                }
                if (ok) {
                    tc_fence_after();
                    const bool interior = !diag && (j0 + 128 <= S) && (i0 + 128 <= S);
#pragma unroll 1
                    for (int ch = 0; ch < 4; ++ch) {
                        float v[32];
                        tmem_ld32(lane_addr + ch * 32, v);
                        const float* jn = jn_s + ch * 32;
                        const float* jz = jz_s + ch * 32;
                        if (interior) {
                            // two elements per instruction (packed fp32 multiply / add): the epilogue is issue-bound
                            float2 acc2 = make_float2(0.f, 0.f);
                            const float2 inv2 = make_float2(inv_i, inv_i);
#pragma unroll
                            for (int jj = 0; jj < 32; jj += 2) {
                                const float2 w = __fmul2_rn(__fmul2_rn(make_float2(v[jj], v[jj + 1]), inv2),
                                                            *reinterpret_cast<const float2*>(jn + jj));
                                const float2 e = make_float2(tr_ex2(w.x), tr_ex2(w.y));
                                if (kPass == 1) acc2 = __fadd2_rn(acc2, e);
                                else acc2 = __ffma2_rn(e, *reinterpret_cast<const float2*>(jz + jj), acc2);
                                v[jj] = e.x; v[jj + 1] = e.y;
                            }
                            accum += acc2.x + acc2.y;
                        } else {
#pragma unroll
                            for (int jj = 0; jj < 32; ++jj) {
                                const int j = j0 + ch * 32 + jj;
                                float e = 0.f;
                                if (j < S && i < S && j != i) {
                                    e = tr_ex2(v[jj] * inv_i * jn[jj]);
                                    if (kPass == 1) accum += e; else accum = fmaf(e, jz[jj], accum);
                                }
                                v[jj] = e;
                            }
                        }
                        if (!diag) {
                            // the same exponentials as column sums: they belong to the rows of block J
                            if (kPass == 2) {
#pragma unroll
                                for (int jj = 0; jj < 32; ++jj) v[jj] *= invz_i;
                            }
                            atomicAdd(&cs[ch * 32 + lane], tr_col_reduce(v, lane));
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&ctl->tempty[grp]);
                }
                if (!diag) {
                    named_bar_sync(1 + grp, 128);                  // the four warps' shares of the column sums are in
                    const int j = j0 + wt;
                    if (ok && j < S) {
                        if (kPass == 1) atomicAdd(&z[sbase + j], cs[wt]);
                        else atomicAdd(&tok_red[size_t(row0_of(slab)) + j], cs[wt] * inv_S);
                    }
                    cs[wt] = 0.f;                                  // used again two blocks later, behind a barrier
                }
            }
            // the warpgroups hold the row sums over interleaved j blocks: the others hand their shares to the first
            if (grp > 0) ctl->part[ic & 1][grp - 1][row] = accum;
            named_bar_sync(1 + kTrGroups, 128 * kTrGroups);
            if (grp == 0 && ok && i < S) {
#pragma unroll
                for (int g = 0; g < kTrGroups - 1; ++g) accum += ctl->part[ic & 1][g][row];
                if (kPass == 1) atomicAdd(&z[sbase + i], accum);
                else atomicAdd(&tok_red[size_t(row0_of(slab)) + i], accum * inv_S);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 128 * kTrGroups);
    }
}

}  // namespace skipkv

using namespace skipkv;

extern "C" int skipkv_token_redundancy(const skipkv_shape* shape, const skipkv_params* params, const void* K,
                                       const int32_t* kv_len, float* tok_red, void* ws, void* stream) {
    if (int rc = check_shape(shape)) return rc;
    if (!params || !K || !kv_len || !tok_red) return SKIPKV_ERR_INVALID_ARG;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255)) return SKIPKV_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(K) & 15) return SKIPKV_ERR_INVALID_ARG;
    const WsLayout L = make_layout(*shape);
    uint8_t* w = static_cast<uint8_t*>(ws);
    const Header* hdr = reinterpret_cast<const Header*>(w + L.header);
    float* inv_norm = reinterpret_cast<float*>(w + L.tr_inv);
    float* z = reinterpret_cast<float*>(w + L.tr_z);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CUtensorMap mapK;
    if (int rc = tmap_rows(&mapK, K, uint64_t(shape->total_rows), 128)) return rc;
    const size_t smem = tr_smem_bytes(L.slabs);
    if (smem > 227 * 1024) return SKIPKV_ERR_UNSUPPORTED;
    const int Hk = shape->n_kv_heads;
    SKIPKV_CUDA(launch_dependent(token_norm_kernel, dim3((shape->max_cap + 63) / 64, L.slabs), dim3(256), 0, st, Hk,
                                 int(shape->max_cap), shape->slab_off, shape->cap, static_cast<const __nv_bfloat16*>(K),
                                 kv_len, params->eps, inv_norm, z, tok_red));
    const long long max_items = (long long)L.slabs * ((shape->max_cap + 127) / 128);
    int grid = num_sms();
    if (max_items < grid) grid = int(max_items);
    SKIPKV_CUDA(cudaFuncSetAttribute(token_red_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
    SKIPKV_CUDA(cudaFuncSetAttribute(token_red_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
    SKIPKV_CUDA(launch_dependent(token_red_kernel<1>, dim3(grid), dim3(kTrThreads), smem, st, mapK, int(L.slabs), Hk,
                                 int(shape->max_cap), shape->slab_off, shape->cap, kv_len, static_cast<const float*>(inv_norm),
                                 z, tok_red, hdr));
    SKIPKV_CUDA(launch_dependent(token_red_kernel<2>, dim3(grid), dim3(kTrThreads), smem, st, mapK, int(L.slabs), Hk,
                                 int(shape->max_cap), shape->slab_off, shape->cap, kv_len, static_cast<const float*>(inv_norm),
                                 z, tok_red, hdr));
    return SKIPKV_OK;
}
