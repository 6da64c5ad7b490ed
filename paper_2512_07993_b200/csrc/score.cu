// skipkv_score: sentence scores per (sequence, KV head) slab (paper Section 4.1).
//
//   sweep 1   log-sum-exp of every window-query row over the slab's tokens (partial per chunk)
//   combine   per-row log-sum-exp
//   sweep 2   tok_imp[t] = (1/alpha) sum_w max_q 2^(s_q[w][t] - lse_q[w])   (max before exp: exp is monotone)
//   pool      per sentence: mean tok_imp, mean key, normalisation
//   gram x2   pairwise cosine G; pass 1: row sums Z_i = sum_{j!=i} e^{G_ij} and lam_i = max_{j>i} G_ij;
//             pass 2: red_i = (1/S) sum_{j!=i} e^{G_ij} / Z_j (G symmetric) and the final score.
//
// Logits are kept in base 2: s = (q.k) * log2(e)/sqrt(d).  |G| <= 1 so the row softmax of G
// needs no max subtraction.
#include "common.cuh"

namespace skipkv {

constexpr int kS1Tile = 32;         // tokens per shared-memory tile in sweep 1
constexpr int kS2Tokens = 128;      // tokens (threads) per CTA in sweep 2
constexpr int kS2RowBlk = 64;       // query rows staged per pass in sweep 2 (multiple of the group size is enforced below)

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

struct SlabView {
    const uint8_t* K;      // first row of the slab
    int N;                 // live rows
    int b, h;
};

__device__ __forceinline__ SlabView slab_view(const uint8_t* K, const int64_t* slab_off, const int32_t* cap,
                                              const int32_t* kv_len, int Hk, int slab) {
    SlabView v;
    v.b = slab / Hk;
    v.h = slab % Hk;
    v.K = K + slab_row0(slab_off, cap, Hk, v.b, v.h) * kRowBytes;
    v.N = min(max(kv_len[slab], 0), cap[v.b]);
    return v;
}

// query row r of a group (r = q_local * window + w) as 128 fp32 registers, pre-scaled
__device__ __forceinline__ void load_row_scaled(const uint8_t* row, float scale, float (&x)[kHeadDim]) {
    const uint4* p = reinterpret_cast<const uint4*>(row);
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const uint4 u = p[i];
        x[8 * i + 0] = bf16lo(u.x) * scale; x[8 * i + 1] = bf16hi(u.x) * scale;
        x[8 * i + 2] = bf16lo(u.y) * scale; x[8 * i + 3] = bf16hi(u.y) * scale;
        x[8 * i + 4] = bf16lo(u.z) * scale; x[8 * i + 5] = bf16hi(u.z) * scale;
        x[8 * i + 6] = bf16lo(u.w) * scale; x[8 * i + 7] = bf16hi(u.w) * scale;
    }
}

// ---------------------------------------------------------------------------------------
// sweep 1: thread = query row (held in registers), tokens broadcast from shared memory
// grid (chunks, slabs, row blocks of 256)
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
score_sweep1_kernel(int Hq, int Hk, int window, int qrows, int sc_chunks, const int64_t* slab_off, const int32_t* cap,
                    const uint8_t* K, const uint8_t* q_win, const int32_t* kv_len, float2* sc_part) {
    __shared__ __align__(16) float kt[kS1Tile][kHeadDim];
    const int slab = blockIdx.y, chunk = blockIdx.x;
    const SlabView sv = slab_view(K, slab_off, cap, kv_len, Hk, slab);
    const int t0 = chunk * kScoreChunk, t1 = min(t0 + kScoreChunk, sv.N);
    if (t0 >= sv.N) return;
    const int n = Hq / Hk;
    const int r = blockIdx.z * 256 + threadIdx.x;
    const bool active = r < qrows;
    float qv[kHeadDim];
    if (active) {
        // q_win[b][Hq][window][128]; rows of the group are contiguous: r = q_local*window + w
        const uint8_t* qrow = q_win + ((size_t(sv.b) * Hq + size_t(sv.h) * n) * window + r) * kRowBytes;
        load_row_scaled(qrow, 1.4426950408889634f * rsqrtf(float(kHeadDim)), qv);
    }
    float m = -INFINITY, sum = 0.f;
    for (int tb = t0; tb < t1; tb += kS1Tile) {
        const int nt = min(kS1Tile, t1 - tb);
        __syncthreads();
        // stage nt rows as fp32: 16-byte chunks, 16 per row
        for (int i = threadIdx.x; i < nt * 16; i += blockDim.x) {
            const int row = i >> 4, c = i & 15;
            const uint4 u = reinterpret_cast<const uint4*>(sv.K + size_t(tb + row) * kRowBytes)[c];
            float4* d = reinterpret_cast<float4*>(&kt[row][c * 8]);
            d[0] = make_float4(bf16lo(u.x), bf16hi(u.x), bf16lo(u.y), bf16hi(u.y));
            d[1] = make_float4(bf16lo(u.z), bf16hi(u.z), bf16lo(u.w), bf16hi(u.w));
        }
        __syncthreads();
        if (active) {
            for (int t = 0; t < nt; ++t) {
                float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
                const float4* kr = reinterpret_cast<const float4*>(kt[t]);
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    const float4 k4 = kr[c];
                    a0 = fmaf(qv[4 * c + 0], k4.x, a0);
                    a1 = fmaf(qv[4 * c + 1], k4.y, a1);
                    a2 = fmaf(qv[4 * c + 2], k4.z, a2);
                    a3 = fmaf(qv[4 * c + 3], k4.w, a3);
                }
                const float s = (a0 + a1) + (a2 + a3);
                if (s > m) { sum *= ex2f(m - s); m = s; }
                sum += ex2f(s - m);
            }
        }
    }
    if (active) sc_part[(size_t(slab) * sc_chunks + chunk) * qrows + r] = make_float2(m, sum);
}

__global__ void score_lse_kernel(int qrows, int sc_chunks, const int32_t* kv_len, const float2* sc_part,
                                 float* sc_lse) {
    const int slab = blockIdx.x;
    const int N = max(kv_len[slab], 0);
    const int nch = min(sc_chunks, (N + kScoreChunk - 1) / kScoreChunk);
    for (int r = threadIdx.x; r < qrows; r += blockDim.x) {
        float M = -INFINITY;
        for (int c = 0; c < nch; ++c) M = fmaxf(M, sc_part[(size_t(slab) * sc_chunks + c) * qrows + r].x);
        float s = 0.f;
        for (int c = 0; c < nch; ++c) {
            const float2 p = sc_part[(size_t(slab) * sc_chunks + c) * qrows + r];
            s += p.y * ex2f(p.x - M);
        }
        sc_lse[size_t(slab) * qrows + r] = (nch > 0) ? M + log2f(s) : 0.f;
    }
}

// ---------------------------------------------------------------------------------------
// sweep 2: thread = token (key row in registers), query rows broadcast from shared memory
// grid (ceil(max_cap/128), slabs)
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kS2Tokens)
score_sweep2_kernel(int Hq, int Hk, int window, int qrows, int max_cap, const int64_t* slab_off, const int32_t* cap,
                    const uint8_t* K, const uint8_t* q_win, const int32_t* kv_len, const float* sc_lse,
                    float* tok_imp_user, float* tok_imp_ws) {
    __shared__ __align__(16) float qs[kS2RowBlk][kHeadDim];
    __shared__ float lse_s[kS2RowBlk];
    const int slab = blockIdx.y;
    const SlabView sv = slab_view(K, slab_off, cap, kv_len, Hk, slab);
    const int t = blockIdx.x * kS2Tokens + threadIdx.x;
    if (blockIdx.x * kS2Tokens >= sv.N) return;
    const bool active = t < sv.N;
    const int n = Hq / Hk;
    float kv[kHeadDim];
    if (active) load_row_scaled(sv.K + size_t(t) * kRowBytes, 1.4426950408889634f * rsqrtf(float(kHeadDim)), kv);
    const uint8_t* qbase = q_win + (size_t(sv.b) * Hq + size_t(sv.h) * n) * window * kRowBytes;
    const float* lse = sc_lse + size_t(slab) * qrows;
    // window rows are staged in blocks of wb rows x n heads, laid out [w][q] so a block is contiguous in w
    const int wb = kS2RowBlk / n;
    float total = 0.f;
    for (int w0 = 0; w0 < window; w0 += wb) {
        const int nw = min(wb, window - w0);
        __syncthreads();
        for (int i = threadIdx.x; i < nw * n * 16; i += kS2Tokens) {
            const int lr = i >> 4, c = i & 15;            // local row lr = wl * n + ql
            const int wl = lr / n, ql = lr % n;
            const uint4 u = reinterpret_cast<const uint4*>(qbase + (size_t(ql) * window + (w0 + wl)) * kRowBytes)[c];
            float4* d = reinterpret_cast<float4*>(&qs[lr][c * 8]);
            d[0] = make_float4(bf16lo(u.x), bf16hi(u.x), bf16lo(u.y), bf16hi(u.y));
            d[1] = make_float4(bf16lo(u.z), bf16hi(u.z), bf16lo(u.w), bf16hi(u.w));
        }
        for (int i = threadIdx.x; i < nw * n; i += kS2Tokens) {
            const int wl = i / n, ql = i % n;
            lse_s[i] = lse[ql * window + (w0 + wl)];
        }
        __syncthreads();
        if (active) {
            for (int wl = 0; wl < nw; ++wl) {
                float best = -INFINITY;
                for (int ql = 0; ql < n; ++ql) {
                    const float4* qr = reinterpret_cast<const float4*>(qs[wl * n + ql]);
                    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        const float4 q4 = qr[c];
                        a0 = fmaf(kv[4 * c + 0], q4.x, a0);
                        a1 = fmaf(kv[4 * c + 1], q4.y, a1);
                        a2 = fmaf(kv[4 * c + 2], q4.z, a2);
                        a3 = fmaf(kv[4 * c + 3], q4.w, a3);
                    }
                    best = fmaxf(best, ((a0 + a1) + (a2 + a3)) - lse_s[wl * n + ql]);
                }
                total += ex2f(best);
            }
        }
    }
    if (active) {
        const float v = total / float(window);
        tok_imp_ws[size_t(slab) * max_cap + t] = v;
        if (tok_imp_user) tok_imp_user[slab_row0(slab_off, cap, Hk, sv.b, sv.h) + t] = v;
    }
}

// ---------------------------------------------------------------------------------------
// pooling: one warp per sentence, 4 channels per lane
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
score_pool_kernel(int Hk, int max_sent, int max_cap, const int64_t* slab_off, const int32_t* cap, const uint8_t* K,
                  const int32_t* kv_len, const int32_t* sent_off, const int32_t* n_sent, float eps,
                  const float* tok_imp_ws, float* sent_imp, float* sc_vbar) {
    const int slab = blockIdx.y;
    const int lane = threadIdx.x & 31;
    const int i = blockIdx.x * 8 + (threadIdx.x >> 5);
    const int S = min(n_sent[slab], max_sent);
    if (i >= S) return;
    const SlabView sv = slab_view(K, slab_off, cap, kv_len, Hk, slab);
    const int32_t* so = sent_off + size_t(slab) * (max_sent + 1);
    const int b = max(so[i], 0), e = min(so[i + 1], sv.N);
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f, ti = 0.f;
    for (int t = b; t < e; ++t) {
        const uint2 u = reinterpret_cast<const uint2*>(sv.K + size_t(t) * kRowBytes)[lane];
        a0 += bf16lo(u.x); a1 += bf16hi(u.x); a2 += bf16lo(u.y); a3 += bf16hi(u.y);
    }
    for (int t = b + lane; t < e; t += 32) ti += tok_imp_ws[size_t(slab) * max_cap + t];
    const float len = float(max(e - b, 1));
    a0 /= len; a1 /= len; a2 /= len; a3 /= len;
    float nn = a0 * a0 + a1 * a1 + a2 * a2 + a3 * a3;
#pragma unroll
    for (int d = 16; d; d >>= 1) {
        nn += __shfl_xor_sync(0xffffffffu, nn, d);
        ti += __shfl_xor_sync(0xffffffffu, ti, d);
    }
    const float inv = 1.f / (sqrtf(nn) + eps);
    reinterpret_cast<float4*>(sc_vbar + (size_t(slab) * max_sent + i) * kHeadDim)[lane] =
        make_float4(a0 * inv, a1 * inv, a2 * inv, a3 * inv);
    if (lane == 0) sent_imp[size_t(slab) * max_sent + i] = (e > b) ? ti / len : 0.f;
}

// ---------------------------------------------------------------------------------------
// Gram passes: CTA = 32 sentences i (one per warp) x all j in tiles of 32 (one per lane)
// ---------------------------------------------------------------------------------------
template <int kPass>
__global__ void __launch_bounds__(1024)
score_gram_kernel(int max_sent, const int32_t* n_sent, float sigma, float tau, const float* sc_vbar, float* sc_z,
                  const float* sent_imp, float* sent_red, float* sent_lam, float* sent_score) {
    __shared__ float vi[32][kHeadDim];
    __shared__ float vj[32][kHeadDim + 1];
    const int slab = blockIdx.y;
    const int S = min(n_sent[slab], max_sent);
    const int i0 = blockIdx.x * 32;
    if (i0 >= S) return;
    const int ti = threadIdx.x >> 5, tj = threadIdx.x & 31;
    const int i = i0 + ti;
    const float* vb = sc_vbar + size_t(slab) * max_sent * kHeadDim;
    for (int k = threadIdx.x; k < 32 * kHeadDim; k += 1024) {
        const int r = k / kHeadDim, c = k % kHeadDim;
        vi[r][c] = (i0 + r < S) ? vb[size_t(i0 + r) * kHeadDim + c] : 0.f;
    }
    float accum = 0.f, mx = -INFINITY;
    for (int j0 = 0; j0 < S; j0 += 32) {
        __syncthreads();
        for (int k = threadIdx.x; k < 32 * kHeadDim; k += 1024) {
            const int r = k / kHeadDim, c = k % kHeadDim;
            vj[r][c] = (j0 + r < S) ? vb[size_t(j0 + r) * kHeadDim + c] : 0.f;
        }
        __syncthreads();
        const int j = j0 + tj;
        float g0 = 0.f, g1 = 0.f, g2 = 0.f, g3 = 0.f;
#pragma unroll 8
        for (int c = 0; c < kHeadDim; c += 4) {
            g0 = fmaf(vi[ti][c + 0], vj[tj][c + 0], g0);
            g1 = fmaf(vi[ti][c + 1], vj[tj][c + 1], g1);
            g2 = fmaf(vi[ti][c + 2], vj[tj][c + 2], g2);
            g3 = fmaf(vi[ti][c + 3], vj[tj][c + 3], g3);
        }
        const float g = (g0 + g1) + (g2 + g3);
        if (j < S && j != i && i < S) {
            const float e = __expf(g);
            if (kPass == 1) {
                accum += e;
                if (j > i) mx = fmaxf(mx, g);
            } else {
                accum += e / sc_z[size_t(slab) * max_sent + j];
            }
        }
    }
#pragma unroll
    for (int d = 16; d; d >>= 1) {
        accum += __shfl_xor_sync(0xffffffffu, accum, d);
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d));
    }
    if (tj == 0 && i < S) {
        const size_t o = size_t(slab) * max_sent + i;
        if (kPass == 1) {
            sc_z[o] = accum;
            sent_lam[o] = (mx > tau) ? mx : 0.f;
        } else {
            const float red = accum / float(S);
            sent_red[o] = red;
            sent_score[o] = sigma * sent_imp[o] - (1.f - sigma) * red - sent_lam[o];
        }
    }
}

}  // namespace skipkv

using namespace skipkv;

extern "C" int skipkv_score(const skipkv_shape* shape, const skipkv_params* params, const void* K, const void* q_win,
                            const int32_t* kv_len, const int32_t* sent_off, const int32_t* n_sent, float* tok_imp,
                            float* sent_imp, float* sent_red, float* sent_lam, float* sent_score, void* ws,
                            void* stream) {
    if (int rc = check_shape(shape)) return rc;
    if (!params || !K || !q_win || !kv_len || !sent_off || !n_sent || !sent_imp || !sent_red || !sent_lam || !sent_score)
        return SKIPKV_ERR_INVALID_ARG;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255)) return SKIPKV_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(K) & 15) || (reinterpret_cast<uintptr_t>(q_win) & 15)) return SKIPKV_ERR_INVALID_ARG;
    if (shape->max_sent <= 0) return SKIPKV_OK;
    const WsLayout L = make_layout(*shape);
    uint8_t* w = static_cast<uint8_t*>(ws);
    float2* sc_part = reinterpret_cast<float2*>(w + L.sc_part);
    float* sc_lse = reinterpret_cast<float*>(w + L.sc_lse);
    float* sc_tok = reinterpret_cast<float*>(w + L.sc_tokimp);
    float* sc_vbar = reinterpret_cast<float*>(w + L.sc_vbar);
    float* sc_z = reinterpret_cast<float*>(w + L.sc_z);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int Hq = shape->n_q_heads, Hk = shape->n_kv_heads;
    const uint8_t* Kb = static_cast<const uint8_t*>(K);
    const uint8_t* Qb = static_cast<const uint8_t*>(q_win);

    {
        const int threads = L.qrows >= 256 ? 256 : ((L.qrows + 31) / 32) * 32;
        dim3 grid(L.sc_chunks, L.slabs, (L.qrows + 255) / 256);
        score_sweep1_kernel<<<grid, threads, 0, st>>>(Hq, Hk, shape->window, L.qrows, L.sc_chunks, shape->slab_off,
                                                      shape->cap, Kb, Qb, kv_len, sc_part);
        SKIPKV_CUDA(cudaGetLastError());
    }
    score_lse_kernel<<<L.slabs, 128, 0, st>>>(L.qrows, L.sc_chunks, kv_len, sc_part, sc_lse);
    SKIPKV_CUDA(cudaGetLastError());
    {
        dim3 grid((shape->max_cap + kS2Tokens - 1) / kS2Tokens, L.slabs);
        score_sweep2_kernel<<<grid, kS2Tokens, 0, st>>>(Hq, Hk, shape->window, L.qrows, shape->max_cap,
                                                        shape->slab_off, shape->cap, Kb, Qb, kv_len, sc_lse, tok_imp,
                                                        sc_tok);
        SKIPKV_CUDA(cudaGetLastError());
    }
    {
        dim3 grid((shape->max_sent + 7) / 8, L.slabs);
        score_pool_kernel<<<grid, 256, 0, st>>>(Hk, shape->max_sent, shape->max_cap, shape->slab_off, shape->cap, Kb,
                                                kv_len, sent_off, n_sent, params->eps, sc_tok, sent_imp, sc_vbar);
        SKIPKV_CUDA(cudaGetLastError());
    }
    {
        dim3 grid((shape->max_sent + 31) / 32, L.slabs);
        score_gram_kernel<1><<<grid, 1024, 0, st>>>(shape->max_sent, n_sent, params->sigma, params->tau, sc_vbar, sc_z,
                                                    sent_imp, sent_red, sent_lam, sent_score);
        SKIPKV_CUDA(cudaGetLastError());
        score_gram_kernel<2><<<grid, 1024, 0, st>>>(shape->max_sent, n_sent, params->sigma, params->tau, sc_vbar, sc_z,
                                                    sent_imp, sent_red, sent_lam, sent_score);
        SKIPKV_CUDA(cudaGetLastError());
    }
    return SKIPKV_OK;
}
