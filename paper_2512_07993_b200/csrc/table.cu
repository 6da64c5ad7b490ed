// Generation-space lookup table T (paper Section 4.1, "Sentence Similarity Score": sentence
// embeddings are means of the last-layer hidden state over a sentence, pairwise similarity is
// their cosine, the earlier sentence of a pair above tau is flagged with that similarity; the
// table is Eq. "sentence-score-input").  Maintained one decode step at a time:
//   table_close_kernel   adds this step's hidden row to the open sentence of every sequence and,
//                        where the token is a delimiter, closes the sentence: mean, normalise,
//                        store the unit embedding, clear the running sum;
//   table_pss_kernel     compares the sentence just closed with every earlier one of the
//                        sequence (a matrix-vector product over the stored embeddings, bound by
//                        reading them once from HBM) and raises the earlier sentence's entry to
//                        the similarity when it exceeds tau.
// The running maximum over closing sentences equals max_{j>i} G_ij of the one-shot definition.
#include "common.cuh"

namespace skipkv {

constexpr int kCloseThreads = 256;
constexpr int kPssThreads = 256;
constexpr int kPssRowsPerWarp = 2;
constexpr int kPssUnroll = 4;
constexpr int kPssRows = (kPssThreads / 32) * kPssRowsPerWarp;     // earlier sentences per CTA

__global__ void __launch_bounds__(kCloseThreads)
table_close_kernel(int d_model, int max_gen_sent, const __nv_bfloat16* hidden_last, const uint8_t* flag, float* acc,
                   int32_t* acc_count, float* emb, int32_t* n_gen_sent, int32_t* closed, float* lam_table, float eps,
                   uint32_t* status) {
    __shared__ float wsum[kCloseThreads / 32];
    const int b = blockIdx.x, tid = threadIdx.x;
    pdl_trigger();
    pdl_wait();
    const int vecs = d_model / 8;
    const bool close = flag[b] != 0;
    const int cnt = acc_count[b] + 1;
    const float inv = 1.f / float(cnt);
    float* a = acc + size_t(b) * d_model;
    const uint4* h = reinterpret_cast<const uint4*>(hidden_last + size_t(b) * d_model);
    float ss = 0.f;
    for (int v = tid; v < vecs; v += kCloseThreads) {
        const uint4 x = h[v];
        float4 lo = reinterpret_cast<float4*>(a)[2 * v], hi = reinterpret_cast<float4*>(a)[2 * v + 1];
        lo.x += bf16lo(x.x); lo.y += bf16hi(x.x); lo.z += bf16lo(x.y); lo.w += bf16hi(x.y);
        hi.x += bf16lo(x.z); hi.y += bf16hi(x.z); hi.z += bf16lo(x.w); hi.w += bf16hi(x.w);
        reinterpret_cast<float4*>(a)[2 * v] = lo;
        reinterpret_cast<float4*>(a)[2 * v + 1] = hi;
        const float m[8] = {lo.x * inv, lo.y * inv, lo.z * inv, lo.w * inv, hi.x * inv, hi.y * inv, hi.z * inv, hi.w * inv};
#pragma unroll
        for (int k = 0; k < 8; ++k) ss = fmaf(m[k], m[k], ss);
    }
    if (!close) {                                        // uniform over the CTA
        if (tid == 0) { acc_count[b] = cnt; closed[b] = -1; }
        return;
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, d);
    if ((tid & 31) == 0) wsum[tid >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < kCloseThreads / 32; ++w) tot += wsum[w];
    const int n = n_gen_sent[b];
    const bool room = n >= 0 && n < max_gen_sent;
    const float scale = inv / (sqrtf(tot) + eps);
    float* e = emb + (size_t(b) * max_gen_sent + (room ? n : 0)) * d_model;
    for (int v = tid; v < vecs; v += kCloseThreads) {     // each thread re-reads what it wrote above
        float4 lo = reinterpret_cast<float4*>(a)[2 * v], hi = reinterpret_cast<float4*>(a)[2 * v + 1];
        if (room) {
            reinterpret_cast<float4*>(e)[2 * v] = make_float4(lo.x * scale, lo.y * scale, lo.z * scale, lo.w * scale);
            reinterpret_cast<float4*>(e)[2 * v + 1] = make_float4(hi.x * scale, hi.y * scale, hi.z * scale, hi.w * scale);
        }
        reinterpret_cast<float4*>(a)[2 * v] = make_float4(0.f, 0.f, 0.f, 0.f);
        reinterpret_cast<float4*>(a)[2 * v + 1] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (tid == 0) {
        acc_count[b] = 0;
        if (room) {
            lam_table[size_t(b) * max_gen_sent + n] = 0.f;   // no later sentence yet
            n_gen_sent[b] = n + 1;
            closed[b] = n;
        } else {
            closed[b] = -1;                                  // table full: the sentence is dropped
            if (status) atomicOr(status, SKIPKV_STATUS_BAD_TABLE);
        }
    }
}

__global__ void __launch_bounds__(kPssThreads)
table_pss_kernel(int d_model, int max_gen_sent, const float* emb, const int32_t* closed, float* lam_table, float tau) {
    extern __shared__ float4 vnew[];                      // the embedding of the sentence just closed
    const int b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pdl_trigger();
    pdl_wait();
    const int j = closed[b];
    const int row0 = blockIdx.x * kPssRows;
    if (j <= 0 || row0 >= j) return;
    const int quads = d_model / 4;
    const float4* E = reinterpret_cast<const float4*>(emb + size_t(b) * max_gen_sent * d_model);
    for (int k = tid; k < quads; k += kPssThreads) vnew[k] = E[size_t(j) * quads + k];
    __syncthreads();
    float dot[kPssRowsPerWarp];
    const float4* rowp[kPssRowsPerWarp];
#pragma unroll
    for (int r = 0; r < kPssRowsPerWarp; ++r) {
        const int i = row0 + warp * kPssRowsPerWarp + r;
        rowp[r] = E + size_t(i < j ? i : 0) * quads;      // rows at or beyond j are computed on row 0 and discarded
        dot[r] = 0.f;
    }
    // kPssUnroll x kPssRowsPerWarp independent 16-byte loads per lane are issued before the first use
    for (int k0 = lane; k0 < quads; k0 += 32 * kPssUnroll) {
        float4 x[kPssUnroll][kPssRowsPerWarp];
#pragma unroll
        for (int u = 0; u < kPssUnroll; ++u) {
            const int k = k0 + 32 * u;
#pragma unroll
            for (int r = 0; r < kPssRowsPerWarp; ++r)
                x[u][r] = (k < quads) ? __ldcs(rowp[r] + k) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < kPssUnroll; ++u) {
            const int k = k0 + 32 * u;
            const float4 v = (k < quads) ? vnew[k] : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int r = 0; r < kPssRowsPerWarp; ++r)
                dot[r] = fmaf(x[u][r].x, v.x, fmaf(x[u][r].y, v.y, fmaf(x[u][r].z, v.z, fmaf(x[u][r].w, v.w, dot[r]))));
        }
    }
#pragma unroll
    for (int r = 0; r < kPssRowsPerWarp; ++r) {
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) dot[r] += __shfl_xor_sync(0xffffffffu, dot[r], d);
        const int i = row0 + warp * kPssRowsPerWarp + r;
        if (lane == 0 && i < j && dot[r] > tau) {          // this thread alone owns entry i during the launch
            float* t = lam_table + size_t(b) * max_gen_sent + i;
            if (dot[r] > *t) *t = dot[r];
        }
    }
}

}  // namespace skipkv

using namespace skipkv;

extern "C" int skipkv_table_step(int32_t batch, int32_t d_model, int32_t max_gen_sent, const void* hidden_last,
                                 const uint8_t* flag, float* acc, int32_t* acc_count, float* emb, int32_t* n_gen_sent,
                                 int32_t* closed, float* lam_table, float tau, float eps, uint32_t* status,
                                 void* stream) {
    if (batch <= 0 || d_model <= 0 || max_gen_sent <= 0) return SKIPKV_ERR_INVALID_ARG;
    if (!hidden_last || !flag || !acc || !acc_count || !emb || !n_gen_sent || !closed || !lam_table)
        return SKIPKV_ERR_INVALID_ARG;
    if (d_model % 8 != 0 || d_model > 16384) return SKIPKV_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(hidden_last) | reinterpret_cast<uintptr_t>(acc) | reinterpret_cast<uintptr_t>(emb)) & 15)
        return SKIPKV_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    SKIPKV_CUDA(launch_dependent(table_close_kernel, dim3(batch), dim3(kCloseThreads), 0, st, int(d_model),
                                 int(max_gen_sent), static_cast<const __nv_bfloat16*>(hidden_last), flag, acc, acc_count,
                                 emb, n_gen_sent, closed, lam_table, eps, status));
    const size_t smem = size_t(d_model) * 4;
    SKIPKV_CUDA(cudaFuncSetAttribute(table_pss_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
    const dim3 grid((max_gen_sent + kPssRows - 1) / kPssRows, batch);
    SKIPKV_CUDA(launch_dependent(table_pss_kernel, grid, dim3(kPssThreads), smem, st, int(d_model), int(max_gen_sent),
                                 static_cast<const float*>(emb), static_cast<const int32_t*>(closed), lam_table, tau));
    return SKIPKV_OK;
}
