// Steering-vector add (paper Section 4.2: H <- H + alpha_t * v at delimiter tokens) and the
// per-step K/V append.  Both are tiny, bandwidth-trivial kernels: 16-byte vector accesses.
#include "common.cuh"
#include "steer.cuh"

namespace skipkv {

__global__ void steer_kernel(int batch, int d_model, __nv_bfloat16* hidden, const __nv_bfloat16* v,
                             const float* alpha, const uint8_t* flag) {
    const int vec_per_row = d_model / 8;
    const int total = batch * vec_per_row;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x)
        steer_vec8(i, vec_per_row, hidden, v, alpha, flag);
}

__global__ void append_kernel(int batch, int Hk, const int64_t* slab_off, const int32_t* cap, uint4* K, uint4* V,
                              const uint4* k_new, const uint4* v_new, int32_t* kv_len, uint32_t* status) {
    // one 16-thread group per (b, h): 16 x 16 B = one 256-byte row
    const int g = (blockIdx.x * blockDim.x + threadIdx.x) / 16;
    const int c = threadIdx.x % 16;
    if (g >= batch * Hk) return;
    const int b = g / Hk, h = g % Hk;
    const int len = kv_len[g];
    if (len >= cap[b] || len < 0) {
        if (c == 0) atomicOr(status, SKIPKV_STATUS_BAD_TABLE);
        return;
    }
    const size_t row = slab_row0(slab_off, cap, Hk, b, h) + len;
    K[row * 16 + c] = k_new[size_t(g) * 16 + c];
    V[row * 16 + c] = v_new[size_t(g) * 16 + c];
    __syncwarp();
    if (c == 0) kv_len[g] = len + 1;
}

// One decode step's bookkeeping: the K/V append of append_kernel, the range-list update for the new token (it
// extends the open last sentence, or starts a new one), and the newest query into its slot of the window.
__global__ void append_step_kernel(int batch, int Hk, int Hq, int window, int max_sent, const int64_t* slab_off,
                                   const int32_t* cap, uint4* K, uint4* V, const uint4* k_new, const uint4* v_new,
                                   int32_t* kv_len, int32_t* sent_off, int32_t* sent_id, int32_t* n_sent,
                                   const uint8_t* new_sent, const int32_t* gen_id, uint4* q_win, const uint4* q,
                                   int slot, uint32_t* status) {
    const int g = (blockIdx.x * blockDim.x + threadIdx.x) / 16;
    const int c = threadIdx.x % 16;
    pdl_trigger();
    pdl_wait();
    if (g < batch * Hk) {
        const int b = g / Hk, h = g % Hk;
        const int len = kv_len[g];
        if (len >= cap[b] || len < 0) {
            if (c == 0) atomicOr(status, SKIPKV_STATUS_BAD_TABLE);
            return;
        }
        const size_t row = slab_row0(slab_off, cap, Hk, b, h) + len;
        K[row * 16 + c] = k_new[size_t(g) * 16 + c];
        V[row * 16 + c] = v_new[size_t(g) * 16 + c];
        // range list (every thread of the group derives the same values; thread 0 writes the scalars)
        int32_t* so = sent_off + size_t(g) * (max_sent + 1);
        const int S0 = n_sent[g];
        if (S0 < 0 || S0 > max_sent) {
            if (c == 0) atomicOr(status, SKIPKV_STATUS_BAD_TABLE);
            return;
        }
        int S = S0;
        if (S0 == 0 || new_sent[b]) {
            if (S0 < max_sent) S = S0 + 1;
            else if (c == 0) atomicOr(status, SKIPKV_STATUS_BAD_TABLE);      // table full: the token joins the last sentence
        }
        __syncwarp();
        if (c == 0) {
            kv_len[g] = len + 1;
            if (S != S0) {
                if (S0 == 0) so[0] = 0;
                sent_id[size_t(g) * max_sent + S0] = gen_id[b];
                n_sent[g] = S;
            }
        }
        for (int i = S + c; i <= max_sent; i += 16) so[i] = len + 1;       // the open sentence ends at the newest token;
                                                                          // entries above n_sent mirror the length
    } else if (q_win != nullptr && g < batch * Hk + batch * Hq) {
        const int bq = g - batch * Hk;                           // (b, q) flattened: q_win is [batch][Hq][window][128]
        q_win[(size_t(bq) * window + slot) * 16 + c] = q[size_t(bq) * 16 + c];
    }
}

}  // namespace skipkv

using namespace skipkv;

extern "C" int skipkv_steer(int32_t batch, int32_t d_model, void* hidden, const void* steer_vec,
                            const float* alpha, const uint8_t* flag, void* stream) {
    if (batch <= 0 || d_model <= 0 || !hidden || !steer_vec || !alpha || !flag) return SKIPKV_ERR_INVALID_ARG;
    if (d_model % 8 != 0) return SKIPKV_ERR_UNSUPPORTED;
    const int total = batch * (d_model / 8);
    const int threads = 256;
    const int blocks = (total + threads - 1) / threads;
    steer_kernel<<<blocks, threads, 0, static_cast<cudaStream_t>(stream)>>>(
        batch, d_model, static_cast<__nv_bfloat16*>(hidden), static_cast<const __nv_bfloat16*>(steer_vec), alpha,
        flag);
    SKIPKV_CUDA(cudaGetLastError());
    return SKIPKV_OK;
}

extern "C" int skipkv_append(const skipkv_shape* shape, void* K, void* V, const void* k_new, const void* v_new,
                             int32_t* kv_len, void* ws, void* stream) {
    if (int rc = check_shape(shape)) return rc;
    if (!K || !V || !k_new || !v_new || !kv_len) return SKIPKV_ERR_INVALID_ARG;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255)) return SKIPKV_ERR_WORKSPACE;
    const int groups = shape->batch * shape->n_kv_heads;
    const int threads = 128;
    const int blocks = (groups * 16 + threads - 1) / threads;
    append_kernel<<<blocks, threads, 0, static_cast<cudaStream_t>(stream)>>>(
        shape->batch, shape->n_kv_heads, shape->slab_off, shape->cap, static_cast<uint4*>(K),
        static_cast<uint4*>(V), static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new), kv_len,
        &static_cast<Header*>(ws)->status);
    SKIPKV_CUDA(cudaGetLastError());
    return SKIPKV_OK;
}

extern "C" int skipkv_append_step(const skipkv_shape* shape, void* K, void* V, const void* k_new, const void* v_new,
                                  int32_t* kv_len, int32_t* sent_off, int32_t* sent_id, int32_t* n_sent,
                                  const uint8_t* new_sent, const int32_t* gen_id, void* q_win, const void* q,
                                  int32_t slot, void* ws, void* stream) {
    if (int rc = check_shape(shape)) return rc;
    if (!K || !V || !k_new || !v_new || !kv_len || !sent_off || !sent_id || !n_sent || !new_sent || !gen_id)
        return SKIPKV_ERR_INVALID_ARG;
    if ((q_win != nullptr) != (q != nullptr)) return SKIPKV_ERR_INVALID_ARG;
    if (q_win && (slot < 0 || slot >= shape->window)) return SKIPKV_ERR_INVALID_ARG;
    if (shape->max_sent <= 0) return SKIPKV_ERR_INVALID_ARG;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255)) return SKIPKV_ERR_WORKSPACE;
    const int groups = shape->batch * (shape->n_kv_heads + (q_win ? shape->n_q_heads : 0));
    const int threads = 128;
    const int blocks = (groups * 16 + threads - 1) / threads;
    SKIPKV_CUDA(launch_dependent(append_step_kernel, dim3(blocks), dim3(threads), 0, static_cast<cudaStream_t>(stream),
                                 int(shape->batch), int(shape->n_kv_heads), int(shape->n_q_heads), int(shape->window),
                                 int(shape->max_sent), shape->slab_off, shape->cap, static_cast<uint4*>(K),
                                 static_cast<uint4*>(V), static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new),
                                 kv_len, sent_off, sent_id, n_sent, new_sent, gen_id, static_cast<uint4*>(q_win),
                                 static_cast<const uint4*>(q), int(slot), &static_cast<Header*>(ws)->status));
    return SKIPKV_OK;
}
