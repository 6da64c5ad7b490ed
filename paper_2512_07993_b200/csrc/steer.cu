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
