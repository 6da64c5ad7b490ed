// Device body of the steering add, shared by skipkv_steer and the decode-attention epilogue.
#pragma once
#include "common.cuh"

namespace skipkv {

// Element group i of 8 bf16: hidden[b][8k..8k+7] = bf16_rne(fmaf(alpha[b], v, hidden)) if flag[b].
__device__ __forceinline__ void steer_vec8(int i, int vec_per_row, __nv_bfloat16* hidden, const __nv_bfloat16* v,
                                           const float* alpha, const uint8_t* flag) {
    const int b = i / vec_per_row, k = i % vec_per_row;
    if (!flag[b]) return;
    const float a = alpha[b];
    uint4* hp = reinterpret_cast<uint4*>(hidden) + size_t(b) * vec_per_row + k;
    uint4 h = *hp;
    const uint4 s = reinterpret_cast<const uint4*>(v)[k];
    uint32_t hw[4] = {h.x, h.y, h.z, h.w};
    const uint32_t sw[4] = {s.x, s.y, s.z, s.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const float lo = __fmaf_rn(a, bf16lo(sw[j]), bf16lo(hw[j]));
        const float hi = __fmaf_rn(a, bf16hi(sw[j]), bf16hi(hw[j]));
        const __nv_bfloat162 r = __floats2bfloat162_rn(lo, hi);
        hw[j] = *reinterpret_cast<const uint32_t*>(&r);
    }
    *hp = make_uint4(hw[0], hw[1], hw[2], hw[3]);
}

}  // namespace skipkv
