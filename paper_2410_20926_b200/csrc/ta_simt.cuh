// Helpers shared by the generic CUDA-core kernels (forward: ta_simt.cu, backward: ta_simt_bwd.cu).
#pragma once

#include <cuda_bf16.h>

namespace ta {
namespace {

// Tensorized positional encoding (Section 3.2): rows of `x` ([rows][ld] fp32 in shared memory)
// sit at positions pos0, pos0 + 1, .. of a segment; feature c is paired with c + D/2 and
// turned by the angle position * base^(-2c/D).
// sign = +1 rotates, -1 rotates back (the transpose, used on gradients).
__device__ __forceinline__ void rope_rows(float *x, int rows, int ld, int D, int pos0, float log2_base,
                                          float sign = 1.f) {
    const int half = D >> 1;
    for (int idx = threadIdx.x; idx < rows * half; idx += blockDim.x) {
        const int r = idx / half, c = idx % half;
        const float theta = exp2f(-2.f * (float)c / (float)D * log2_base);
        float sn, cs;
        sincosf((float)(pos0 + r) * theta, &sn, &cs);
        sn *= sign;
        const float x1 = x[r * ld + c], x2 = x[r * ld + c + half];
        x[r * ld + c] = x1 * cs - x2 * sn;
        x[r * ld + c + half] = x2 * cs + x1 * sn;
    }
}

template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
    for (int o = 16; o; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
    return x;
}
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

}  // namespace
}  // namespace ta
