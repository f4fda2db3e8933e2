// Head dims the tensor-core kernels do not take (bf16, D < 128, D != 64 -- OpenLlama-3B's 100, 80,
// 96, ...): the hops of Algorithm 1 run on zero-padded copies with D' = 64 or 128 columns.  Zero
// columns add nothing to Q K^T (Eq. 4) and give zero output columns, so the hop results are those of
// the unpadded problem; the softmax scale stays 1 / sqrt(D).  Layout of a padded row: the first
// floor(D / 2) columns at 0, the rest at D' / 2 -- the two halves the positional encoding pairs
// (feature c with c + D / 2, Section 3.2) stay paired under D' (c with c + D' / 2); its
// frequencies base^(-2c / D) are kept by running the padded problem with base^(D' / D).
#include <cuda_bf16.h>

#include <cmath>

#include "ta_internal.h"

namespace ta {
namespace {

// source column of padded column `col` (or -1: zero)
__device__ __forceinline__ int source_col(int col, int D, int DP) {
    const int h = D >> 1, half = DP >> 1;
    if (col < half) return col < h ? col : -1;
    return col - half < D - h ? h + col - half : -1;
}

// Fast path, rows and halves made of whole 4-byte units (bf16 with D % 4 == 0, any fp32 row): a warp
// moves four rows at a time, lane l the units l, l + 32, ... of each padded row (at most 128 units);
// all loads of the four rows are issued before the first store.
// U: units per unpadded row, UH: units of its first half, UP: units per padded row.
template <bool kPad>
__global__ void pad_units_kernel(const uint32_t *__restrict__ src, uint32_t *__restrict__ dst, long long rows, int U,
                                 int UH, int UP) {
    const int lane = threadIdx.x & 31;
    const long long warp = (blockIdx.x * (long long)blockDim.x + threadIdx.x) >> 5;
    const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
    const int uph = UP >> 1;
    constexpr int kT = 4;
    int su[kT];
#pragma unroll
    for (int t = 0; t < kT; ++t) {
        const int u = lane + 32 * t;
        su[t] = u >= UP ? -2 : (u < uph ? (u < UH ? u : -1) : (u - uph < U - UH ? UH + u - uph : -1));
    }
    for (long long row0 = warp * 4; row0 < rows; row0 += nwarps * 4) {
        uint32_t val[4][kT];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int t = 0; t < kT; ++t) {
                val[r][t] = 0u;
                if (row0 + r < rows && su[t] >= 0)
                    val[r][t] = kPad ? __ldg(src + (row0 + r) * U + su[t]) : __ldg(src + (row0 + r) * UP + lane + 32 * t);
            }
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int t = 0; t < kT; ++t) {
                if (row0 + r >= rows) continue;
                if (kPad) {
                    if (su[t] >= -1) dst[(row0 + r) * UP + lane + 32 * t] = val[r][t];
                } else if (su[t] >= 0) {
                    dst[(row0 + r) * U + su[t]] = val[r][t];
                }
            }
    }
}

// Any other row length: element by element.
template <typename T>
__global__ void pad_rows_kernel(const T *__restrict__ src, T *__restrict__ dst, long long rows, int D, int DP) {
    const long long total = rows * DP;
    for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const long long row = idx / DP;
        const int sc = source_col((int)(idx % DP), D, DP);
        dst[idx] = sc >= 0 ? src[row * D + sc] : T(0);
    }
}

template <typename T>
__global__ void unpad_rows_kernel(const T *__restrict__ src, T *__restrict__ dst, long long rows, int D, int DP) {
    const int h = D >> 1, half = DP >> 1;
    const long long total = rows * D;
    for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const long long row = idx / D;
        const int c = (int)(idx % D);
        dst[idx] = src[row * DP + (c < h ? c : half + c - h)];
    }
}

unsigned blocks_for(long long threads) {
    const long long b = (threads + 255) / 256;
    const long long cap = 32ll * current_device_sms(nullptr);
    return (unsigned)(b < 1 ? 1 : (b < cap ? b : cap));
}

}  // namespace

bool pad_eligible(int D, int dtype, unsigned flags) {
    return dtype == TA_DTYPE_BF16 && D >= 1 && D < 128 && D != 64 && !(flags & TA_FLAG_NO_TENSOR_CORE);
}
int padded_dim(int D) { return D <= 64 ? 64 : 128; }
float padded_rope_base(float base, int D, int DP) {
    const double b = pow((double)base, (double)DP / (double)D);
    return b < 1e30 ? (float)b : 0.f;
}

namespace {
template <bool kPad>
int launch_pad_any(const void *src, void *dst, long long rows, int D, int DP, int elem, cudaStream_t stream) {
    if (rows <= 0) return TA_OK;
    const bool units = elem == 4 || (D % 4) == 0;      // rows and their halves are whole 4-byte units
    const bool aligned = ((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 3u) == 0;
    if (units && aligned) {
        const int per = 4 / elem;                       // elements per unit
        const unsigned grid = blocks_for((rows + 3) / 4 * 32);
        return launch_kernel(pad_units_kernel<kPad>, grid, 256, 0, stream, false, (const uint32_t *)src, (uint32_t *)dst,
                             rows, D / per, (D / 2) / per, DP / per);
    }
    const unsigned grid = blocks_for(rows * (kPad ? DP : D));
    if (elem == 2) {
        if (kPad)
            return launch_kernel(pad_rows_kernel<unsigned short>, grid, 256, 0, stream, false, (const unsigned short *)src,
                                 (unsigned short *)dst, rows, D, DP);
        return launch_kernel(unpad_rows_kernel<unsigned short>, grid, 256, 0, stream, false, (const unsigned short *)src,
                             (unsigned short *)dst, rows, D, DP);
    }
    if (kPad)
        return launch_kernel(pad_rows_kernel<unsigned int>, grid, 256, 0, stream, false, (const unsigned int *)src,
                             (unsigned int *)dst, rows, D, DP);
    return launch_kernel(unpad_rows_kernel<unsigned int>, grid, 256, 0, stream, false, (const unsigned int *)src,
                         (unsigned int *)dst, rows, D, DP);
}
}  // namespace

int launch_pad_rows(const void *src, void *dst, long long rows, int D, int DP, int elem, cudaStream_t stream) {
    return launch_pad_any<true>(src, dst, rows, D, DP, elem, stream);
}
int launch_unpad_rows(const void *src, void *dst, long long rows, int D, int DP, int elem, cudaStream_t stream) {
    return launch_pad_any<false>(src, dst, rows, D, DP, elem, stream);
}

}  // namespace ta
