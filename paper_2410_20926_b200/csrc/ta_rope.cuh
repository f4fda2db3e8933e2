// In-place RoPE of an operand tile in shared memory (tensorized positional encoding, Section
// 3.2: hop i rotates queries and keys by their coordinate along dimension i; feature c is
// paired with c + D/2 and turned by the angle position * base^(-2c/D)).  Shared by the forward
// and the backward tensor-core kernels, whose tiles have the same layout: 128 rows of 128 bytes
// per 64-column slab, 128-byte swizzled, row r at position r mod n of its segment.
//
// 256 threads (two warpgroups) rotate a tile.  A thread owns one 16-byte chunk of features
// (8 adjacent c < D/2, and their partners c + D/2) at the positions t = tsub, tsub + kTStep, ..
// (< n) of EVERY segment of the tile, and the row -> position map is the same in every tile,
// so the cos / sin it needs never change: they sit in registers as fp16 pairs (absolute error
// 2^-12, far below bf16), computed once per launch, and a tile costs one 16-byte load and
// store per 8 features plus the multiply-adds.
#pragma once

#include <cuda_fp16.h>
#include <stdint.h>

#include "ta_ptx.cuh"

namespace ta {
namespace {

template <int D>
struct RopeRotator {
    static constexpr int kChunks = D / 16;            // 16-byte chunks of the first half of a row
    static constexpr int kTStep = 256 / kChunks;      // positions covered by one sweep of the threads
    static constexpr int kMaxPos = 128 / kTStep;      // sweeps to reach n = 128
    static constexpr uint32_t kSlabBytes = 128 * 128;

    int chunk, tsub, n, segs;
    __half2 cs[kMaxPos][8];                           // (cos, sin) of position x frequency

    // rt: index of the thread among the 256 rotating threads; rows = segs * n valid rows per tile
    __device__ __forceinline__ void init(int rt, int n_, int rows, float log2_base) {
        chunk = rt % kChunks;
        tsub = rt / kChunks;                          // 0 .. 31 (D = 128) or 0 .. 63 (D = 64)
        n = n_;
        segs = rows / n_;
#pragma unroll
        for (int pi = 0; pi < kMaxPos; ++pi)
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float ang = (float)(tsub + kTStep * pi) * exp2f(-2.f * (float)(8 * chunk + e) / (float)D * log2_base);
                cs[pi][e] = __floats2half2_rn(__cosf(ang), __sinf(ang));
            }
    }

    // rotates this thread's share of the tile at shared address `tile`, then makes the writes
    // visible to the async proxy (the MMA reads the tile) and reconverges the warp
    __device__ __forceinline__ void rotate(uint32_t tile) const {
#pragma unroll
        for (int pi = 0; pi < kMaxPos; ++pi) {
            const int t = tsub + kTStep * pi;
            if (t >= n) break;
#pragma unroll 2
            for (int sg = 0; sg < segs; ++sg) {
                const int r = sg * n + t;
                const uint32_t row = tile + (uint32_t)r * 128u;
                const uint32_t addr_a = row + (((uint32_t)chunk ^ (uint32_t)(r & 7)) << 4);
                const uint32_t addr_b = D == 128 ? addr_a + kSlabBytes                       // partner: second slab
                                                 : row + (((uint32_t)(chunk + 4) ^ (uint32_t)(r & 7)) << 4);
                uint32_t ua[4], ub[4];
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                             : "=r"(ua[0]), "=r"(ua[1]), "=r"(ua[2]), "=r"(ua[3]) : "r"(addr_a) : "memory");
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                             : "=r"(ub[0]), "=r"(ub[1]), "=r"(ub[2]), "=r"(ub[3]) : "r"(addr_b) : "memory");
#pragma unroll
                for (int e2 = 0; e2 < 4; ++e2) {
                    const float a0 = __uint_as_float(ua[e2] << 16), a1 = __uint_as_float(ua[e2] & 0xFFFF0000u);
                    const float b0 = __uint_as_float(ub[e2] << 16), b1 = __uint_as_float(ub[e2] & 0xFFFF0000u);
                    const float2 f0 = __half22float2(cs[pi][2 * e2]), f1 = __half22float2(cs[pi][2 * e2 + 1]);
                    ua[e2] = pack_bf16x2(a0 * f0.x - b0 * f0.y, a1 * f1.x - b1 * f1.y);
                    ub[e2] = pack_bf16x2(b0 * f0.x + a0 * f0.y, b1 * f1.x + a1 * f1.y);
                }
                st_shared_v4(addr_a, ua[0], ua[1], ua[2], ua[3]);
                st_shared_v4(addr_b, ub[0], ub[1], ub[2], ub[3]);
            }
        }
        fence_proxy_async_smem();
        __syncwarp();
    }
};

}  // namespace
}  // namespace ta
