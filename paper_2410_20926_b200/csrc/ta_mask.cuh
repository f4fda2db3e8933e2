// Explicit per-hop masks inside the tensor-core kernels (Eq. 3 allows any mask M_i): the host
// combines the caller's n x n mask with the causal flag and the window into a HopMask (bit u of
// row t: key position u is visible from query position t) and passes it by value as a kernel
// parameter.  A thread that owns tile row r (position t = r mod n of segment r / n) turns its
// row of the mask into a 128-bit mask over the TILE's key columns -- the n bits shifted to the
// segment's columns -- and keeps it in four registers.
#pragma once

#include <stdint.h>

#include "ta_internal.h"

namespace ta {
namespace {

struct NoMask {};
template <bool kMask> struct MaskArg { using type = NoMask; };
template <> struct MaskArg<true> { using type = HopMask; };

// w[0..3] <- (the 128 bits in[0..3]) << seg_offset, as a 128-bit value (little-endian words)
__device__ __forceinline__ void shift_row_mask(const uint32_t (&in)[4], int seg_offset, uint32_t (&w)[4]) {
    const int k = seg_offset >> 5, lo = seg_offset & 31;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        uint32_t x = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (j == i - k) x |= in[j] << lo;
            if (lo != 0 && j == i - k - 1) x |= in[j] >> (32 - lo);
        }
        w[i] = x;
    }
}
// w[0..3] <- (bits of row t of hm) << seg_offset
__device__ __forceinline__ void tile_row_mask(const HopMask &hm, int t, int seg_offset, uint32_t (&w)[4]) {
    const uint32_t in[4] = {hm.bits[t][0], hm.bits[t][1], hm.bits[t][2], hm.bits[t][3]};
    shift_row_mask(in, seg_offset, w);
}
// the same from a bit matrix in device memory (n <= 128: four words per row); `rows` points at the
// matrix of the tile's query head
__device__ __forceinline__ void tile_row_mask(const uint32_t *rows, int t, int seg_offset, uint32_t (&w)[4]) {
    const uint4 v = __ldg(reinterpret_cast<const uint4 *>(rows + 4 * (size_t)t));
    const uint32_t in[4] = {v.x, v.y, v.z, v.w};
    shift_row_mask(in, seg_offset, w);
}
__device__ __forceinline__ void tile_row_mask(const NoMask &, int, int, uint32_t (&w)[4]) {
    w[0] = w[1] = w[2] = w[3] = 0u;
}
// the 32 bits of chunk c (c = 0..3) of such a mask
__device__ __forceinline__ uint32_t mask_chunk(const uint32_t (&w)[4], int c) {
    return c == 0 ? w[0] : (c == 1 ? w[1] : (c == 2 ? w[2] : w[3]));
}

}  // namespace
}  // namespace ta
