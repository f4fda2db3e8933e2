// Fused trailing hops of tensorized attention on sm_100a (Algorithm 1, several iterations of
// its loop in one pass), bf16 storage, head dim 64 or 128.
//
// When the last dimensions i0..m-1 of the token tensor together span at most 128 tokens, a
// contiguous block of prod(dims[i0..]) rows is closed under the hops of all those dimensions:
// every mode-i vector of such a hop lies inside one block.  A 128-row tile then holds whole
// blocks, and the hops i0, i0+1, .., m-1 run back to back on the tile without leaving the SM:
//
//     S = Q K^T                                   once (all these hops use the same Q and K)
//     for each fused hop f:  P_f = softmax(S masked to the row's mode-f vector),  X <- P_f X
//
// with X updated in place in shared memory (bf16, exactly the rounding an unfused run applies
// when it writes the value tensor to global memory between hops; the two differ only in the
// order of the fp32 sums over a row's keys).
// Q, K and the value tile are read once and the result is written once for all fused hops.
// The rows a row attends to in hop f are not a contiguous range of the tile, so each row keeps
// one 128-bit visibility mask per fused hop in shared memory.
//
// One CTA of 128 threads per SM, persistent; the loads of the next tile are issued before the
// current one is processed (two stages of Q, K, X).  S, P (bf16, A operand of the value MMA) and
// O live in tensor memory.  Every wait is bounded; on expiry the CTA records an error word,
// stops issuing work, lets its copies land, frees its TMEM and returns.
#include <cuda_bf16.h>

#include "ta_internal.h"
#include "ta_ptx.cuh"

namespace ta {
namespace {

constexpr int kTileRows = 128;
constexpr int kThreads = 128;

struct FusedArgs {
    int block, rows, co, causal, g, H, H_kv, xin_is_kv, nf;
    int sub_n[TA_MAX_DIMS], sub_stride[TA_MAX_DIMS];
    long long tiles_outer, total_tiles;
    float scale_log2;
};

template <int D>
struct FusedCfg {
    static constexpr int kHalves = D / 64;
    static constexpr uint32_t kSlabBytes = kTileRows * 128;
    static constexpr uint32_t kTileBytes = kHalves * kSlabBytes;
    static constexpr uint32_t kStageBytes = 3 * kTileBytes;                 // Q, K, X
    static constexpr uint32_t kOffMask = 2 * kStageBytes;                   // [nf][128 rows][4 words]
    static constexpr uint32_t kMaskBytes = TA_MAX_DIMS * kTileRows * 16;
    static constexpr uint32_t kOffBar = kOffMask + kMaskBytes;
    static constexpr uint32_t kSmemBytes = kOffBar + 4 * 8 + 16 + 1024;
    static constexpr uint32_t kTmemCols = 512;
    static constexpr uint32_t kColS = 0, kColP = 128, kColO = 256;
};

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
hop_fused_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_xin, const __grid_constant__ CUtensorMap map_xout,
                 const FusedArgs a) {
    using C = FusedCfg<D>;
    constexpr int kHalves = C::kHalves;
    constexpr uint32_t kSlabBytes = C::kSlabBytes, kTileBytes = C::kTileBytes;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t s0 = smem_u32(smem);
    auto sQ = [&](int s) { return s0 + (uint32_t)s * C::kStageBytes; };
    auto sK = [&](int s) { return s0 + (uint32_t)s * C::kStageBytes + kTileBytes; };
    auto sX = [&](int s) { return s0 + (uint32_t)s * C::kStageBytes + 2 * kTileBytes; };
    uint32_t *masks = (uint32_t *)(smem + C::kOffMask);
    const uint32_t bar0 = s0 + C::kOffBar;
    auto full = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    const uint32_t bar_s = bar0 + 16, bar_o = bar0 + 24;
    uint32_t *tmem_slot = (uint32_t *)(smem + C::kOffBar + 32);

    const int tid = threadIdx.x, warp = tid >> 5;

    // ---- one-time setup: zero the operand stages (rows a box never fills must stay finite),
    // barriers, tensor memory, and the visibility masks of this thread's row
    for (uint32_t i = tid; i < C::kOffBar / 16; i += kThreads) ((uint4 *)smem)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) {
        for (int i = 0; i < 4; ++i) mbar_init(bar0 + 8u * (uint32_t)i, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const int r = tid;                                // this thread's tile row = TMEM lane
    const bool row_valid = r < a.rows;
    const int blk = r / a.block, rr = r % a.block;
    if (row_valid) {
        for (int f = 0; f < a.nf; ++f) {
            // the mode-f vector through row rr: same block, every coordinate but the f-th equal
            const int st = a.sub_stride[f], n = a.sub_n[f];
            const int coord = (rr / st) % n;
            const int first = blk * a.block + rr - coord * st;
            const int last = a.causal ? coord : n - 1;
            uint32_t w[4] = {0u, 0u, 0u, 0u};
            for (int u = 0; u <= last; ++u) {
                const int col = first + u * st;
                w[col >> 5] |= 1u << (col & 31);
            }
            uint32_t *m = masks + ((size_t)f * kTileRows + r) * 4;
            m[0] = w[0]; m[1] = w[1]; m[2] = w[2]; m[3] = w[3];
        }
    }
    fence_proxy_async_smem();
    if (warp == 0) {
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(C::kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_lane = tmem_base + ((uint32_t)(warp * 32) << 16);

    constexpr uint32_t idesc_s = instr_desc(128, 0);
    constexpr uint32_t idesc_o = instr_desc(D, 1);
    // columns any row of this warp can see: the blocks its 32 rows belong to (causal: up to the row)
    const int w_lo = ((warp * 32) / a.block) * a.block;
    int w_hi = min(a.rows, ((warp * 32 + 31) / a.block + 1) * a.block);
    if (a.causal) w_hi = min(w_hi, warp * 32 + 32);
    const bool warp_valid = warp * 32 < a.rows;
    const int nchunks = (a.rows + 31) >> 5;
    const int kblocks = (a.rows + 15) >> 4;
    const uint32_t slab_tx = (uint32_t)a.rows * 128u;

    auto issue_loads = [&](long long tile, int s) {
        long long rest = tile;
        const int hg = (int)(rest % a.g); rest /= a.g;
        const int c_outer = (int)(rest % a.tiles_outer) * a.co; rest /= a.tiles_outer;
        const int kv_head = (int)rest;
        const int q_head = (kv_head / a.H_kv) * a.H + (kv_head % a.H_kv) * a.g + hg;
        const int x_head = a.xin_is_kv ? kv_head : q_head;
        mbar_expect_tx(full(s), 3 * kHalves * slab_tx);
#pragma unroll
        for (int h = 0; h < kHalves; ++h) tma_load_5d(sQ(s) + h * kSlabBytes, &map_q, full(s), 64 * h, 0, 0, c_outer, q_head);
#pragma unroll
        for (int h = 0; h < kHalves; ++h) tma_load_5d(sK(s) + h * kSlabBytes, &map_k, full(s), 64 * h, 0, 0, c_outer, kv_head);
#pragma unroll
        for (int h = 0; h < kHalves; ++h) tma_load_5d(sX(s) + h * kSlabBytes, &map_xin, full(s), 64 * h, 0, 0, c_outer, x_head);
    };

    bool ok = true;
    bool prefetched = false;                          // thread 0: a load is in flight into the other stage
    uint32_t it = 0, uses_o = 0;
    if (tid == 0 && (long long)blockIdx.x < a.total_tiles) issue_loads(blockIdx.x, 0);
    for (long long tile = blockIdx.x; tile < a.total_tiles; tile += gridDim.x, ++it) {
        const int s = it & 1;
        long long rest = tile;
        const int hg = (int)(rest % a.g); rest /= a.g;
        const int c_outer = (int)(rest % a.tiles_outer) * a.co; rest /= a.tiles_outer;
        const int kv_head = (int)rest;
        const int q_head = (kv_head / a.H_kv) * a.H + (kv_head % a.H_kv) * a.g + hg;

        if (tid == 0) {
            // the other stage was read out by the store of the previous tile (waited for below)
            prefetched = tile + gridDim.x < a.total_tiles;
            if (prefetched) issue_loads(tile + gridDim.x, s ^ 1);
            ok = mbar_wait(full(s), (it >> 1) & 1, 0x81);
            if (ok) {
                tc_fence_after();
#pragma unroll
                for (int kb = 0; kb < D / 16; ++kb) {
                    const uint32_t off = (kb >> 2) * kSlabBytes + (kb & 3) * 32;
                    tc_mma_ss(tmem_base + C::kColS, smem_desc_sw128(sQ(s) + off, 16, 1024),
                              smem_desc_sw128(sK(s) + off, 16, 1024), idesc_s, kb > 0);
                }
                tc_commit(bar_s);
            }
        }
        __syncwarp();
        if (ok) ok = mbar_wait(bar_s, it & 1, 0x82);
        ok = __syncthreads_and(ok ? 1 : 0) != 0;
        if (!ok) break;
        tc_fence_after();

        for (int f = 0; f < a.nf; ++f, ++uses_o) {
            // ---- softmax of this row over its mode-f vector; P (un-normalised, bf16) -> tensor memory
            const uint32_t *mword = masks + ((size_t)f * kTileRows + r) * 4;   // this row's visibility bits
            float m = -INFINITY;
            uint32_t v[32];
#pragma unroll 1
            for (int c = 0; c < nchunks; ++c) {
                if (!(warp_valid && 32 * c < w_hi && 32 * c + 32 > w_lo)) continue;   // warp-uniform
                tmem_ld32(tmem_lane + C::kColS + 32 * c, v);
                const uint32_t bits = mword[c];
#pragma unroll
                for (int jj = 0; jj < 32; ++jj)
                    if ((bits >> jj) & 1u) m = fmaxf(m, __uint_as_float(v[jj]));
            }
            const float m_scaled = row_valid ? m * a.scale_log2 : 0.f;
            float sum = 0.f;
#pragma unroll 1
            for (int c = 0; c < nchunks; ++c) {
                uint32_t pk[16];
                if (warp_valid && 32 * c < w_hi && 32 * c + 32 > w_lo) {
                    tmem_ld32(tmem_lane + C::kColS + 32 * c, v);
                    const uint32_t bits = mword[c];
#pragma unroll
                    for (int jj = 0; jj < 32; jj += 2) {
                        float p0 = fast_exp2(__uint_as_float(v[jj]) * a.scale_log2 - m_scaled);
                        float p1 = fast_exp2(__uint_as_float(v[jj + 1]) * a.scale_log2 - m_scaled);
                        p0 = ((bits >> jj) & 1u) ? p0 : 0.f;
                        p1 = ((bits >> (jj + 1)) & 1u) ? p1 : 0.f;
                        const uint32_t w = pack_bf16x2(p0, p1);
                        pk[jj >> 1] = w;
                        sum += __uint_as_float(w << 16) + __uint_as_float(w & 0xFFFF0000u);
                    }
                } else {
#pragma unroll
                    for (int jj = 0; jj < 16; ++jj) pk[jj] = 0u;
                }
                tmem_st16(tmem_lane + C::kColP + 16 * c, pk);
            }
            tmem_st_wait();
            const float inv = row_valid ? 1.f / sum : 1.f;
            tc_fence_before();
            __syncthreads();

            // ---- X <- P X
            if (tid == 0) {
                tc_fence_after();
                for (int kb = 0; kb < kblocks; ++kb)
                    tc_mma_ts(tmem_base + C::kColO, tmem_base + C::kColP + kb * 8,
                              smem_desc_sw128(sX(s) + kb * 2048, kSlabBytes, 1024), idesc_o, kb > 0);
                tc_commit(bar_o);
            }
            __syncwarp();
            ok = mbar_wait(bar_o, uses_o & 1, 0x83);
            ok = __syncthreads_and(ok ? 1 : 0) != 0;
            if (!ok) break;
            tc_fence_after();
            if (warp_valid) {
                const uint32_t x_row = sX(s) + (uint32_t)r * 128u;
#pragma unroll 1
                for (int c = 0; c < D / 32; ++c) {
                    tmem_ld32(tmem_lane + C::kColO + 32 * c, v);
                    uint32_t pk[16];
#pragma unroll
                    for (int jj = 0; jj < 32; jj += 2)
                        pk[jj >> 1] = pack_bf16x2(__uint_as_float(v[jj]) * inv, __uint_as_float(v[jj + 1]) * inv);
                    if (row_valid) {
                        const uint32_t slab = x_row + (uint32_t)(c >> 1) * kSlabBytes;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const uint32_t chunk = (uint32_t)(((c & 1) * 4 + i) ^ (r & 7));
                            st_shared_v4(slab + chunk * 16, pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
                        }
                    }
                }
            }
            fence_proxy_async_smem();     // the next MMA (or the store) reads X through the async proxy
            tc_fence_before();
            __syncthreads();
        }
        if (!ok) break;
        if (tid == 0) {
#pragma unroll
            for (int h = 0; h < kHalves; ++h) tma_store_5d(&map_xout, sX(s) + h * kSlabBytes, 64 * h, 0, 0, c_outer, q_head);
            tma_store_commit_and_wait_read();
            prefetched = false;           // (re-evaluated at the top of the next iteration)
        }
    }
    if (tid == 0) {
        if (!ok && prefetched) {
            // leaving early: let the load in flight land before shared memory is released
            const unsigned long long t0 = globaltimer_ns();
            while (!mbar_try_wait(full((it & 1) ^ 1), ((it + 1) >> 1) & 1) && globaltimer_ns() - t0 < 10000000ull) {
            }
        }
        tma_store_wait_all();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::kTmemCols) : "memory");
    }
}

template <int D>
int launch_fused_d(const Problem &pb, const HopDesc &hd, const void *xin, int xin_heads, void *xout) {
    CUtensorMap mq, mk, mxi, mxo;
    int rc;
    if ((rc = make_hop_map(&mq, pb.q, pb.B * pb.H, pb.N, D, hd, 2)) != TA_OK) return rc;
    if ((rc = make_hop_map(&mk, pb.k, pb.B * pb.H_kv, pb.N, D, hd, 2)) != TA_OK) return rc;
    if ((rc = make_hop_map(&mxi, xin, pb.B * xin_heads, pb.N, D, hd, 2)) != TA_OK) return rc;
    if ((rc = make_hop_map(&mxo, xout, pb.B * pb.H, pb.N, D, hd, 2)) != TA_OK) return rc;

    FusedArgs a;
    a.block = hd.n; a.rows = hd.rows; a.co = hd.co; a.causal = pb.causal;
    a.g = pb.H / pb.H_kv; a.H = pb.H; a.H_kv = pb.H_kv; a.xin_is_kv = xin_heads != pb.H ? 1 : 0;
    a.nf = hd.nf;
    for (int f = 0; f < TA_MAX_DIMS; ++f) {
        a.sub_n[f] = f < hd.nf ? hd.sub_n[f] : 1;
        a.sub_stride[f] = f < hd.nf ? hd.sub_stride[f] : 1;
    }
    a.tiles_outer = hd.tiles_outer;
    a.total_tiles = (long long)pb.B * pb.H * hd.tiles_outer;
    a.scale_log2 = pb.scale * 1.4426950408889634f;

    static int num_sms = 0;
    if (num_sms == 0) {
        int dev = 0;
        cudaGetDevice(&dev);
        if (cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || num_sms <= 0)
            num_sms = 148;
    }
    constexpr size_t smem = FusedCfg<D>::kSmemBytes;
    auto kern = hop_fused_kernel<D>;
    static bool configured = false;
    if (!configured) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return TA_ERR_CUDA;
        configured = true;
    }
    const unsigned grid = (unsigned)(a.total_tiles < num_sms ? a.total_tiles : num_sms);
    kern<<<grid, kThreads, smem, pb.stream>>>(mq, mk, mxi, mxo, a);
    count_launch();
    return cudaPeekAtLastError() == cudaSuccess ? TA_OK : TA_ERR_CUDA;
}

}  // namespace

int launch_hop_tc_fused(const Problem &pb, const HopDesc &hd, const void *xin, int xin_heads, void *xout) {
    if (hd.stride != 1 || hd.ci != 1 || hd.tiles_inner != 1) return TA_ERR_INVALID_ARG;
    if (pb.D == 128) return launch_fused_d<128>(pb, hd, xin, xin_heads, xout);
    if (pb.D == 64) return launch_fused_d<64>(pb, hd, xin, xin_heads, xout);
    return TA_ERR_UNSUPPORTED;
}

int read_status_tc_fused(unsigned int *word) {
    if (cudaMemcpyFromSymbol(word, g_status_word, sizeof(*word)) != cudaSuccess) return TA_ERR_CUDA;
    if (*word != 0) {
        unsigned int z = 0;
        cudaMemcpyToSymbol(g_status_word, &z, sizeof(z));
    }
    return TA_OK;
}

}  // namespace ta
