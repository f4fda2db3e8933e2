// Tensor-core backward kernel for one hop of tensorized attention on sm_100a (bf16 storage,
// head dim 64 or 128, n_i <= 128).  The paper gives no backward formula; this is the chain rule
// through one hop of Algorithm 1, X_{i+1} = A_i X_i with A_i = softmax(Q K^T * scale o M_i):
//
//     P   = A_i                                  (recomputed from Q, K)
//     dP  = G_{i+1} X_i^T
//     dS  = P o (dP - rowsum(P o dP)) * scale
//     G_i = P^T G_{i+1}          dQ += dS K          dK += dS^T Q
//
// Tiles, strided TMA maps and the block-diagonal packing of short segments are those of the
// forward kernel.  Per tile: two MMAs into TMEM (S = Q K^T, dP = G X^T), the softmax and its
// derivative in registers, P and dS (bf16) to shared memory, then three MMAs: G_i (A = P as an
// MN-major operand, i.e. P^T), dQ (A = dS K-major) and dK (A = dS MN-major).  dQ / dK / dV are
// accumulated in fp32 global buffers by TMA reduce-add (they sum over hops and, for dK / dV,
// over the query heads of a GQA group); G_i is carried to the next hop as bf16, in place.
#include <cuda_bf16.h>

#include "ta_internal.h"
#include "ta_ptx.cuh"

namespace ta {
namespace {

constexpr int kTileRows = 128;
constexpr int kThreads = 128;

struct BwdArgs {
    int n, rows, ci, co, causal, g, H, H_kv, x_is_kv, first_hop;
    long long tiles_inner, tiles_outer, total_tiles;
    float scale_log2, scale;
};

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

template <int D>
__global__ void __launch_bounds__(kThreads)
hop_tc_bwd_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_gin,
                  const __grid_constant__ CUtensorMap map_gout, const __grid_constant__ CUtensorMap map_dq,
                  const __grid_constant__ CUtensorMap map_dk, const __grid_constant__ CUtensorMap map_dv,
                  const BwdArgs a) {
    constexpr int kHalves = D / 64;
    constexpr uint32_t kSlabBytes = kTileRows * 128;          // [128 rows][128 bytes]
    constexpr uint32_t kTileBytes = kHalves * kSlabBytes;     // one bf16 input tile
    constexpr uint32_t kPBytes = 2 * kSlabBytes;              // 128 x 128 bf16
    constexpr uint32_t kStageBytes = 2 * kTileBytes;          // one fp32 output tile
    constexpr uint32_t kTmemCols = 512;
    constexpr uint32_t kColS = 0, kColDP = 128, kColG = 256, kColDQ = 384, kColDK = 0;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t s0 = smem_u32(smem);
    const uint32_t sQ = s0, sK = sQ + kTileBytes, sX = sK + kTileBytes, sG = sX + kTileBytes;
    const uint32_t sP = sG + kTileBytes, sdS = sP + kPBytes;
    constexpr uint32_t kDataBytes = 4 * kTileBytes + 2 * kPBytes;
    // output staging after all MMAs have completed (every input is dead by then)
    const uint32_t stDQ = s0, stDK = s0 + kStageBytes, stG = s0 + 2 * kStageBytes;
    uint64_t *bars = (uint64_t *)(smem + kDataBytes);
    const uint32_t bar_qk = smem_u32(bars + 0), bar_gx = smem_u32(bars + 1), bar_s = smem_u32(bars + 2),
                   bar_o = smem_u32(bars + 3);
    uint32_t *tmem_slot = (uint32_t *)(bars + 4);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    for (uint32_t i = tid; i < kDataBytes / 16; i += kThreads) ((uint4 *)smem)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) {
        mbar_init(bar_qk, 1);
        mbar_init(bar_gx, 1);
        mbar_init(bar_s, 1);
        mbar_init(bar_o, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    fence_proxy_async_smem();
    if (warp == 0) {
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_lane = tmem_base + ((uint32_t)(warp * 32) << 16);

    constexpr uint32_t idesc_s = instr_desc(128, 0, 0);        // A, B K-major, N = 128
    constexpr uint32_t idesc_g = instr_desc(D, 1, 1);          // A = P^T / dS^T (MN-major), B MN-major
    constexpr uint32_t idesc_dq = instr_desc(D, 1, 0);         // A = dS K-major, B MN-major

    const int r = warp * 32 + lane;
    const int seg = r / a.n;
    const bool row_valid = r < a.rows;
    const int c_lo = seg * a.n;
    const int c_hi = a.causal ? r + 1 : c_lo + a.n;
    const int w_lo = ((warp * 32) / a.n) * a.n;
    int w_hi = min(a.rows, ((warp * 32 + 31) / a.n + 1) * a.n);
    if (a.causal) w_hi = min(w_hi, warp * 32 + 32);
    const bool warp_valid = warp * 32 < a.rows;

    bool ok = true;
    uint32_t it = 0;
    for (long long tile = blockIdx.x; tile < a.total_tiles; tile += gridDim.x, ++it) {
        const uint32_t parity = it & 1u;
        long long rest = tile;
        const int hg = (int)(rest % a.g); rest /= a.g;
        const int c_inner = (int)(rest % a.tiles_inner) * a.ci; rest /= a.tiles_inner;
        const int c_outer = (int)(rest % a.tiles_outer) * a.co; rest /= a.tiles_outer;
        const int kv_head = (int)rest;
        const int q_head = (kv_head / a.H_kv) * a.H + (kv_head % a.H_kv) * a.g + hg;
        const int x_head = a.x_is_kv ? kv_head : q_head;

        if (tid == 0) {
            const uint32_t slab_tx = (uint32_t)a.rows * 128u;
            mbar_expect_tx(bar_qk, 2 * kHalves * slab_tx);
#pragma unroll
            for (int h = 0; h < kHalves; ++h) tma_load_5d(sQ + h * kSlabBytes, &map_q, bar_qk, 64 * h, 0, c_inner, c_outer, q_head);
#pragma unroll
            for (int h = 0; h < kHalves; ++h) tma_load_5d(sK + h * kSlabBytes, &map_k, bar_qk, 64 * h, 0, c_inner, c_outer, kv_head);
            mbar_expect_tx(bar_gx, 2 * kHalves * slab_tx);
#pragma unroll
            for (int h = 0; h < kHalves; ++h) tma_load_5d(sG + h * kSlabBytes, &map_gin, bar_gx, 64 * h, 0, c_inner, c_outer, q_head);
#pragma unroll
            for (int h = 0; h < kHalves; ++h) tma_load_5d(sX + h * kSlabBytes, &map_x, bar_gx, 64 * h, 0, c_inner, c_outer, x_head);

            ok = mbar_wait(bar_qk, parity, 0x11);
            if (ok) {
                tc_fence_after();
#pragma unroll
                for (int kb = 0; kb < D / 16; ++kb) {
                    const uint32_t off = (kb >> 2) * kSlabBytes + (kb & 3) * 32;
                    tc_mma_ss(tmem_base + kColS, smem_desc_sw128(sQ + off, 16, 1024),
                              smem_desc_sw128(sK + off, 16, 1024), idesc_s, kb > 0);
                }
                ok = mbar_wait(bar_gx, parity, 0x12);
            }
            if (ok) {
#pragma unroll
                for (int kb = 0; kb < D / 16; ++kb) {
                    const uint32_t off = (kb >> 2) * kSlabBytes + (kb & 3) * 32;
                    tc_mma_ss(tmem_base + kColDP, smem_desc_sw128(sG + off, 16, 1024),
                              smem_desc_sw128(sX + off, 16, 1024), idesc_s, kb > 0);
                }
                tc_commit(bar_s);
            }
        }
        __syncwarp();
        if (ok) ok = mbar_wait(bar_s, parity, 0x13);
        ok = __all_sync(0xffffffffu, ok);
        tc_fence_after();

        // ---- softmax and its derivative for this thread's row
        if (ok) {
            uint32_t vs[32], vd[32];
            float m = -INFINITY;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                if (!(warp_valid && 32 * c < w_hi && 32 * c + 32 > w_lo)) continue;
                tmem_ld32(tmem_lane + kColS + 32 * c, vs);
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const int col = 32 * c + j;
                    if (col >= c_lo && col < c_hi) m = fmaxf(m, __uint_as_float(vs[j]));
                }
            }
            const float m_s = row_valid ? m * a.scale_log2 : 0.f;
            float l = 0.f, dot = 0.f;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                if (!(warp_valid && 32 * c < w_hi && 32 * c + 32 > w_lo)) continue;
                tmem_ld32(tmem_lane + kColS + 32 * c, vs);
                tmem_ld32(tmem_lane + kColDP + 32 * c, vd);
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const int col = 32 * c + j;
                    float p = fast_exp2(__uint_as_float(vs[j]) * a.scale_log2 - m_s);
                    const bool vis = row_valid && col >= c_lo && col < c_hi;
                    p = vis ? p : 0.f;
                    l += p;
                    dot += vis ? p * __uint_as_float(vd[j]) : 0.f;
                }
            }
            const float inv_l = row_valid ? 1.f / l : 0.f;
            const float delta = dot * inv_l;
            const uint32_t rowP = sP + (uint32_t)r * 128u, rowS = sdS + (uint32_t)r * 128u;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                uint32_t pp[16], ps[16];
                if (warp_valid && 32 * c < w_hi && 32 * c + 32 > w_lo) {
                    tmem_ld32(tmem_lane + kColS + 32 * c, vs);
                    tmem_ld32(tmem_lane + kColDP + 32 * c, vd);
#pragma unroll
                    for (int j = 0; j < 32; j += 2) {
                        float pv[2], dv[2];
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int col = 32 * c + j + e;
                            const bool vis = row_valid && col >= c_lo && col < c_hi;
                            float p = fast_exp2(__uint_as_float(vs[j + e]) * a.scale_log2 - m_s) * inv_l;
                            p = vis ? p : 0.f;
                            pv[e] = p;
                            dv[e] = vis ? p * (__uint_as_float(vd[j + e]) - delta) * a.scale : 0.f;
                        }
                        pp[j >> 1] = pack_bf16x2(pv[0], pv[1]);
                        ps[j >> 1] = pack_bf16x2(dv[0], dv[1]);
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 16; ++j) { pp[j] = 0u; ps[j] = 0u; }
                }
                const uint32_t slab = (uint32_t)(c >> 1) * kSlabBytes;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t chunk = (uint32_t)(((c & 1) * 4 + i) ^ (r & 7)) * 16;
                    st_shared_v4(rowP + slab + chunk, pp[4 * i], pp[4 * i + 1], pp[4 * i + 2], pp[4 * i + 3]);
                    st_shared_v4(rowS + slab + chunk, ps[4 * i], ps[4 * i + 1], ps[4 * i + 2], ps[4 * i + 3]);
                }
            }
        }
        fence_proxy_async_smem();
        tc_fence_before();
        __syncthreads();

        if (tid == 0 && ok) {
            tc_fence_after();
            const int kblocks = (a.rows + 15) >> 4;
            for (int kb = 0; kb < kblocks; ++kb) {
                const uint32_t k_off = kb * 2048;                                  // 16 rows of 128 bytes
                const uint32_t a_off = (kb >> 2) * kSlabBytes + (kb & 3) * 32;     // 16 columns of a K-major tile
                // G_i[key, d] = sum_q P[q, key] G[q, d]
                tc_mma_ss(tmem_base + kColG, smem_desc_sw128(sP + k_off, kSlabBytes, 1024),
                          smem_desc_sw128(sG + k_off, kSlabBytes, 1024), idesc_g, kb > 0);
                // dQ[q, d] = sum_key dS[q, key] K[key, d]
                tc_mma_ss(tmem_base + kColDQ, smem_desc_sw128(sdS + a_off, 16, 1024),
                          smem_desc_sw128(sK + k_off, kSlabBytes, 1024), idesc_dq, kb > 0);
                // dK[key, d] = sum_q dS[q, key] Q[q, d]
                tc_mma_ss(tmem_base + kColDK, smem_desc_sw128(sdS + k_off, kSlabBytes, 1024),
                          smem_desc_sw128(sQ + k_off, kSlabBytes, 1024), idesc_g, kb > 0);
            }
            tc_commit(bar_o);
        }
        __syncwarp();
        if (ok) ok = mbar_wait(bar_o, parity, 0x14);
        ok = __all_sync(0xffffffffu, ok);
        tc_fence_after();

        // ---- epilogue: TMEM -> shared staging (box layouts) -> TMA reduce-add / store
        if (ok && warp_valid) {
            uint32_t v[32];
#pragma unroll 1
            for (int which = 0; which < 3; ++which) {
                const uint32_t col0 = which == 0 ? kColDQ : (which == 1 ? kColDK : kColG);
                const uint32_t stage = which == 0 ? stDQ : (which == 1 ? stDK : stG);
                const bool as_bf16 = which == 2 && !a.first_hop;
#pragma unroll 1
                for (int c = 0; c < D / 32; ++c) {
                    tmem_ld32(tmem_lane + col0 + 32 * c, v);
                    if (!row_valid) continue;
                    if (as_bf16) {
                        uint32_t pk[16];
#pragma unroll
                        for (int j = 0; j < 32; j += 2)
                            pk[j >> 1] = pack_bf16x2(__uint_as_float(v[j]), __uint_as_float(v[j + 1]));
                        const uint32_t row = stage + (uint32_t)(c >> 1) * kSlabBytes + (uint32_t)r * 128u;
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            st_shared_v4(row + (uint32_t)((((c & 1) * 4 + i) ^ (r & 7)) * 16), pk[4 * i], pk[4 * i + 1],
                                         pk[4 * i + 2], pk[4 * i + 3]);
                    } else {
                        const uint32_t row = stage + (uint32_t)c * kSlabBytes + (uint32_t)r * 128u;   // 32 floats
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            st_shared_v4(row + (uint32_t)((i ^ (r & 7)) * 16), v[4 * i], v[4 * i + 1], v[4 * i + 2],
                                         v[4 * i + 3]);
                    }
                }
            }
        }
        fence_proxy_async_smem();
        tc_fence_before();
        const int all_ok = __syncthreads_and(ok ? 1 : 0);
        if (tid == 0 && all_ok) {
#pragma unroll
            for (int s = 0; s < D / 32; ++s) {
                tma_reduce_add_5d(&map_dq, stDQ + s * kSlabBytes, 32 * s, 0, c_inner, c_outer, q_head);
                tma_reduce_add_5d(&map_dk, stDK + s * kSlabBytes, 32 * s, 0, c_inner, c_outer, kv_head);
            }
            if (a.first_hop) {
#pragma unroll
                for (int s = 0; s < D / 32; ++s)
                    tma_reduce_add_5d(&map_dv, stG + s * kSlabBytes, 32 * s, 0, c_inner, c_outer, kv_head);
            } else {
#pragma unroll
                for (int h = 0; h < kHalves; ++h)
                    tma_store_5d(&map_gout, stG + h * kSlabBytes, 64 * h, 0, c_inner, c_outer, q_head);
            }
            tma_store_commit_and_wait_read();
        }
        __syncthreads();
        if (!all_ok) break;
    }

    if (tid == 0) tma_store_wait_all();
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

__global__ void f32_to_bf16_kernel(const float *__restrict__ src, __nv_bfloat16 *__restrict__ dst, long long n) {
    for (long long i = (blockIdx.x * (long long)blockDim.x + threadIdx.x) * 4; i < n;
         i += (long long)gridDim.x * blockDim.x * 4) {
        if (i + 3 < n) {
            const float4 f = *reinterpret_cast<const float4 *>(src + i);
            __nv_bfloat162 lo = __floats2bfloat162_rn(f.x, f.y), hi = __floats2bfloat162_rn(f.z, f.w);
            uint2 u;
            u.x = *reinterpret_cast<uint32_t *>(&lo);
            u.y = *reinterpret_cast<uint32_t *>(&hi);
            *reinterpret_cast<uint2 *>(dst + i) = u;
        } else {
            for (long long j = i; j < n; ++j) dst[j] = __float2bfloat16_rn(src[j]);
        }
    }
}

// dv[b, kvh] = sum over the group's query heads of dout[b, h]  (no real hop: out = broadcast v)
template <typename TO>
__global__ void group_sum_kernel(const __nv_bfloat16 *__restrict__ dout, TO *__restrict__ dv, long long per_head,
                                 int H, int H_kv, long long total_kv) {
    const int g = H / H_kv;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total_kv;
         i += (long long)gridDim.x * blockDim.x) {
        const long long bkv = i / per_head, rr = i % per_head;
        const long long b = bkv / H_kv, kvh = bkv % H_kv;
        float s = 0.f;
        for (int j = 0; j < g; ++j) s += __bfloat162float(dout[((b * H + kvh * g + j) * per_head) + rr]);
        if constexpr (sizeof(TO) == 4) dv[i] = s;
        else dv[i] = __float2bfloat16_rn(s);
    }
}

template <int D>
int launch_bwd_d(const Problem &pb, const HopDesc &hd, const void *x, int x_heads, const void *g_in, void *g_out,
                 float *dq_acc, float *dk_acc, float *dv_acc, bool first_hop) {
    CUtensorMap mq, mk, mx, mgi, mgo, mdq, mdk, mdv;
    int rc;
    if ((rc = make_hop_map(&mq, pb.q, pb.B * pb.H, pb.N, D, hd, 2)) != TA_OK) return rc;
    if ((rc = make_hop_map(&mk, pb.k, pb.B * pb.H_kv, pb.N, D, hd, 2)) != TA_OK) return rc;
    if ((rc = make_hop_map(&mx, x, pb.B * x_heads, pb.N, D, hd, 2)) != TA_OK) return rc;
    if ((rc = make_hop_map(&mgi, g_in, pb.B * pb.H, pb.N, D, hd, 2)) != TA_OK) return rc;
    if ((rc = make_hop_map(&mgo, g_out ? g_out : g_in, pb.B * pb.H, pb.N, D, hd, 2)) != TA_OK) return rc;
    if ((rc = make_hop_map(&mdq, dq_acc, pb.B * pb.H, pb.N, D, hd, 4)) != TA_OK) return rc;
    if ((rc = make_hop_map(&mdk, dk_acc, pb.B * pb.H_kv, pb.N, D, hd, 4)) != TA_OK) return rc;
    if ((rc = make_hop_map(&mdv, dv_acc, pb.B * pb.H_kv, pb.N, D, hd, 4)) != TA_OK) return rc;

    BwdArgs a;
    a.n = hd.n; a.rows = hd.rows; a.ci = hd.ci; a.co = hd.co; a.causal = pb.causal;
    a.g = pb.H / pb.H_kv; a.H = pb.H; a.H_kv = pb.H_kv; a.x_is_kv = x_heads != pb.H ? 1 : 0;
    a.first_hop = first_hop ? 1 : 0;
    a.tiles_inner = hd.tiles_inner; a.tiles_outer = hd.tiles_outer;
    a.total_tiles = (long long)pb.B * pb.H * hd.tiles_inner * hd.tiles_outer;
    a.scale = pb.scale;
    a.scale_log2 = pb.scale * 1.4426950408889634f;

    static int num_sms = 0;
    if (num_sms == 0) {
        int dev = 0;
        cudaGetDevice(&dev);
        if (cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || num_sms <= 0)
            num_sms = 148;
    }
    constexpr size_t smem = 4 * (size_t)(D / 64) * kTileRows * 128 + 2 * 2 * kTileRows * 128 + 1024 + 64;
    auto kern = hop_tc_bwd_kernel<D>;
    static bool configured = false;
    if (!configured) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return TA_ERR_CUDA;
        configured = true;
    }
    const unsigned grid = (unsigned)(a.total_tiles < num_sms ? a.total_tiles : num_sms);
    kern<<<grid, kThreads, smem, pb.stream>>>(mq, mk, mx, mgi, mgo, mdq, mdk, mdv, a);
    count_launch();
    return cudaPeekAtLastError() == cudaSuccess ? TA_OK : TA_ERR_CUDA;
}

}  // namespace

int launch_hop_tc_bwd(const Problem &pb, const HopDesc &hd, const void *x, int x_heads, const void *g_in,
                      void *g_out, float *dq_acc, float *dk_acc, float *dv_acc, bool first_hop) {
    if (pb.D == 128) return launch_bwd_d<128>(pb, hd, x, x_heads, g_in, g_out, dq_acc, dk_acc, dv_acc, first_hop);
    if (pb.D == 64) return launch_bwd_d<64>(pb, hd, x, x_heads, g_in, g_out, dq_acc, dk_acc, dv_acc, first_hop);
    return TA_ERR_UNSUPPORTED;
}

int launch_f32_to_bf16(const float *src, void *dst, long long n, cudaStream_t stream) {
    if (n <= 0) return TA_OK;
    long long blocks = (n / 4 + 255) / 256;
    if (blocks > 148 * 32) blocks = 148 * 32;
    if (blocks < 1) blocks = 1;
    f32_to_bf16_kernel<<<(unsigned)blocks, 256, 0, stream>>>(src, (__nv_bfloat16 *)dst, n);
    count_launch();
    return cudaPeekAtLastError() == cudaSuccess ? TA_OK : TA_ERR_CUDA;
}

int launch_group_sum(const void *dout, void *dv, int dv_is_f32, int B, int H, int H_kv, long long per_head,
                     cudaStream_t stream) {
    const long long total = (long long)B * H_kv * per_head;
    long long blocks = (total + 255) / 256;
    if (blocks > 148 * 32) blocks = 148 * 32;
    if (dv_is_f32)
        group_sum_kernel<float><<<(unsigned)blocks, 256, 0, stream>>>((const __nv_bfloat16 *)dout, (float *)dv, per_head,
                                                                     H, H_kv, total);
    else
        group_sum_kernel<__nv_bfloat16><<<(unsigned)blocks, 256, 0, stream>>>(
            (const __nv_bfloat16 *)dout, (__nv_bfloat16 *)dv, per_head, H, H_kv, total);
    count_launch();
    return cudaPeekAtLastError() == cudaSuccess ? TA_OK : TA_ERR_CUDA;
}

int read_status_tc_backward(unsigned int *word) {
    if (cudaMemcpyFromSymbol(word, g_status_word, sizeof(*word)) != cudaSuccess) return TA_ERR_CUDA;
    if (*word != 0) {
        unsigned int z = 0;
        cudaMemcpyToSymbol(g_status_word, &z, sizeof(z));
    }
    return TA_OK;
}

}  // namespace ta
