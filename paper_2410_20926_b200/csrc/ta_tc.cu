// Tensor-core kernel for one hop of tensorized attention on sm_100a (Algorithm 1 loop body,
// Eq. 4), bf16 storage, head dim 64 or 128, segment length n_i <= 128.
//
// A tile is 128 rows = ci*co whole segments of the hop's strided view X[outer][t][inner][D].
// The view is never materialised: a rank-5 TMA tensor map per tensor lists the dimensions as
// (D, t, inner, outer, head) -- strides inner*D, D, n*inner*D, N*D elements -- so that one box
// (64, n, ci, co, 1) lands in shared memory with the rows of a segment adjacent (row =
// segment_in_tile * n + t), 128 bytes per row, 128B-swizzled: exactly the K-major operand
// layout of tcgen05.mma for Q and K, and the MN-major one for the value tile.
//
// Per tile:  S = Q K^T (tcgen05.mma, fp32 in TMEM)  ->  block-diagonal + causal mask, row softmax
// in fp32 registers (tcgen05.ld), un-normalised weights rounded to bf16 into shared memory
// (over the Q/K tiles, which are dead by then)  ->  O = P X (tcgen05.mma, fp32 in TMEM)  ->
// O / rowsum -> bf16 -> shared memory (over the X tile)  ->  TMA store to the same strided rows.
// Because a tile owns whole segments, the value tensor is updated in place.
#include <cuda_bf16.h>

#include <mutex>

#include "ta_internal.h"
#include "ta_ptx.cuh"

namespace ta {

namespace {

constexpr int kTileRows = 128;
constexpr int kThreads = 128;

struct TcArgs {
    int n, rows, ci, co, causal, g, H, H_kv, xin_is_kv;
    long long tiles_inner, tiles_outer, total_tiles;
    float scale_log2;
};

// ----------------------------------------------------------------------------- the kernel
template <int D>
__global__ void __launch_bounds__(kThreads)
hop_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
              const __grid_constant__ CUtensorMap map_xin, const __grid_constant__ CUtensorMap map_xout,
              const TcArgs a) {
    constexpr int kHalves = D / 64;                 // 64-column (128-byte) slabs per row
    constexpr uint32_t kSlabBytes = kTileRows * 128;  // one [128 rows][64 cols] bf16 slab
    constexpr uint32_t kTileBytes = kHalves * kSlabBytes;
    constexpr uint32_t kTmemCols = 256;             // S: 128 columns, O: D columns
    constexpr uint32_t kOCol = 128;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t sQ = smem_u32(smem);
    const uint32_t sK = sQ + kTileBytes;
    const uint32_t sX = sK + kTileBytes;
    const uint32_t sP = sQ;                         // P (128 x 128 bf16, 32 KB) reuses the Q/K space
    uint64_t *bars = (uint64_t *)(smem + 3 * kTileBytes);
    const uint32_t bar_qk = smem_u32(bars + 0), bar_x = smem_u32(bars + 1), bar_s = smem_u32(bars + 2),
                   bar_o = smem_u32(bars + 3);
    uint32_t *tmem_slot = (uint32_t *)(bars + 4);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // ---- one-time setup
    for (uint32_t i = tid; i < 3 * kTileBytes / 16; i += kThreads)
        ((uint4 *)smem)[i] = make_uint4(0, 0, 0, 0);   // rows a box never fills must stay finite
    if (tid == 0) {
        mbar_init(bar_qk, 1);
        mbar_init(bar_x, 1);
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

    constexpr uint32_t idesc_s = instr_desc(128, 0);
    constexpr uint32_t idesc_o = instr_desc(D, 1);

    const int r = warp * 32 + lane;                 // this thread's tile row = TMEM lane
    const int seg = r / a.n;
    const bool row_valid = r < a.rows;
    const int c_lo = seg * a.n;
    const int c_hi = a.causal ? r + 1 : c_lo + a.n; // visible key columns [c_lo, c_hi)
    // columns any row of this warp needs (warp-uniform)
    const int w_lo = ((warp * 32) / a.n) * a.n;
    int w_hi = min(a.rows, ((warp * 32 + 31) / a.n + 1) * a.n);
    if (a.causal) w_hi = min(w_hi, warp * 32 + 32);
    const bool warp_valid = warp * 32 < a.rows;

    bool ok = true;
    uint32_t it = 0;
    for (long long tile = blockIdx.x; tile < a.total_tiles; tile += gridDim.x, ++it) {
        const uint32_t parity = it & 1u;
        // tile -> (query head of the group, inner tile, outer tile, kv head, batch); the heads
        // of a GQA group are adjacent so that their common K (and V) tile is hot in L2.
        long long rest = tile;
        const int hg = (int)(rest % a.g); rest /= a.g;
        const int c_inner = (int)(rest % a.tiles_inner) * a.ci; rest /= a.tiles_inner;
        const int c_outer = (int)(rest % a.tiles_outer) * a.co; rest /= a.tiles_outer;
        const int kv_head = (int)rest;                              // b * H_kv + kvh
        const int q_head = (kv_head / a.H_kv) * a.H + (kv_head % a.H_kv) * a.g + hg;
        const int x_head = a.xin_is_kv ? kv_head : q_head;

        if (tid == 0) {
            const uint32_t slab_tx = (uint32_t)a.rows * 128u;
            mbar_expect_tx(bar_qk, 2 * kHalves * slab_tx);
#pragma unroll
            for (int h = 0; h < kHalves; ++h) tma_load_5d(sQ + h * kSlabBytes, &map_q, bar_qk, 64 * h, 0, c_inner, c_outer, q_head);
#pragma unroll
            for (int h = 0; h < kHalves; ++h) tma_load_5d(sK + h * kSlabBytes, &map_k, bar_qk, 64 * h, 0, c_inner, c_outer, kv_head);
            mbar_expect_tx(bar_x, kHalves * slab_tx);
#pragma unroll
            for (int h = 0; h < kHalves; ++h) tma_load_5d(sX + h * kSlabBytes, &map_xin, bar_x, 64 * h, 0, c_inner, c_outer, x_head);

            ok = mbar_wait(bar_qk, parity, 1);
            if (ok) {
                tc_fence_after();
                // S[128 x 128] = Q[128 x D] K^T : D/16 instructions of K = 16
#pragma unroll
                for (int kb = 0; kb < D / 16; ++kb) {
                    const uint32_t off = (kb >> 2) * kSlabBytes + (kb & 3) * 32;
                    tc_mma_ss(tmem_base, smem_desc_sw128(sQ + off, 16, 1024), smem_desc_sw128(sK + off, 16, 1024),
                              idesc_s, kb > 0);
                }
                tc_commit(bar_s);
            }
        }
        __syncwarp();
        if (ok) ok = mbar_wait(bar_s, parity, 2);
        ok = __all_sync(0xffffffffu, ok);          // keep every warp converged for the aligned TMEM ops
        tc_fence_after();

        // ---- softmax over the row's visible columns; P (un-normalised, bf16) -> sP
        float row_sum = 1.f;
        if (ok) {
            float m = -INFINITY;
            uint32_t v[32];
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                if (!(warp_valid && 32 * c < w_hi && 32 * c + 32 > w_lo)) continue;   // warp-uniform
                tmem_ld32(tmem_lane + 32 * c, v);
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const int col = 32 * c + j;
                    const float s = __uint_as_float(v[j]);
                    if (col >= c_lo && col < c_hi) m = fmaxf(m, s);
                }
            }
            const float m_scaled = row_valid ? m * a.scale_log2 : 0.f;
            float sum = 0.f;
            const uint32_t row_base = sP + (uint32_t)r * 128u;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                uint32_t pk[16];
                if (warp_valid && 32 * c < w_hi && 32 * c + 32 > w_lo) {
                    tmem_ld32(tmem_lane + 32 * c, v);
#pragma unroll
                    for (int j = 0; j < 32; j += 2) {
                        const int col = 32 * c + j;
                        float p0 = fast_exp2(__uint_as_float(v[j]) * a.scale_log2 - m_scaled);
                        float p1 = fast_exp2(__uint_as_float(v[j + 1]) * a.scale_log2 - m_scaled);
                        p0 = (row_valid && col >= c_lo && col < c_hi) ? p0 : 0.f;
                        p1 = (row_valid && col + 1 >= c_lo && col + 1 < c_hi) ? p1 : 0.f;
                        const uint32_t w = pack_bf16x2(p0, p1);
                        pk[j >> 1] = w;
                        sum += __uint_as_float(w << 16) + __uint_as_float(w & 0xFFFF0000u);
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 16; ++j) pk[j] = 0u;
                }
                const uint32_t slab = row_base + (uint32_t)(c >> 1) * kSlabBytes;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t chunk = (uint32_t)(((c & 1) * 4 + i) ^ (r & 7));
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(slab + chunk * 16), "r"(pk[4 * i]),
                                 "r"(pk[4 * i + 1]), "r"(pk[4 * i + 2]), "r"(pk[4 * i + 3])
                                 : "memory");
                }
            }
            row_sum = row_valid ? sum : 1.f;
        }
        fence_proxy_async_smem();
        tc_fence_before();
        __syncthreads();

        if (tid == 0 && ok) {
            tc_fence_after();
            ok = mbar_wait(bar_x, parity, 3);
            if (ok) {
                // O[128 x D] = P[128 x rows] X[rows x D]; X rows are keys (MN-major B operand)
                const int kblocks = (a.rows + 15) >> 4;
                for (int kb = 0; kb < kblocks; ++kb) {
                    const uint32_t a_off = (kb >> 2) * kSlabBytes + (kb & 3) * 32;
                    tc_mma_ss(tmem_base + kOCol, smem_desc_sw128(sP + a_off, 16, 1024),
                              smem_desc_sw128(sX + kb * 2048, kSlabBytes, 1024), idesc_o, kb > 0);
                }
                tc_commit(bar_o);
            }
        }
        __syncwarp();
        if (ok) ok = mbar_wait(bar_o, parity, 4);
        ok = __all_sync(0xffffffffu, ok);
        tc_fence_after();

        // ---- epilogue: O / rowsum -> bf16 -> sX (same swizzled box layout) -> TMA store
        if (ok && warp_valid) {
            const float inv = 1.f / row_sum;
            uint32_t v[32];
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
                tmem_ld32(tmem_lane + kOCol + 32 * c, v);   // whole warp, rows beyond `rows` discard it
                uint32_t pk[16];
#pragma unroll
                for (int j = 0; j < 32; j += 2)
                    pk[j >> 1] = pack_bf16x2(__uint_as_float(v[j]) * inv, __uint_as_float(v[j + 1]) * inv);
                const uint32_t slab = sX + (uint32_t)(c >> 1) * kSlabBytes + (uint32_t)r * 128u;
                if (row_valid) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint32_t chunk = (uint32_t)(((c & 1) * 4 + i) ^ (r & 7));
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(slab + chunk * 16),
                                     "r"(pk[4 * i]), "r"(pk[4 * i + 1]), "r"(pk[4 * i + 2]), "r"(pk[4 * i + 3])
                                     : "memory");
                    }
                }
            }
        }
        fence_proxy_async_smem();
        tc_fence_before();
        const int all_ok = __syncthreads_and(ok ? 1 : 0);
        if (tid == 0 && all_ok) {
#pragma unroll
            for (int h = 0; h < kHalves; ++h) tma_store_5d(&map_xout, sX + h * kSlabBytes, 64 * h, 0, c_inner, c_outer, q_head);
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

// ----------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    });
    return fn;
}

}  // namespace

// Rank-5 map of one tensor [heads][N][D] seen through hop `hd`: dims (D, t, inner, outer, head),
// box (128 bytes of D, n, ci, co, 1), 128-byte swizzle.  elem = 2 (bf16) or 4 (fp32).
int make_hop_map(CUtensorMap *map, const void *base, int heads_total, int N, int D, const HopDesc &hd, int elem) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return TA_ERR_CUDA;
    const cuuint64_t e = (cuuint64_t)elem;
    cuuint64_t gdim[5] = {(cuuint64_t)D, (cuuint64_t)hd.n, (cuuint64_t)hd.stride, (cuuint64_t)hd.outer,
                          (cuuint64_t)heads_total};
    cuuint64_t gstr[4] = {(cuuint64_t)hd.stride * D * e, (cuuint64_t)D * e, (cuuint64_t)hd.n * hd.stride * D * e,
                          (cuuint64_t)N * D * e};
    cuuint32_t box[5] = {(cuuint32_t)(128 / elem), (cuuint32_t)hd.n, (cuuint32_t)hd.ci, (cuuint32_t)hd.co, 1u};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    CUresult r = enc(map, elem == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 5,
                     const_cast<void *>(base), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? TA_OK : TA_ERR_CUDA;
}

namespace {

template <int D>
int launch_d(const Problem &pb, const HopDesc &hd, const void *xin, int xin_heads, void *xout) {
    CUtensorMap mq, mk, mxi, mxo;
    int rc;
    if ((rc = make_hop_map(&mq, pb.q, pb.B * pb.H, pb.N, D, hd, 2)) != TA_OK) return rc;
    if ((rc = make_hop_map(&mk, pb.k, pb.B * pb.H_kv, pb.N, D, hd, 2)) != TA_OK) return rc;
    if ((rc = make_hop_map(&mxi, xin, pb.B * xin_heads, pb.N, D, hd, 2)) != TA_OK) return rc;
    if ((rc = make_hop_map(&mxo, xout, pb.B * pb.H, pb.N, D, hd, 2)) != TA_OK) return rc;

    TcArgs a;
    a.n = hd.n; a.rows = hd.rows; a.ci = hd.ci; a.co = hd.co; a.causal = pb.causal;
    a.g = pb.H / pb.H_kv; a.H = pb.H; a.H_kv = pb.H_kv; a.xin_is_kv = xin_heads != pb.H ? 1 : 0;
    a.tiles_inner = hd.tiles_inner; a.tiles_outer = hd.tiles_outer;
    a.total_tiles = (long long)pb.B * pb.H * hd.tiles_inner * hd.tiles_outer;
    a.scale_log2 = pb.scale * 1.4426950408889634f;

    static int num_sms = 0;
    if (num_sms == 0) {
        int dev = 0;
        cudaGetDevice(&dev);
        if (cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || num_sms <= 0)
            num_sms = 148;
    }
    constexpr size_t smem = 3 * (size_t)(D / 64) * kTileRows * 128 + 1024 /*alignment slack*/ + 64 /*barriers*/;
    auto kern = hop_tc_kernel<D>;
    static bool configured = false;
    if (!configured) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return TA_ERR_CUDA;
        configured = true;
    }
    const long long max_ctas = 2ll * num_sms;
    const unsigned grid = (unsigned)(a.total_tiles < max_ctas ? a.total_tiles : max_ctas);
    kern<<<grid, kThreads, smem, pb.stream>>>(mq, mk, mxi, mxo, a);
    count_launch();
    return cudaPeekAtLastError() == cudaSuccess ? TA_OK : TA_ERR_CUDA;
}

}  // namespace

int launch_hop_tc(const Problem &pb, const HopDesc &hd, const void *xin, int xin_heads, void *xout) {
    if (pb.D == 128) return launch_d<128>(pb, hd, xin, xin_heads, xout);
    if (pb.D == 64) return launch_d<64>(pb, hd, xin, xin_heads, xout);
    return TA_ERR_UNSUPPORTED;
}

int read_status_tc_forward(unsigned int *word) {
    if (cudaMemcpyFromSymbol(word, g_status_word, sizeof(*word)) != cudaSuccess) return TA_ERR_CUDA;
    if (*word != 0) {
        unsigned int z = 0;
        cudaMemcpyToSymbol(g_status_word, &z, sizeof(z));
    }
    return TA_OK;
}

}  // namespace ta
