// Tensor-core kernel for one hop of tensorized attention over LONG segments (n_i > 128;
// ndims == 1 is ordinary attention over the whole sequence), bf16, head dim 64 or 128
// (Algorithm 1 loop body, Eq. 4; the softmax row no longer fits one tile, so it is taken
// block by block with a running maximum and sum -- "online" softmax in fp32).
//
// A work item is 128 consecutive positions t0 .. t0+127 of one segment of one query head.  Its
// Q tile stays in shared memory while the segment's keys go by in blocks of 128 (causal: up to
// the block of the diagonal); per key block j
//     S_j = Q K_j^T (tcgen05.mma, fp32 in TMEM, double-buffered)
//     m <- max(m, rowmax S_j),  alpha = 2^(m_old - m),  l <- alpha l + rowsum P_j,
//     P_j = 2^(S_j scale log2e - m)  (bf16, written back to TMEM over S_j)
//     O <- alpha O  (in TMEM, only when some row's maximum moved)   then   O += P_j X_j
// and finally O / l -> bf16 -> shared memory -> TMA store.  Rows of the strided view are reached
// with the same rank-5 TMA maps as the short-segment kernel (box = 128 positions of one
// segment); positions past n are zero-filled on load and clipped on store.  Several items read
// the value rows another item writes, so the hop is not in place: xin != xout.
//
// Persistent, one CTA per SM: warp 0 TMA producer (Q per item, K_j / X_j into a two-stage
// ring), warp 1 MMA issuer, warps 4-7 softmax / rescaling / epilogue (one TMEM lane = one
// query row per thread), warp 2 TMA store.  Every wait is bounded; when one expires the CTA
// raises a flag that ends all its roles, waits for its copies in flight, frees its TMEM and
// returns.
#include <cuda_bf16.h>

#include "ta_internal.h"
#include "ta_ptx.cuh"

namespace ta {
namespace {

constexpr int kTileRows = 128;
constexpr int kThreads = 256;
constexpr int kNQ = 2;    // Q slots (one per item in flight)
constexpr int kNKV = 2;   // key / value block ring

struct LongArgs {
    int n, causal, g, H, H_kv, xin_is_kv, qblocks;
    int window;                // 0, or w: keys within w positions of the query (blocks outside are skipped)
    long long stride, outer, total_items;
    float scale_log2;
};

template <int D>
struct LongCfg {
    static constexpr int kHalves = D / 64;
    static constexpr uint32_t kSlabBytes = kTileRows * 128;
    static constexpr uint32_t kTileBytes = kHalves * kSlabBytes;
    static constexpr uint32_t kOffQ = 0;
    static constexpr uint32_t kOffKV = kOffQ + kNQ * kTileBytes;           // per stage: K then X
    static constexpr uint32_t kOffOut = kOffKV + kNKV * 2 * kTileBytes;    // output staging
    static constexpr uint32_t kOffBar = kOffOut + kTileBytes;
    static constexpr int kNumBars = 2 * kNQ + 2 * kNKV + 2 + 2 + 1 + 2;
    static constexpr uint32_t kSmemBytes = kOffBar + kNumBars * 8 + 16 + 1024;
    static constexpr uint32_t kTmemCols = 512;
    static constexpr uint32_t kColS = 0, kColO = 256;   // S: 2 x 128 (P over the first 64 of each), O: D
};

struct LongItem {
    int t0, inner, outer, q_head, kv_head;
    int j0, nkv, keys_end;     // key blocks j0 .. j0+nkv-1 (128 keys each), keys [.., keys_end) in all
};
// item -> (query block, inner, outer, head).  Query blocks of a segment are adjacent, later
// (longer, when causal) blocks first, so that the CTAs of one wave carry similar loads.
__device__ __forceinline__ LongItem decode_long_item(const LongArgs &a, long long item) {
    LongItem c;
    long long rest = item;
    const int qb = a.qblocks - 1 - (int)(rest % a.qblocks); rest /= a.qblocks;
    c.inner = (int)(rest % a.stride); rest /= a.stride;
    c.outer = (int)(rest % a.outer); rest /= a.outer;
    c.q_head = (int)rest;                                          // b * H + h
    c.kv_head = (c.q_head / a.H) * a.H_kv + (c.q_head % a.H) / a.g;
    c.t0 = qb * kTileRows;
    // keys any row of the tile can see: [first, keys_end)
    int first = 0;
    c.keys_end = a.causal ? min(c.t0 + kTileRows, a.n) : a.n;
    if (a.window > 0) {
        first = max(0, c.t0 - a.window + 1);
        if (!a.causal) c.keys_end = min(a.n, c.t0 + kTileRows - 1 + a.window);
    }
    c.j0 = first / kTileRows;
    c.nkv = (c.keys_end + kTileRows - 1) / kTileRows - c.j0;
    return c;
}

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32]) {
    __syncwarp();
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
          "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]),
          "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
        : "memory");
}

template <int D, bool kWindow>
__global__ void __launch_bounds__(kThreads, 1)
hop_long_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_xin, const __grid_constant__ CUtensorMap map_xout,
                const LongArgs a) {
    using C = LongCfg<D>;
    constexpr int kHalves = C::kHalves;
    constexpr uint32_t kSlabBytes = C::kSlabBytes, kTileBytes = C::kTileBytes;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t s0 = smem_u32(smem);
    auto sQ = [&](int s) { return s0 + C::kOffQ + (uint32_t)s * kTileBytes; };
    auto sKb = [&](int s) { return s0 + C::kOffKV + (uint32_t)s * 2 * kTileBytes; };
    auto sXb = [&](int s) { return s0 + C::kOffKV + (uint32_t)s * 2 * kTileBytes + kTileBytes; };
    const uint32_t sOut = s0 + C::kOffOut;
    const uint32_t bar0 = s0 + C::kOffBar;
    auto q_full = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    auto q_free = [&](int i) { return bar0 + 8u * (uint32_t)(kNQ + i); };
    auto kv_full = [&](int i) { return bar0 + 8u * (uint32_t)(2 * kNQ + i); };
    auto kv_free = [&](int i) { return bar0 + 8u * (uint32_t)(2 * kNQ + kNKV + i); };
    constexpr int kB1 = 2 * kNQ + 2 * kNKV;
    auto s_full = [&](int i) { return bar0 + 8u * (uint32_t)(kB1 + i); };
    auto p_full = [&](int i) { return bar0 + 8u * (uint32_t)(kB1 + 2 + i); };
    const uint32_t pv_done = bar0 + 8u * (uint32_t)(kB1 + 4);
    const uint32_t out_full = bar0 + 8u * (uint32_t)(kB1 + 5), out_free = bar0 + 8u * (uint32_t)(kB1 + 6);
    uint32_t *tmem_slot = (uint32_t *)(smem + C::kOffBar + C::kNumBars * 8);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    for (uint32_t i = tid; i < C::kOffBar / 16; i += kThreads) ((uint4 *)smem)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) {
        for (int i = 0; i < C::kNumBars; ++i) {
            const uint32_t bar = bar0 + 8u * (uint32_t)i;
            // arrivals: one per softmax warp on p_full / out_full, a single thread or commit elsewhere
            mbar_init(bar, (bar == p_full(0) || bar == p_full(1) || bar == out_full) ? 4 : 1);
        }
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    fence_proxy_async_smem();
    if (warp == 3) {
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

    if (warp == 0) {
        // =============================================================== TMA producer
        if (lane == 0) {
            uint32_t ic = 0, g = 0;
            uint32_t armed = 0, last_par = 0;        // bits: q 0-1, kv 2-3
            auto arm = [&](uint32_t bit, uint32_t parity) {
                armed |= bit;
                last_par = parity ? (last_par | bit) : (last_par & ~bit);
            };
            bool ok = true;
            for (long long item = blockIdx.x; ok && item < a.total_items; item += gridDim.x, ++ic) {
                const LongItem c = decode_long_item(a, item);
                const int x_head = a.xin_is_kv ? c.kv_head : c.q_head;
                const int qs = ic & 1;
                ok = mbar_wait_abortable(q_free(qs), ((ic >> 1) & 1) ^ 1, 0xD0, abort_flag);
                if (!ok) break;
                mbar_expect_tx(q_full(qs), kTileBytes);
                arm(1u << qs, (ic >> 1) & 1);
#pragma unroll
                for (int h = 0; h < kHalves; ++h)
                    tma_load_5d(sQ(qs) + h * kSlabBytes, &map_q, q_full(qs), 64 * h, c.t0, c.inner, c.outer, c.q_head);
                for (int j = 0; j < c.nkv; ++j, ++g) {
                    const int st = g % kNKV;
                    const uint32_t par = (g / kNKV) & 1;
                    ok = mbar_wait_abortable(kv_free(st), par ^ 1, 0xD1, abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(kv_full(st), 2 * kTileBytes);
                    arm(4u << st, par);
#pragma unroll
                    for (int h = 0; h < kHalves; ++h)
                        tma_load_5d(sKb(st) + h * kSlabBytes, &map_k, kv_full(st), 64 * h, kTileRows * (c.j0 + j), c.inner, c.outer, c.kv_head);
#pragma unroll
                    for (int h = 0; h < kHalves; ++h)
                        tma_load_5d(sXb(st) + h * kSlabBytes, &map_xin, kv_full(st), 64 * h, kTileRows * (c.j0 + j), c.inner, c.outer, x_head);
                }
            }
            if (!ok) {
                const unsigned long long t0 = globaltimer_ns();
                for (int slot = 0; slot < 4; ++slot) {
                    if (!(armed & (1u << slot))) continue;
                    const uint32_t bar = slot < 2 ? q_full(slot) : kv_full(slot - 2);
                    while (!mbar_try_wait(bar, (last_par >> slot) & 1u) && globaltimer_ns() - t0 < 10000000ull) {
                    }
                }
            }
        }
    } else if (warp == 1) {
        // =============================================================== MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc_s = instr_desc(128, 0);
            constexpr uint32_t idesc_o = instr_desc(D, 1);
            uint32_t ic = 0, g0 = 0;
            bool ok = true;
            for (long long item = blockIdx.x; ok && item < a.total_items; item += gridDim.x, ++ic) {
                const LongItem c = decode_long_item(a, item);
                const int qs = ic & 1;
                ok = mbar_wait_abortable(q_full(qs), (ic >> 1) & 1, 0xE0, abort_flag);
                if (!ok) break;
                auto issue_s = [&](int j) -> bool {
                    const uint32_t g = g0 + j;
                    const int st = g % kNKV;
                    if (!mbar_wait_abortable(kv_full(st), (g / kNKV) & 1, 0xE1, abort_flag)) return false;
                    tc_fence_after();
#pragma unroll
                    for (int kb = 0; kb < D / 16; ++kb) {
                        const uint32_t off = (kb >> 2) * kSlabBytes + (kb & 3) * 32;
                        tc_mma_ss(tmem_base + C::kColS + (g & 1) * 128, smem_desc_sw128(sQ(qs) + off, 16, 1024),
                                  smem_desc_sw128(sKb(st) + off, 16, 1024), idesc_s, kb > 0);
                    }
                    tc_commit(s_full(g & 1));
                    return true;
                };
                auto issue_pv = [&](int j) -> bool {
                    const uint32_t g = g0 + j;
                    const int st = g % kNKV;
                    if (!mbar_wait_abortable(p_full(g & 1), (g >> 1) & 1, 0xE2, abort_flag)) return false;
                    tc_fence_after();
                    const int keys = min(kTileRows, c.keys_end - kTileRows * (c.j0 + j));
                    const int kblocks = (keys + 15) >> 4;
                    for (int kb = 0; kb < kblocks; ++kb)
                        tc_mma_ts(tmem_base + C::kColO, tmem_base + C::kColS + (g & 1) * 128 + kb * 8,
                                  smem_desc_sw128(sXb(st) + kb * 2048, kSlabBytes, 1024), idesc_o, (kb > 0 || j > 0) ? 1u : 0u);
                    tc_commit(kv_free(st));
                    tc_commit(pv_done);
                    return true;
                };
                ok = issue_s(0);
                for (int j = 0; ok && j < c.nkv; ++j) {
                    if (j + 1 < c.nkv) {
                        ok = issue_s(j + 1);
                        if (!ok) break;
                    }
                    if (j + 1 == c.nkv) tc_commit(q_free(qs));     // every S of this item has been issued
                    ok = issue_pv(j);
                }
                g0 += c.nkv;
            }
        }
    } else if (warp == 2) {
        // =============================================================== TMA store
        if (lane == 0) {
            uint32_t ic = 0;
            bool ok = true;
            for (long long item = blockIdx.x; ok && item < a.total_items; item += gridDim.x, ++ic) {
                const LongItem c = decode_long_item(a, item);
                ok = mbar_wait_abortable(out_full, ic & 1, 0xF0, abort_flag);
                if (!ok) break;
#pragma unroll
                for (int h = 0; h < kHalves; ++h)
                    tma_store_5d(&map_xout, sOut + h * kSlabBytes, 64 * h, c.t0, c.inner, c.outer, c.q_head);
                tma_store_commit_and_wait_read();
                mbar_arrive(out_free);
            }
            tma_store_wait_all();
        }
    } else if (warp >= 4) {
        // =============================================================== softmax, rescaling, epilogue
        const int wq = warp & 3;                        // TMEM lane quarter of this warp
        const uint32_t tmem_lane = tmem_base + ((uint32_t)(wq * 32) << 16);
        const int r = wq * 32 + lane;                   // this thread's query row of the tile
        const uint32_t o_col = tmem_lane + C::kColO;

        bool ok = true;
        uint32_t ic = 0, g = 0;
        for (long long item = blockIdx.x; ok && item < a.total_items; item += gridDim.x, ++ic) {
            const LongItem c = decode_long_item(a, item);
            const int t = c.t0 + r;                     // position of this row in the segment
            const bool row_valid = t < a.n;
            float m_run = -INFINITY, l_run = 0.f;       // running maximum (scaled, log2 domain) and sum
            for (int j = 0; j < c.nkv; ++j, ++g) {
                const uint32_t buf = g & 1;
                const uint32_t s_col = tmem_lane + C::kColS + buf * 128;
                const int u0 = kTileRows * (c.j0 + j);
                const int keys = min(kTileRows, c.keys_end - u0);          // key columns of this block
                // columns any row of this warp can see in this block (warp-uniform)
                const bool diag = a.causal && u0 == c.t0;
                const int w_hi = diag ? min(keys, wq * 32 + 32) : keys;
                // this row: columns [c_lo, c_hi) of the block
                int c_hi = !row_valid ? 0 : (diag ? min(keys, r + 1) : keys);
                int c_lo = 0;                           // stays a compile-time 0 without a window
                if (kWindow) {
                    c_lo = max(0, t - a.window + 1 - u0);
                    if (!a.causal) c_hi = min(c_hi, t + a.window - u0);
                }
                const int nchunks = (keys + 31) >> 5;

                ok = mbar_wait_abortable(s_full(buf), (g >> 1) & 1, 0xF4, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();

                float bm = -INFINITY;
                uint32_t v[32];
#pragma unroll 1
                for (int cc = 0; cc < nchunks; ++cc) {
                    if (32 * cc >= w_hi) continue;      // warp-uniform
                    tmem_ld32(s_col + 32 * cc, v);
#pragma unroll
                    for (int jj = 0; jj < 32; ++jj)
                        if (32 * cc + jj >= c_lo && 32 * cc + jj < c_hi) bm = fmaxf(bm, __uint_as_float(v[jj]));
                }
                // (with a window a row may see nothing in a block: the running maximum then stays -inf
                // until its first visible key, and the reference below keeps the arithmetic finite)
                const float m_new = fmaxf(m_run, bm * a.scale_log2);
                const float m_ref = m_new == -INFINITY ? 0.f : m_new;
                const float alpha = m_run == -INFINITY ? 1.f : fast_exp2(m_run - m_ref);

                // ---- O <- alpha O, once the previous block's value MMA has completed
                if (j > 0) {
                    ok = mbar_wait_abortable(pv_done, (g - 1) & 1, 0xF5, abort_flag);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    tc_fence_after();
                    if (__any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll 1
                        for (int cc = 0; cc < D / 32; ++cc) {
                            tmem_ld32(o_col + 32 * cc, v);
#pragma unroll
                            for (int jj = 0; jj < 32; ++jj) v[jj] = __float_as_uint(__uint_as_float(v[jj]) * alpha);
                            tmem_st32(o_col + 32 * cc, v);
                        }
                    }
                }

                // ---- P_j (un-normalised, bf16) over the S columns already consumed
                float sum = 0.f;
#pragma unroll 1
                for (int cc = 0; cc < nchunks; ++cc) {
                    uint32_t pk[16];
                    if (32 * cc < w_hi) {
                        tmem_ld32(s_col + 32 * cc, v);
#pragma unroll
                        for (int jj = 0; jj < 32; jj += 2) {
                            const int col = 32 * cc + jj;
                            float p0 = fast_exp2(__uint_as_float(v[jj]) * a.scale_log2 - m_ref);
                            float p1 = fast_exp2(__uint_as_float(v[jj + 1]) * a.scale_log2 - m_ref);
                            p0 = (col >= c_lo && col < c_hi) ? p0 : 0.f;
                            p1 = (col + 1 >= c_lo && col + 1 < c_hi) ? p1 : 0.f;
                            const uint32_t w = pack_bf16x2(p0, p1);
                            pk[jj >> 1] = w;
                            sum += __uint_as_float(w << 16) + __uint_as_float(w & 0xFFFF0000u);
                        }
                    } else {
#pragma unroll
                        for (int jj = 0; jj < 16; ++jj) pk[jj] = 0u;
                    }
                    tmem_st16(s_col + 16 * cc, pk);
                }
                tmem_st_wait();
                l_run = l_run * alpha + sum;
                m_run = m_new;
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(p_full(buf));
            }
            if (!ok) break;

            // ---- epilogue: O / l -> bf16 -> staging (box layout) -> store warp
            ok = mbar_wait_abortable(pv_done, (g - 1) & 1, 0xF6, abort_flag);
            if (ok) ok = mbar_wait_abortable(out_free, (ic & 1) ^ 1, 0xF7, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            {
                const float inv = (row_valid && l_run > 0.f) ? 1.f / l_run : 0.f;
                uint32_t v[32];
                const uint32_t row = sOut + (uint32_t)r * 128u;
#pragma unroll 1
                for (int cc = 0; cc < D / 32; ++cc) {
                    tmem_ld32(o_col + 32 * cc, v);
                    uint32_t pk[16];
#pragma unroll
                    for (int jj = 0; jj < 32; jj += 2)
                        pk[jj >> 1] = pack_bf16x2(__uint_as_float(v[jj]) * inv, __uint_as_float(v[jj + 1]) * inv);
                    const uint32_t slab = row + (uint32_t)(cc >> 1) * kSlabBytes;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint32_t chunk = (uint32_t)(((cc & 1) * 4 + i) ^ (r & 7));
                        st_shared_v4(slab + chunk * 16, pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
                    }
                }
            }
            fence_proxy_async_smem();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(out_full);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 3) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::kTmemCols) : "memory");
    }
}

template <int D>
int launch_long_d(const Problem &pb, const HopDesc &hd, const void *xin, int xin_heads, void *xout) {
    CUtensorMap mq, mk, mxi, mxo;
    int rc;
    // box: 128 positions of one segment (positions past n are zero-filled / clipped)
    if ((rc = make_view_map(&mq, pb.q, pb.B * pb.H, pb.N, D, hd, 2, kTileRows, 1, 1)) != TA_OK) return rc;
    if ((rc = make_view_map(&mk, pb.k, pb.B * pb.H_kv, pb.N, D, hd, 2, kTileRows, 1, 1)) != TA_OK) return rc;
    if ((rc = make_view_map(&mxi, xin, pb.B * xin_heads, pb.N, D, hd, 2, kTileRows, 1, 1)) != TA_OK) return rc;
    if ((rc = make_view_map(&mxo, xout, pb.B * pb.H, pb.N, D, hd, 2, kTileRows, 1, 1)) != TA_OK) return rc;

    LongArgs a;
    a.n = hd.n; a.causal = pb.causal; a.g = pb.H / pb.H_kv; a.H = pb.H; a.H_kv = pb.H_kv;
    a.xin_is_kv = xin_heads != pb.H ? 1 : 0;
    a.qblocks = (hd.n + kTileRows - 1) / kTileRows;
    a.stride = hd.stride; a.outer = hd.outer;
    a.total_items = (long long)pb.B * pb.H * hd.outer * hd.stride * a.qblocks;
    a.window = pb.window[hd.hop];
    a.scale_log2 = pb.scale * 1.4426950408889634f;

    static int num_sms = 0;
    if (num_sms == 0) {
        int dev = 0;
        cudaGetDevice(&dev);
        if (cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || num_sms <= 0)
            num_sms = 148;
    }
    constexpr size_t smem = LongCfg<D>::kSmemBytes;
    static bool configured = false;
    if (!configured) {
        if (cudaFuncSetAttribute(hop_long_kernel<D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
                cudaSuccess ||
            cudaFuncSetAttribute(hop_long_kernel<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
                cudaSuccess)
            return TA_ERR_CUDA;
        configured = true;
    }
    const unsigned grid = (unsigned)(a.total_items < num_sms ? a.total_items : num_sms);
    if (a.window > 0)
        hop_long_kernel<D, true><<<grid, kThreads, smem, pb.stream>>>(mq, mk, mxi, mxo, a);
    else
        hop_long_kernel<D, false><<<grid, kThreads, smem, pb.stream>>>(mq, mk, mxi, mxo, a);
    count_launch();
    return cudaPeekAtLastError() == cudaSuccess ? TA_OK : TA_ERR_CUDA;
}

}  // namespace

int launch_hop_tc_long(const Problem &pb, const HopDesc &hd, const void *xin, int xin_heads, void *xout) {
    if (xin == xout) return TA_ERR_INVALID_ARG;
    if (pb.D == 128) return launch_long_d<128>(pb, hd, xin, xin_heads, xout);
    if (pb.D == 64) return launch_long_d<64>(pb, hd, xin, xin_heads, xout);
    return TA_ERR_UNSUPPORTED;
}

int read_status_tc_long(unsigned int *word) {
    if (cudaMemcpyFromSymbol(word, g_status_word, sizeof(*word)) != cudaSuccess) return TA_ERR_CUDA;
    if (*word != 0) {
        unsigned int z = 0;
        cudaMemcpyToSymbol(g_status_word, &z, sizeof(z));
    }
    return TA_OK;
}

}  // namespace ta
