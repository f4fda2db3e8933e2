// Tensor-core backward kernel for one hop with segments longer than a tile (n_i > 128) on sm_100a:
// bf16 storage, head dim 64 or 128, causal flag, sliding window and valid lengths as in the forward
// (explicit masks run on the generic kernels; with the positional encoding the hop runs on rotated
// copies of q and k and its dQ, dK are turned back afterwards).  The chain rule through X_{i+1} = A_i X_i (the paper gives
// no backward), block by block as in the long-segment forward:
//
//     P_ij  = exp2(S_ij * scale * log2 e - lse_i)          S_ij = Q_i K_j^T,  lse_i from the statistics pass
//     dP_ij = G_i X_j^T,   dS_ij = P_ij o (dP_ij - delta_i) * scale,   delta_i = <G_i, O_i> row by row
//     Gin_j += P_ij^T G_i        dK_j += dS_ij^T Q_i        dQ_i += dS_ij K_j
//
// A work item is one block of 128 key positions of one segment and KV head.  It walks the query
// heads of the GQA group and, per head, the query tiles that can see the block (all of them, or
// those at and after it when causal); per (head, query tile) the five MMAs, shared-memory slots
// and the load / compute overlap are those of the short-segment backward kernel (ta_tc_bwd.cu).
// Gin_j accumulates in tensor memory over the query tiles of a head and leaves as bf16 once per
// head (first hop: it is dV and accumulates over the whole group); dK_j accumulates over the whole
// item; dQ_i is added to the fp32 buffer in global memory by TMA reduce-add, because every key
// block contributes to it (the buffer is cleared by the host if this is the first hop processed;
// the order of those adds is not fixed, so dQ is reproducible only up to fp32 summation order).
// Row statistics (lse_i, delta_i) come from launch_hop_tc_long_stats.
// Every wait is bounded; on expiry the CTA raises a flag, lets its copies land, frees its TMEM
// and returns.
#include <cuda_bf16.h>

#include "ta_internal.h"
#include "ta_ptx.cuh"

namespace ta {
namespace {

constexpr int kTileRows = 128;
constexpr int kThreads = 160;          // 4 compute warps + the producer warp

struct LongBwdArgs {
    int n, causal, g, H, H_kv, x_is_kv, first_hop, accumulate_dk, N;
    int nblocks;                       // ceil(n / 128): key blocks = query tiles of a segment
    long long stride, outer, total_items;
    float scale_log2, scale;
    const float2 *stats;               // [B*H][N]: (lse in the log2 domain, delta)
    int window;                        // 0, or sliding window along the hop's dimension
    const int *lens;                   // device, valid length per batch entry, or nullptr
    int gi, hsplit;                    // query heads per item, items per (key block, KV head): gi * hsplit == g
};

template <int D>
struct LongBwdCfg {
    static constexpr int kHalves = D / 64;
    static constexpr uint32_t kSlabBytes = kTileRows * 128;          // [128 rows][128 bytes]
    static constexpr uint32_t kTileBytes = kHalves * kSlabBytes;     // one bf16 operand tile
    static constexpr uint32_t kPBytes = 2 * kSlabBytes;              // 128 x 128 bf16
    static constexpr uint32_t kStageBytes = 2 * kTileBytes;          // {Q, G} of one step = one fp32 output tile
    static constexpr uint32_t kOffK = 0;
    static constexpr uint32_t kOffStage = kOffK + kTileBytes;        // 2 stages
    static constexpr uint32_t kOffXP = kOffStage + 2 * kStageBytes;  // X, then P
    static constexpr uint32_t kOffDS = kOffXP + kPBytes;             // dS, then the bf16 Gin staging
    static constexpr uint32_t kOffBar = kOffDS + kPBytes;
    static constexpr int kNumBars = 10;
    static constexpr uint32_t kSmemBytes = kOffBar + kNumBars * 8 + 16 + 1024;
    static constexpr uint32_t kTmemCols = 512;
    // S | dP then dQ | dK of the item | Gin of the head (first hop: dV of the item)
    static constexpr uint32_t kColS = 0, kColDP = 128, kColDK = 256, kColG = 384;
};

struct LongBwdItem {
    int jb, inner, outer, kv_head, q_head0;
    int i_lo, steps_per_head;          // query tiles [i_lo, i_lo + steps_per_head) can see this key block
    int exist;                         // positions of the segment that are tokens (n without valid lengths)
};
__device__ __forceinline__ LongBwdItem decode_item(const LongBwdArgs &a, long long item) {
    LongBwdItem c;
    // Items are numbered with the key block slowest: when causal, block 0 meets every query tile and
    // the last block one, so the numbering runs from the longest items to the shortest (see
    // item_of_round for how they are dealt to the CTAs).
    const long long per_block = a.total_items / a.nblocks;
    c.jb = (int)(item / per_block);
    long long rest = item % per_block;
    const int hs = (int)(rest % a.hsplit); rest /= a.hsplit;       // which of the group's head chunks
    c.inner = (int)(rest % a.stride); rest /= a.stride;
    c.outer = (int)(rest % a.outer); rest /= a.outer;
    c.kv_head = (int)rest;
    c.q_head0 = (c.kv_head / a.H_kv) * a.H + (c.kv_head % a.H_kv) * a.g + hs * a.gi;
    c.i_lo = a.causal ? c.jb : 0;
    int i_hi = a.nblocks - 1;
    if (a.window > 0) {                // tiles with a row within the window of one of the block's keys
        const int u0 = kTileRows * c.jb, u1 = min(a.n, u0 + kTileRows) - 1;
        if (!a.causal) c.i_lo = max(0, u0 - a.window + 1) / kTileRows;
        i_hi = min(i_hi, (u1 + a.window - 1) / kTileRows);
    }
    c.steps_per_head = i_hi - c.i_lo + 1;
    c.exist = a.n;
    if (a.lens != nullptr) {
        const long long len = min(max(__ldg(a.lens + c.kv_head / a.H_kv), 0), a.N);
        const long long first_token = (long long)c.outer * a.n * a.stride + c.inner;
        const long long left = (len - first_token + a.stride - 1) / a.stride;
        c.exist = len <= first_token ? 0 : (int)(left < a.n ? left : a.n);
    }
    return c;
}

// The item a CTA takes in its k-th round: the rounds run forth and back over the CTAs, so that the
// CTA that got the longest item of one round gets the shortest of the next (items are numbered
// longest first).  -1: none in this round.
__device__ __forceinline__ long long item_of_round(const LongBwdArgs &a, long long k) {
    const long long g = gridDim.x, b = blockIdx.x;
    const long long item = k * g + ((k & 1) ? g - 1 - b : b);
    return item < a.total_items ? item : -1;
}

__device__ __forceinline__ bool wg_all(bool pred) {
    uint32_t r;
    asm volatile(
        "{\n .reg .pred p, q;\n setp.ne.b32 q, %1, 0;\n bar.red.and.pred p, 1, 128, q;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(r)
        : "r"((uint32_t)pred)
        : "memory");
    return r != 0;
}
__device__ __forceinline__ void wg_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
hop_tc_bwd_long_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                       const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_gin,
                       const __grid_constant__ CUtensorMap map_gout, const __grid_constant__ CUtensorMap map_dq,
                       const __grid_constant__ CUtensorMap map_dk, const __grid_constant__ CUtensorMap map_dv,
                       const LongBwdArgs a) {
    using C = LongBwdCfg<D>;
    constexpr int kHalves = C::kHalves;
    constexpr uint32_t kSlabBytes = C::kSlabBytes, kTileBytes = C::kTileBytes, kStageBytes = C::kStageBytes;
    constexpr uint32_t kTileTx = kHalves * kSlabBytes;               // bytes of one bf16 tile load

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t s0 = smem_u32(smem);
    const uint32_t sK = s0 + C::kOffK, sXP = s0 + C::kOffXP, sdS = s0 + C::kOffDS;
    auto sQ = [&](int s) { return s0 + C::kOffStage + (uint32_t)s * kStageBytes; };
    auto sG = [&](int s) { return s0 + C::kOffStage + (uint32_t)s * kStageBytes + kTileBytes; };
    const uint32_t bar0 = s0 + C::kOffBar;
    const uint32_t k_full = bar0, k_free = bar0 + 8, x_full = bar0 + 48, xp_free = bar0 + 56, s_done = bar0 + 64,
                   o_done = bar0 + 72;
    auto qg_full = [&](int s) { return bar0 + 16u + 8u * (uint32_t)s; };
    auto qg_free = [&](int s) { return bar0 + 32u + 8u * (uint32_t)s; };
    uint32_t *tmem_slot = (uint32_t *)(smem + C::kOffBar + C::kNumBars * 8);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    for (uint32_t i = tid; i < C::kOffBar / 16; i += blockDim.x) ((uint4 *)smem)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) {
        for (int i = 0; i < C::kNumBars; ++i) mbar_init(bar0 + 8u * (uint32_t)i, 1);
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
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

    if (warp == 4) {
        // =============================================================== TMA producer
        if (lane == 0) {
            uint32_t t = 0, it = 0;
            bool ok = true;
            uint32_t armed = 0, last_par = 0;        // bits: 0 k, 1-2 qg, 3 x
            auto arm = [&](uint32_t bit, uint32_t parity) {
                armed |= bit;
                last_par = parity ? (last_par | bit) : (last_par & ~bit);
            };
            for (long long round = 0; ok && round * gridDim.x < a.total_items; ++round) {
                const long long item = item_of_round(a, round);
                if (item < 0) continue;
                const LongBwdItem c = decode_item(a, item);
                const int steps = a.gi * c.steps_per_head;
                for (int v = 0; v < steps; ++v, ++t) {
                    const int q_head = c.q_head0 + v / c.steps_per_head;
                    const int qi = c.i_lo + v % c.steps_per_head;
                    const int x_head = a.x_is_kv ? c.kv_head : q_head;
                    const int s = t & 1;
                    const uint32_t par = (t >> 1) & 1;
                    ok = mbar_wait_abortable(qg_free(s), par ^ 1, 0x60, abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(qg_full(s), 2 * kTileTx);
                    arm(2u << s, par);
#pragma unroll
                    for (int h = 0; h < kHalves; ++h)
                        tma_load_5d(sQ(s) + h * kSlabBytes, &map_q, qg_full(s), 64 * h, kTileRows * qi, c.inner, c.outer, q_head);
#pragma unroll
                    for (int h = 0; h < kHalves; ++h)
                        tma_load_5d(sG(s) + h * kSlabBytes, &map_gin, qg_full(s), 64 * h, kTileRows * qi, c.inner, c.outer, q_head);
                    if (v == 0) {
                        ok = mbar_wait_abortable(k_free, (it & 1) ^ 1, 0x61, abort_flag);
                        if (!ok) break;
                        mbar_expect_tx(k_full, kTileTx);
                        arm(1u, it & 1);
#pragma unroll
                        for (int h = 0; h < kHalves; ++h)
                            tma_load_5d(sK + h * kSlabBytes, &map_k, k_full, 64 * h, kTileRows * c.jb, c.inner, c.outer, c.kv_head);
                    }
                    ok = mbar_wait_abortable(xp_free, (t & 1) ^ 1, 0x62, abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(x_full, kTileTx);
                    arm(8u, t & 1);
#pragma unroll
                    for (int h = 0; h < kHalves; ++h)
                        tma_load_5d(sXP + h * kSlabBytes, &map_x, x_full, 64 * h, kTileRows * c.jb, c.inner, c.outer, x_head);
                }
                ++it;
            }
            if (!ok) {
                const unsigned long long t0 = globaltimer_ns();
                for (int b = 0; b < 4; ++b) {
                    if (!(armed & (1u << b))) continue;
                    const uint32_t bar = b == 0 ? k_full : (b == 3 ? x_full : qg_full(b - 1));
                    while (!mbar_try_wait(bar, (last_par >> b) & 1u) && globaltimer_ns() - t0 < 10000000ull) {
                    }
                }
            }
        }
    } else if (warp < 4) {
        // =============================================================== compute warps
        const uint32_t tmem_lane = tmem_base + ((uint32_t)(warp * 32) << 16);
        constexpr uint32_t idesc_s = instr_desc(128, 0, 0);        // A, B K-major, N = 128
        constexpr uint32_t idesc_g = instr_desc(D, 1, 1);          // A = P^T / dS^T (MN-major), B MN-major
        constexpr uint32_t idesc_dq = instr_desc(D, 1, 0);         // A = dS K-major, B MN-major
        const int r = warp * 32 + lane;                            // this thread's row of the query tile
        constexpr int kblocks = kTileRows / 16;                    // rows past n are zero in every operand

        // fp32 accumulator columns -> shared staging in the layout of the fp32 maps (32-column slabs)
        auto stage_f32 = [&](uint32_t col0, uint32_t stage) {
            uint32_t v[32];
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
                tmem_ld32(tmem_lane + col0 + 32 * c, v);
                const uint32_t row = stage + (uint32_t)c * kSlabBytes + (uint32_t)r * 128u;
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    st_shared_v4(row + (uint32_t)((i ^ (r & 7)) * 16), v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
            }
        };

        uint32_t t = 0, it = 0;
        bool ok = true;
        int pending_stage = -1;   // thread 0: stage whose output stores have been issued but not yet read out
        for (long long round = 0; ok && round * gridDim.x < a.total_items; ++round, ++it) {
            const long long item = item_of_round(a, round);
            if (item < 0) { --it; continue; }
            const LongBwdItem c = decode_item(a, item);
            const int steps = a.gi * c.steps_per_head;
            // key positions of the block that are tokens (none: every weight is 0 and the item writes zeros)
            const int keys = max(0, min(kTileRows, min(a.n, c.exist) - kTileRows * c.jb));
            for (int v = 0; v < steps; ++v, ++t) {
                const int s = t & 1;
                const uint32_t par = t & 1;
                const int hh = v / c.steps_per_head, qstep = v % c.steps_per_head;
                const int q_head = c.q_head0 + hh;
                const int qi = c.i_lo + qstep;
                const bool head_first = qstep == 0, head_last = qstep == c.steps_per_head - 1;
                const bool item_last = v == steps - 1;
                const uint32_t q_base = sQ(s), g_base = sG(s);

                // ---- S = Q K^T and dP = G X^T
                if (tid == 0) {
                    bool k0 = true;
                    if (v == 0) k0 = mbar_wait_abortable(k_full, it & 1, 0x71, abort_flag);
                    if (k0) k0 = mbar_wait_abortable(qg_full(s), (t >> 1) & 1, 0x72, abort_flag);
                    if (k0) {
                        tc_fence_after();
#pragma unroll
                        for (int kb = 0; kb < D / 16; ++kb) {
                            const uint32_t off = (kb >> 2) * kSlabBytes + (kb & 3) * 32;
                            tc_mma_ss(tmem_base + C::kColS, smem_desc_sw128(q_base + off, 16, 1024),
                                      smem_desc_sw128(sK + off, 16, 1024), idesc_s, kb > 0);
                        }
                        k0 = mbar_wait_abortable(x_full, par, 0x73, abort_flag);
                    }
                    if (k0) {
                        tc_fence_after();
#pragma unroll
                        for (int kb = 0; kb < D / 16; ++kb) {
                            const uint32_t off = (kb >> 2) * kSlabBytes + (kb & 3) * 32;
                            tc_mma_ss(tmem_base + C::kColDP, smem_desc_sw128(g_base + off, 16, 1024),
                                      smem_desc_sw128(sXP + off, 16, 1024), idesc_s, kb > 0);
                        }
                        tc_commit(s_done);
                    }
                    if (pending_stage >= 0) {
                        // the previous step's stores overlap this step's score MMAs; their staging
                        // space (that stage and the dS slot) is needed again only from here on
                        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                        mbar_arrive(qg_free(pending_stage));
                        pending_stage = -1;
                    }
                    ok = k0;
                }
                __syncwarp();
                if (ok) ok = mbar_wait_abortable(s_done, par, 0x74, abort_flag);
                ok = wg_all(ok);
                if (!ok) break;
                tc_fence_after();

                // ---- P and dS of this thread's query row from its statistics; P -> X slot, dS -> its slot
                {
                    const int tq = kTileRows * qi + r;                       // position of the row in the segment
                    const bool row_in = tq < min(a.n, c.exist);
                    float2 st = make_float2(INFINITY, 0.f);
                    if (row_in)
                        st = __ldg(a.stats + (long long)q_head * a.N + ((long long)c.outer * a.n + tq) * a.stride + c.inner);
                    // key columns this row sees in the block: [c_lo, c_hi)
                    int c_hi = !row_in ? 0 : ((a.causal && qi == c.jb) ? min(keys, r + 1) : keys);
                    int c_lo = 0;
                    if (a.window > 0) {
                        const int u0 = kTileRows * c.jb;
                        c_lo = max(0, tq - a.window + 1 - u0);
                        if (!a.causal) c_hi = min(c_hi, tq + a.window - u0);
                    }
                    const uint32_t rowP = sXP + (uint32_t)r * 128u, rowS = sdS + (uint32_t)r * 128u;
                    uint32_t vs[32], vd[32];
#pragma unroll 1
                    for (int cc = 0; cc < 4; ++cc) {
                        uint32_t pp[16], ps[16];
                        tmem_ld32(tmem_lane + C::kColS + 32 * cc, vs);
                        tmem_ld32(tmem_lane + C::kColDP + 32 * cc, vd);
#pragma unroll
                        for (int jj = 0; jj < 32; jj += 2) {
                            float pv[2], dv[2];
#pragma unroll
                            for (int e = 0; e < 2; ++e) {
                                const bool vis = 32 * cc + jj + e >= c_lo && 32 * cc + jj + e < c_hi;
                                float p = fast_exp2(__uint_as_float(vs[jj + e]) * a.scale_log2 - st.x);
                                p = vis ? p : 0.f;
                                pv[e] = p;
                                dv[e] = vis ? p * (__uint_as_float(vd[jj + e]) - st.y) * a.scale : 0.f;
                            }
                            pp[jj >> 1] = pack_bf16x2(pv[0], pv[1]);
                            ps[jj >> 1] = pack_bf16x2(dv[0], dv[1]);
                        }
                        const uint32_t slab = (uint32_t)(cc >> 1) * kSlabBytes;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const uint32_t chunk = (uint32_t)(((cc & 1) * 4 + i) ^ (r & 7)) * 16;
                            st_shared_v4(rowP + slab + chunk, pp[4 * i], pp[4 * i + 1], pp[4 * i + 2], pp[4 * i + 3]);
                            st_shared_v4(rowS + slab + chunk, ps[4 * i], ps[4 * i + 1], ps[4 * i + 2], ps[4 * i + 3]);
                        }
                    }
                }
                fence_proxy_async_smem();
                tc_fence_before();
                wg_sync();

                // ---- Gin += P^T G (first hop: dV), dQ = dS K, dK += dS^T Q
                if (tid == 0) {
                    tc_fence_after();
                    for (int kb = 0; kb < kblocks; ++kb) {
                        const uint32_t k_off = kb * 2048;                                  // 16 rows of 128 bytes
                        const uint32_t a_off = (kb >> 2) * kSlabBytes + (kb & 3) * 32;     // 16 columns of a K-major tile
                        // Gin[key, d] += sum_q P[q, key] G[q, d]   (over the query tiles of the head;
                        // in the first hop over the whole item: dV)
                        tc_mma_ss(tmem_base + C::kColG, smem_desc_sw128(sXP + k_off, kSlabBytes, 1024),
                                  smem_desc_sw128(g_base + k_off, kSlabBytes, 1024), idesc_g,
                                  (kb > 0 || !(a.first_hop ? v == 0 : head_first)) ? 1u : 0u);
                        // dQ[q, d] = sum_key dS[q, key] K[key, d]
                        tc_mma_ss(tmem_base + C::kColDP, smem_desc_sw128(sdS + a_off, 16, 1024),
                                  smem_desc_sw128(sK + k_off, kSlabBytes, 1024), idesc_dq, kb > 0);
                        // dK[key, d] += sum_q dS[q, key] Q[q, d]   (over the whole item)
                        tc_mma_ss(tmem_base + C::kColDK, smem_desc_sw128(sdS + k_off, kSlabBytes, 1024),
                                  smem_desc_sw128(q_base + k_off, kSlabBytes, 1024), idesc_g,
                                  (kb > 0 || v > 0) ? 1u : 0u);
                    }
                    tc_commit(o_done);
                    tc_commit(xp_free);                // the X / P slot may take the next step's X
                    if (item_last) tc_commit(k_free);
                }
                __syncwarp();
                ok = mbar_wait_abortable(o_done, par, 0x75, abort_flag);
                ok = wg_all(ok);
                if (!ok) break;
                tc_fence_after();

                // ---- epilogue: dQ (fp32, over this step's Q and G tiles); at a head's last query tile
                // also its Gin (bf16, over dS)
                stage_f32(C::kColDP, q_base);
                const bool write_gin = !a.first_hop && head_last;
                if (write_gin) {
                    uint32_t vv[32];
#pragma unroll 1
                    for (int cc = 0; cc < D / 32; ++cc) {
                        tmem_ld32(tmem_lane + C::kColG + 32 * cc, vv);
                        uint32_t pk[16];
#pragma unroll
                        for (int jj = 0; jj < 32; jj += 2)
                            pk[jj >> 1] = pack_bf16x2(__uint_as_float(vv[jj]), __uint_as_float(vv[jj + 1]));
                        const uint32_t row = sdS + (uint32_t)(cc >> 1) * kSlabBytes + (uint32_t)r * 128u;
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            st_shared_v4(row + (uint32_t)((((cc & 1) * 4 + i) ^ (r & 7)) * 16), pk[4 * i], pk[4 * i + 1],
                                         pk[4 * i + 2], pk[4 * i + 3]);
                    }
                }
                fence_proxy_async_smem();
                tc_fence_before();
                wg_sync();
                if (tid == 0) {
#pragma unroll
                    for (int sl = 0; sl < D / 32; ++sl)
                        tma_reduce_add_5d(&map_dq, q_base + sl * kSlabBytes, 32 * sl, kTileRows * qi, c.inner, c.outer, q_head);
                    if (write_gin) {
#pragma unroll
                        for (int h = 0; h < kHalves; ++h)
                            tma_store_5d(&map_gout, sdS + h * kSlabBytes, 64 * h, kTileRows * c.jb, c.inner, c.outer, q_head);
                    }
                    if (item_last) tma_store_commit_and_wait_read();   // the staging space is reused right below
                    else asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
                if (item_last) {
                    // ---- once per item: dK (and, in the first hop, dV) of the key block
                    wg_sync();                         // the staging space has been read out
                    tc_fence_after();
                    stage_f32(C::kColDK, q_base);
                    fence_proxy_async_smem();
                    tc_fence_before();
                    wg_sync();
                    if (tid == 0) {
#pragma unroll
                        for (int sl = 0; sl < D / 32; ++sl) {
                            if (a.accumulate_dk)
                                tma_reduce_add_5d(&map_dk, q_base + sl * kSlabBytes, 32 * sl, kTileRows * c.jb, c.inner, c.outer, c.kv_head);
                            else
                                tma_store_5d(&map_dk, q_base + sl * kSlabBytes, 32 * sl, kTileRows * c.jb, c.inner, c.outer, c.kv_head);
                        }
                        tma_store_commit_and_wait_read();
                    }
                    if (a.first_hop) {
                        wg_sync();
                        tc_fence_after();
                        stage_f32(C::kColG, q_base);
                        fence_proxy_async_smem();
                        tc_fence_before();
                        wg_sync();
                        if (tid == 0) {
#pragma unroll
                            for (int sl = 0; sl < D / 32; ++sl) {
                                if (a.hsplit > 1)      // several items share the block: summed in global memory
                                    tma_reduce_add_5d(&map_dv, q_base + sl * kSlabBytes, 32 * sl, kTileRows * c.jb, c.inner, c.outer, c.kv_head);
                                else
                                    tma_store_5d(&map_dv, q_base + sl * kSlabBytes, 32 * sl, kTileRows * c.jb, c.inner, c.outer, c.kv_head);
                            }
                            tma_store_commit_and_wait_read();
                        }
                    }
                }
                if (tid == 0) {
                    if (item_last) mbar_arrive(qg_free(s));   // read out: this stage may take the step after next
                    else pending_stage = s;                   // handed back once the stores have been read
                }
            }
        }
        if (tid == 0) tma_store_wait_all();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::kTmemCols) : "memory");
    }
}

template <int D>
int launch_d(const Problem &pb, const HopDesc &hd, const void *x, int x_heads, const void *g_in, void *g_out,
             float *dq_acc, float *dk_acc, float *dv_acc, void *stats, bool first_hop, bool accumulate) {
    // row statistics of the hop: (lse, <G, O>) per query row
    int rc = launch_hop_tc_long_stats(pb, hd, x, x_heads, g_in, stats);
    if (rc != TA_OK) return rc;
    const size_t tq = (size_t)pb.B * pb.H * pb.N * pb.D;
    // dQ is reduce-added by every key block: the first hop processed starts from zeros
    if (!accumulate && cudaMemsetAsync(dq_acc, 0, tq * sizeof(float), pb.stream) != cudaSuccess)
        return cuda_fail(cudaPeekAtLastError());

    CUtensorMap mq, mk, mx, mgi, mgo, mdq, mdk, mdv;
    // box: 128 positions of one segment (positions past n are zero-filled on load, clipped on store)
    if ((rc = make_view_map(&mq, pb.q, pb.B * pb.H, pb.N, D, hd, 2, kTileRows, 1, 1)) != TA_OK) return rc;
    if ((rc = make_view_map(&mk, pb.k, pb.B * pb.H_kv, pb.N, D, hd, 2, kTileRows, 1, 1)) != TA_OK) return rc;
    if ((rc = make_view_map(&mx, x, pb.B * x_heads, pb.N, D, hd, 2, kTileRows, 1, 1)) != TA_OK) return rc;
    if ((rc = make_view_map(&mgi, g_in, pb.B * pb.H, pb.N, D, hd, 2, kTileRows, 1, 1)) != TA_OK) return rc;
    if ((rc = make_view_map(&mgo, g_out ? g_out : g_in, pb.B * pb.H, pb.N, D, hd, 2, kTileRows, 1, 1)) != TA_OK) return rc;
    if ((rc = make_view_map(&mdq, dq_acc, pb.B * pb.H, pb.N, D, hd, 4, kTileRows, 1, 1)) != TA_OK) return rc;
    if ((rc = make_view_map(&mdk, dk_acc, pb.B * pb.H_kv, pb.N, D, hd, 4, kTileRows, 1, 1)) != TA_OK) return rc;
    if ((rc = make_view_map(&mdv, dv_acc, pb.B * pb.H_kv, pb.N, D, hd, 4, kTileRows, 1, 1)) != TA_OK) return rc;

    LongBwdArgs a;
    a.n = hd.n; a.causal = pb.causal; a.g = pb.H / pb.H_kv; a.H = pb.H; a.H_kv = pb.H_kv;
    a.x_is_kv = x_heads != pb.H ? 1 : 0;
    a.first_hop = first_hop ? 1 : 0;
    a.accumulate_dk = accumulate ? 1 : 0;      // (forced below when the heads of a group are split over items)
    a.N = pb.N;
    a.nblocks = (hd.n + kTileRows - 1) / kTileRows;
    a.stride = hd.stride; a.outer = hd.outer;
    int dev = 0;
    const int num_sms = current_device_sms(&dev);
    // the query heads of a group are split over several items when there are too few items to fill
    // the GPU; their dK (and dV) are then summed in global memory by reduce-adds into cleared buffers
    const long long blocks_total = (long long)pb.B * pb.H_kv * hd.outer * hd.stride * a.nblocks;
    a.hsplit = 1;
    for (int d = 2; d <= a.g && blocks_total * a.hsplit < 4ll * num_sms; ++d)
        if (a.g % d == 0) a.hsplit = d;
    a.gi = a.g / a.hsplit;
    a.total_items = blocks_total * a.hsplit;
    const size_t tkv = (size_t)pb.B * pb.H_kv * pb.N * pb.D;
    if (a.hsplit > 1) {
        if (!accumulate && cudaMemsetAsync(dk_acc, 0, tkv * sizeof(float), pb.stream) != cudaSuccess)
            return cuda_fail(cudaPeekAtLastError());
        if (first_hop && cudaMemsetAsync(dv_acc, 0, tkv * sizeof(float), pb.stream) != cudaSuccess)
            return cuda_fail(cudaPeekAtLastError());
    }
    a.scale = pb.scale;
    a.scale_log2 = pb.scale * 1.4426950408889634f;
    a.stats = (const float2 *)stats;
    a.window = pb.window[hd.hop];
    a.lens = pb.seq_lens;

    if (a.hsplit > 1) a.accumulate_dk = 1;
    constexpr size_t smem = LongBwdCfg<D>::kSmemBytes;
    static PerDeviceOnce configured;
    if (!configured.is_done(dev)) {
        if (cudaFuncSetAttribute(hop_tc_bwd_long_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
            cudaSuccess)
            return cuda_fail(cudaPeekAtLastError());
        configured.mark(dev);
    }
    const unsigned grid = (unsigned)(a.total_items < num_sms ? a.total_items : num_sms);
    return launch_kernel(hop_tc_bwd_long_kernel<D>, grid, kThreads, smem, pb.stream, false, mq, mk, mx, mgi, mgo, mdq, mdk,
                         mdv, a);
}

}  // namespace

// Conditions under which this kernel takes a long-segment hop (else the generic backward does).
bool tc_bwd_long_eligible(const Problem &pb, const HopDesc &hd) {
    return hd.path == PATH_TC_LONG && pb.dtype == TA_DTYPE_BF16 && (pb.D == 64 || pb.D == 128) &&
           pb.masks[hd.hop] == nullptr;
}

int launch_hop_tc_bwd_long(const Problem &pb, const HopDesc &hd, const void *x, int x_heads, const void *g_in,
                           void *g_out, float *dq_acc, float *dk_acc, float *dv_acc, void *stats, bool first_hop,
                           bool accumulate) {
    if (!tc_bwd_long_eligible(pb, hd)) return TA_ERR_UNSUPPORTED;
    if (!first_hop && (g_out == nullptr || g_out == g_in)) return TA_ERR_INVALID_ARG;   // other items read g_in
    if (pb.rope_base > 0.f) {
        // Positional encoding: the hop runs on rotated copies of q and k (as in the forward); its dQ
        // and dK are gradients with respect to the rotated vectors, so they go to scratch of their own
        // and are turned back (R^T) while they are stored in / added to the accumulators.
        const size_t tq = (size_t)pb.B * pb.H * pb.N * pb.D, tkv = (size_t)pb.B * pb.H_kv * pb.N * pb.D;
        Problem hop = pb;
        void *extra = nullptr, *pooled = nullptr;
        int rc = rope_rotated_copies(pb, hd, &hop.q, &hop.k, (tq + tkv) * sizeof(float), &extra, &pooled);
        if (rc == TA_OK) {
            hop.rope_base = 0.f;
            float *dq_rot = (float *)extra, *dk_rot = dq_rot + tq;
            rc = pb.D == 128
                     ? launch_d<128>(hop, hd, x, x_heads, g_in, g_out, dq_rot, dk_rot, dv_acc, stats, first_hop, false)
                     : launch_d<64>(hop, hd, x, x_heads, g_in, g_out, dq_rot, dk_rot, dv_acc, stats, first_hop, false);
            if (rc == TA_OK) rc = rope_unrotate_add(pb, hd, dq_rot, dq_acc, pb.H, accumulate);
            if (rc == TA_OK) rc = rope_unrotate_add(pb, hd, dk_rot, dk_acc, pb.H_kv, accumulate);
        }
        pool_free(pooled, pb.stream);
        return rc;
    }
    if (pb.D == 128)
        return launch_d<128>(pb, hd, x, x_heads, g_in, g_out, dq_acc, dk_acc, dv_acc, stats, first_hop, accumulate);
    return launch_d<64>(pb, hd, x, x_heads, g_in, g_out, dq_acc, dk_acc, dv_acc, stats, first_hop, accumulate);
}

int read_status_tc_backward_long(unsigned int *word) {
    if (cudaMemcpyFromSymbol(word, g_status_word, sizeof(*word)) != cudaSuccess) return TA_ERR_CUDA;
    if (*word != 0) {
        unsigned int z = 0;
        cudaMemcpyToSymbol(g_status_word, &z, sizeof(z));
    }
    return TA_OK;
}

}  // namespace ta
