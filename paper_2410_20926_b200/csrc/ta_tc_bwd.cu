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
// forward kernel.  A work item is one tile position of one KV head; the H/H_kv query heads of
// the group are processed in turn against the same K tile, and their dK (and, in the first
// hop, dV = G_0) contributions are summed in tensor memory and leave the SM once per item.
// Per head: two MMAs into TMEM (S = Q K^T, dP = G X^T), the softmax and its derivative in
// registers, P (over the X tile, dead by then) and dS (bf16) to shared memory, then three
// MMAs: G_i (A = P as an MN-major operand, i.e. P^T; over the S columns), dQ (A = dS K-major;
// over the dP columns) and dK (A = dS MN-major).  dQ and dK go to fp32 buffers in global
// memory -- plain TMA stores in the first hop processed, TMA reduce-add afterwards (they sum
// over hops) -- and G_i is carried to the next hop as bf16, in place.
//
// Persistent, one CTA per SM.  Warps 0-3 compute (thread 0 issues the MMAs and the stores);
// warp 4 issues the TMA loads: Q and G of the next head land in a second stage while the
// current head computes, X and K as soon as the MMAs that read their slots have completed, so
// that loads overlap the epilogue.  With the tensorized positional encoding (Section 3.2, per-hop
// RoPE; template parameter kRope) warps 5-12 rotate the K and Q tiles in place in shared memory
// before thread 0 sees them, exactly as in the forward kernel, and the epilogue turns dQ and dK --
// gradients with respect to the rotated vectors -- back by the transposed rotation before they
// leave the SM.  Every wait is bounded; when one expires the CTA raises a
// flag that ends both roles, lets its copies land, frees its TMEM and returns.
#include <cuda_bf16.h>

#include <cstring>

#include "ta_internal.h"
#include "ta_ptx.cuh"
#include "ta_rope.cuh"
#include "ta_mask.cuh"

namespace ta {
namespace {

constexpr int kTileRows = 128;
constexpr int kThreads = 160;          // + the producer warp
constexpr int kThreadsRope = 416;      // + two warpgroups that rotate Q and K tiles

struct BwdArgs {
    int n, rows, ci, co, causal, g, H, H_kv, x_is_kv, first_hop;
    int accumulate;                    // 0: dQ / dK are stored (first hop processed), 1: reduce-added
    int window;                        // 0, or sliding window along the hop's dimension
    long long tiles_inner, tiles_outer, total_items;
    float scale_log2, scale;
    float rope_log2_base;              // log2 of the RoPE base (rotating variant only)
    int stride;                        // token stride of the hop's dimension
    const int *lens;                   // device, valid length per batch entry, or nullptr (masked variant only)
    const uint32_t *dmask;             // masked variant, masks that differ per head: [H][n][4] words in device
                                       // memory (causal flag and window folded in); nullptr: the kernel parameter
};

template <int D>
struct BwdCfg {
    static constexpr int kHalves = D / 64;
    static constexpr uint32_t kSlabBytes = kTileRows * 128;          // [128 rows][128 bytes]
    static constexpr uint32_t kTileBytes = kHalves * kSlabBytes;     // one bf16 operand tile
    static constexpr uint32_t kPBytes = 2 * kSlabBytes;              // 128 x 128 bf16
    static constexpr uint32_t kStageBytes = 2 * kTileBytes;          // {Q, G} of one head = one fp32 output tile
    static constexpr uint32_t kOffK = 0;
    static constexpr uint32_t kOffStage = kOffK + kTileBytes;        // 2 stages
    static constexpr uint32_t kOffXP = kOffStage + 2 * kStageBytes;  // X, then P
    static constexpr uint32_t kOffDS = kOffXP + kPBytes;             // dS, then the bf16 G_i staging
    static constexpr uint32_t kOffBar = kOffDS + kPBytes;
    static constexpr int kNumBars = 13;
    static constexpr uint32_t kOffTheta = kOffBar + kNumBars * 8 + 16;   // D/2 RoPE frequencies (fp32)
    static constexpr uint32_t kSmemBytes = kOffTheta + 64 * 4 + 1024;
    static constexpr uint32_t kTmemCols = 512;
    // S then G_i | dP then dQ | dK summed over the group | dV summed over the group (first hop)
    static constexpr uint32_t kColS = 0, kColDP = 128, kColDK = 256, kColDV = 384;
};

struct BwdItem {
    int c_inner, c_outer, kv_head, q_head0;
};
__device__ __forceinline__ BwdItem decode_bwd_item(const BwdArgs &a, long long item) {
    BwdItem c;
    long long rest = item;
    c.c_inner = (int)(rest % a.tiles_inner) * a.ci; rest /= a.tiles_inner;
    c.c_outer = (int)(rest % a.tiles_outer) * a.co; rest /= a.tiles_outer;
    c.kv_head = (int)rest;
    c.q_head0 = (c.kv_head / a.H_kv) * a.H + (c.kv_head % a.H_kv) * a.g;
    return c;
}

// barrier + AND over the 128 compute threads (named barrier 1)
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

template <int D, bool kRope, bool kMask>
__global__ void __launch_bounds__(kRope ? kThreadsRope : kThreads, 1)
hop_tc_bwd_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_gin,
                  const __grid_constant__ CUtensorMap map_gout, const __grid_constant__ CUtensorMap map_dq,
                  const __grid_constant__ CUtensorMap map_dk, const __grid_constant__ CUtensorMap map_dv,
                  const BwdArgs a, const __grid_constant__ typename MaskArg<kMask>::type hop_mask) {
    using C = BwdCfg<D>;
    constexpr int kHalves = C::kHalves;
    constexpr uint32_t kSlabBytes = C::kSlabBytes, kTileBytes = C::kTileBytes, kStageBytes = C::kStageBytes;

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
    const uint32_t k_rot = bar0 + 80;                                // rotated K ready (8 warps)
    auto q_rot = [&](int s) { return bar0 + 88u + 8u * (uint32_t)s; };   // rotated Q of stage s ready
    float *theta_tab = (float *)(smem + C::kOffTheta);
    uint32_t *tmem_slot = (uint32_t *)(smem + C::kOffBar + C::kNumBars * 8);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    for (uint32_t i = tid; i < C::kOffBar / 16; i += blockDim.x) ((uint4 *)smem)[i] = make_uint4(0, 0, 0, 0);
    if (kRope && tid < D / 2) theta_tab[tid] = exp2f(-2.f * (float)tid / (float)D * a.rope_log2_base);
    if (tid == 0) {
        for (int i = 0; i < C::kNumBars; ++i) mbar_init(bar0 + 8u * (uint32_t)i, i >= 10 ? 8 : 1);
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
    const uint32_t slab_tx = (uint32_t)a.rows * 128u;

    if (warp == 4) {
        // =============================================================== TMA producer
        if (lane == 0) {
            uint32_t t = 0, it = 0;
            bool ok = true;
            // phases armed last on each barrier, for the drain on an early exit
            uint32_t armed = 0, last_par = 0;        // bits: 0 k, 1-2 qg, 3 x
            auto arm = [&](uint32_t bit, uint32_t parity) {
                armed |= bit;
                last_par = parity ? (last_par | bit) : (last_par & ~bit);
            };
            for (long long item = blockIdx.x; ok && item < a.total_items; item += gridDim.x, ++it) {
                const BwdItem c = decode_bwd_item(a, item);
                for (int j = 0; j < a.g; ++j, ++t) {
                    const int q_head = c.q_head0 + j;
                    const int x_head = a.x_is_kv ? c.kv_head : q_head;
                    const int s = t & 1;
                    const uint32_t par = (t >> 1) & 1;
                    ok = mbar_wait_abortable(qg_free(s), par ^ 1, 0x60, abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(qg_full(s), 2 * kHalves * slab_tx);
                    arm(2u << s, par);
#pragma unroll
                    for (int h = 0; h < kHalves; ++h)
                        tma_load_5d(sQ(s) + h * kSlabBytes, &map_q, qg_full(s), 64 * h, 0, c.c_inner, c.c_outer, q_head);
#pragma unroll
                    for (int h = 0; h < kHalves; ++h)
                        tma_load_5d(sG(s) + h * kSlabBytes, &map_gin, qg_full(s), 64 * h, 0, c.c_inner, c.c_outer, q_head);
                    if (j == 0) {
                        ok = mbar_wait_abortable(k_free, (it & 1) ^ 1, 0x61, abort_flag);
                        if (!ok) break;
                        mbar_expect_tx(k_full, kHalves * slab_tx);
                        arm(1u, it & 1);
#pragma unroll
                        for (int h = 0; h < kHalves; ++h)
                            tma_load_5d(sK + h * kSlabBytes, &map_k, k_full, 64 * h, 0, c.c_inner, c.c_outer, c.kv_head);
                    }
                    ok = mbar_wait_abortable(xp_free, (t & 1) ^ 1, 0x62, abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(x_full, kHalves * slab_tx);
                    arm(8u, t & 1);
#pragma unroll
                    for (int h = 0; h < kHalves; ++h)
                        tma_load_5d(sXP + h * kSlabBytes, &map_x, x_full, 64 * h, 0, c.c_inner, c.c_outer, x_head);
                }
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
    } else if (kRope && warp >= 5) {
        // =============================================================== RoPE on the K and Q tiles
        // (the rotation shared with the forward kernel)
        RopeRotator<D> rot;
        rot.init(tid - 5 * 32, a.n, a.rows, a.rope_log2_base);
        bool ok = true;
        uint32_t t = 0, it = 0;
        for (long long item = blockIdx.x; ok && item < a.total_items; item += gridDim.x, ++it) {
            for (int j = 0; j < a.g; ++j, ++t) {
                const int s = t & 1;
                ok = mbar_wait_abortable(qg_full(s), (t >> 1) & 1, 0x68, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                rot.rotate(sQ(s));
                if (lane == 0) mbar_arrive(q_rot(s));
                if (j == 0) {
                    ok = mbar_wait_abortable(k_full, it & 1, 0x69, abort_flag);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    rot.rotate(sK);
                    if (lane == 0) mbar_arrive(k_rot);
                }
            }
        }
    } else if (warp < 4) {
        // =============================================================== compute warps
        const uint32_t tmem_lane = tmem_base + ((uint32_t)(warp * 32) << 16);
        constexpr uint32_t idesc_s = instr_desc(128, 0, 0);        // A, B K-major, N = 128
        constexpr uint32_t idesc_g = instr_desc(D, 1, 1);          // A = P^T / dS^T (MN-major), B MN-major
        constexpr uint32_t idesc_dq = instr_desc(D, 1, 0);         // A = dS K-major, B MN-major

        const int r = warp * 32 + lane;
        const int seg = r / a.n;
        const bool row_valid = r < a.rows;
        int c_lo = seg * a.n;
        int c_hi = a.causal ? r + 1 : c_lo + a.n;
        if (a.window > 0) {
            c_lo = max(c_lo, r - a.window + 1);
            if (!a.causal) c_hi = min(c_hi, r + a.window);
        }
        const int w_lo = ((warp * 32) / a.n) * a.n;
        int w_hi = min(a.rows, ((warp * 32 + 31) / a.n + 1) * a.n);
        if (a.causal) w_hi = min(w_hi, warp * 32 + 32);
        const bool warp_valid = warp * 32 < a.rows;
        // explicit mask (already combined with the causal flag and the window): this row's bits
        // over the tile's key columns
        uint32_t mrow[4];
        tile_row_mask(hop_mask, row_valid ? r % a.n : 0, seg * a.n, mrow);
        if (kMask && !row_valid) mrow[0] = mrow[1] = mrow[2] = mrow[3] = 0u;
        uint32_t mt[4] = {mrow[0], mrow[1], mrow[2], mrow[3]};   // ... and below the batch entry's valid length
        auto visible = [&](int cc, int jj) -> bool {
            if (kMask) return ((mask_chunk(mt, cc) >> jj) & 1u) != 0;
            const int col = 32 * cc + jj;
            return row_valid && col >= c_lo && col < c_hi;
        };
        const int kblocks = (a.rows + 15) >> 4;

        // fp32 accumulator columns -> shared staging in the layout of the fp32 maps (32-column slabs)
        auto stage_f32 = [&](uint32_t col0, uint32_t stage) {
            if (!warp_valid) return;
            uint32_t v[32];
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
                tmem_ld32(tmem_lane + col0 + 32 * c, v);
                if (!row_valid) continue;
                const uint32_t row = stage + (uint32_t)c * kSlabBytes + (uint32_t)r * 128u;
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    st_shared_v4(row + (uint32_t)((i ^ (r & 7)) * 16), v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
            }
        };

        // the same for a gradient with respect to ROTATED vectors (dQ, dK under the positional
        // encoding): row r sits at position r mod n, feature c is paired with c + D/2, and the
        // gradient of the un-rotated vector is the transposed rotation of the rotated one's
        const float pos = (float)(r % a.n);
        auto stage_f32_unrotated = [&](uint32_t col0, uint32_t stage) {
            if (!warp_valid) return;
            constexpr int kHalfChunks = D / 64;          // 32-column chunks in half a row
            uint32_t va[32], vb[32];
#pragma unroll 1
            for (int c = 0; c < kHalfChunks; ++c) {
                tmem_ld32(tmem_lane + col0 + 32 * c, va);
                tmem_ld32(tmem_lane + col0 + 32 * (c + kHalfChunks), vb);
                if (!row_valid) continue;
#pragma unroll
                for (int jj = 0; jj < 32; ++jj) {
                    const float ang = pos * theta_tab[32 * c + jj];
                    const float cs = __cosf(ang), sn = __sinf(ang);
                    const float x1 = __uint_as_float(va[jj]), x2 = __uint_as_float(vb[jj]);
                    va[jj] = __float_as_uint(x1 * cs + x2 * sn);
                    vb[jj] = __float_as_uint(x2 * cs - x1 * sn);
                }
                const uint32_t row_a = stage + (uint32_t)c * kSlabBytes + (uint32_t)r * 128u;
                const uint32_t row_b = stage + (uint32_t)(c + kHalfChunks) * kSlabBytes + (uint32_t)r * 128u;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    st_shared_v4(row_a + (uint32_t)((i ^ (r & 7)) * 16), va[4 * i], va[4 * i + 1], va[4 * i + 2], va[4 * i + 3]);
                    st_shared_v4(row_b + (uint32_t)((i ^ (r & 7)) * 16), vb[4 * i], vb[4 * i + 1], vb[4 * i + 2], vb[4 * i + 3]);
                }
            }
        };

        uint32_t t = 0, it = 0;
        bool ok = true;
        int pending_stage = -1;   // thread 0: stage whose output stores have been issued but not yet read out
        for (long long item = blockIdx.x; ok && item < a.total_items; item += gridDim.x, ++it) {
            const BwdItem c = decode_bwd_item(a, item);
            uint32_t lim[4] = {~0u, ~0u, ~0u, ~0u};        // columns below the batch entry's valid length
            if (kMask && a.lens != nullptr) {
                // only the first `exist` positions of this row's segment are tokens; a padding row
                // sees nothing (its P and dS rows are 0, so nothing flows through it)
                const int len = __ldg(a.lens + c.kv_head / a.H_kv);
                const long long first = (long long)(c.c_outer + seg / a.ci) * a.n * a.stride + (c.c_inner + seg % a.ci);
                const long long left = ((long long)len - first + a.stride - 1) / a.stride;
                const int exist = len <= first ? 0 : (int)(left < a.n ? left : a.n);
                const int limit = (r % a.n) < exist ? seg * a.n + exist : 0;
#pragma unroll
                for (int cch = 0; cch < 4; ++cch) {
                    const int nb = limit - 32 * cch;
                    lim[cch] = nb >= 32 ? 0xffffffffu : (nb <= 0 ? 0u : ((1u << nb) - 1u));
                    mt[cch] = mrow[cch] & lim[cch];
                }
            }
            for (int j = 0; j < a.g; ++j, ++t) {
                if (kMask && a.dmask != nullptr) {
                    // this query head has a mask of its own
                    tile_row_mask(a.dmask + (size_t)((c.q_head0 + j) % a.H) * a.n * 4, row_valid ? r % a.n : 0, seg * a.n, mt);
#pragma unroll
                    for (int cch = 0; cch < 4; ++cch) mt[cch] = row_valid ? (mt[cch] & lim[cch]) : 0u;
                }
                const int s = t & 1;
                const uint32_t par = t & 1;
                const int q_head = c.q_head0 + j;
                const bool last_head = j == a.g - 1;
                const uint32_t q_base = sQ(s), g_base = sG(s);

                // ---- S = Q K^T and dP = G X^T
                if (tid == 0) {
                    bool k0 = true;
                    if (j == 0) k0 = mbar_wait_abortable(kRope ? k_rot : k_full, it & 1, 0x71, abort_flag);
                    if (k0) k0 = mbar_wait_abortable(qg_full(s), (t >> 1) & 1, 0x72, abort_flag);
                    if (kRope && k0) k0 = mbar_wait_abortable(q_rot(s), (t >> 1) & 1, 0x76, abort_flag);
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
                        // the previous head's stores overlap this head's score MMAs; their staging
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

                // ---- softmax and its derivative for this thread's row; P -> X slot, dS -> its slot
                const int cc_lo = w_lo >> 5, cc_hi = (max(w_hi, w_lo + 1) - 1) >> 5;
                if (warp_valid && cc_lo == cc_hi) {
                    // Every key this warp's rows can see lies in ONE 32-column chunk (segments of at
                    // most 32 positions aligned to the chunks: the usual case): the scores and dP are
                    // read from tensor memory once and the weights stay in registers between the passes.
                    const int cc = cc_lo;
                    uint32_t vs[32], vd[32];
                    tmem_ld32(tmem_lane + C::kColS + 32 * cc, vs);
                    tmem_ld32(tmem_lane + C::kColDP + 32 * cc, vd);
                    float m = -INFINITY;
#pragma unroll
                    for (int jj = 0; jj < 32; ++jj)
                        if (visible(cc, jj)) m = fmaxf(m, __uint_as_float(vs[jj]));
                    const float m_s = (row_valid && !(kMask && m == -INFINITY)) ? m * a.scale_log2 : 0.f;
                    float l = 0.f, dot = 0.f;
#pragma unroll
                    for (int jj = 0; jj < 32; ++jj) {
                        float p = fast_exp2(__uint_as_float(vs[jj]) * a.scale_log2 - m_s);
                        p = visible(cc, jj) ? p : 0.f;
                        vs[jj] = __float_as_uint(p);                   // un-normalised weight
                        l += p;
                        dot += p * __uint_as_float(vd[jj]);            // p is 0 where the key is invisible
                    }
                    const float inv_l = (row_valid && !(kMask && l == 0.f)) ? 1.f / l : 0.f;
                    const float delta = dot * inv_l;
                    const uint32_t rowP = sXP + (uint32_t)r * 128u, rowS = sdS + (uint32_t)r * 128u;
#pragma unroll 1
                    for (int c4 = 0; c4 < 4; ++c4) {
                        uint32_t pp[16], ps[16];
                        if (c4 == cc) {
#pragma unroll
                            for (int jj = 0; jj < 32; jj += 2) {
                                const float p0 = __uint_as_float(vs[jj]) * inv_l, p1 = __uint_as_float(vs[jj + 1]) * inv_l;
                                pp[jj >> 1] = pack_bf16x2(p0, p1);
                                ps[jj >> 1] = pack_bf16x2(p0 * (__uint_as_float(vd[jj]) - delta) * a.scale,
                                                          p1 * (__uint_as_float(vd[jj + 1]) - delta) * a.scale);
                            }
                        } else {
#pragma unroll
                            for (int jj = 0; jj < 16; ++jj) { pp[jj] = 0u; ps[jj] = 0u; }
                        }
                        const uint32_t slab = (uint32_t)(c4 >> 1) * kSlabBytes;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const uint32_t chunk = (uint32_t)(((c4 & 1) * 4 + i) ^ (r & 7)) * 16;
                            st_shared_v4(rowP + slab + chunk, pp[4 * i], pp[4 * i + 1], pp[4 * i + 2], pp[4 * i + 3]);
                            st_shared_v4(rowS + slab + chunk, ps[4 * i], ps[4 * i + 1], ps[4 * i + 2], ps[4 * i + 3]);
                        }
                    }
                } else {
                    uint32_t vs[32], vd[32];
                    float m = -INFINITY;
#pragma unroll 1
                    for (int cc = 0; cc < 4; ++cc) {
                        if (!(warp_valid && 32 * cc < w_hi && 32 * cc + 32 > w_lo)) continue;
                        tmem_ld32(tmem_lane + C::kColS + 32 * cc, vs);
#pragma unroll
                        for (int jj = 0; jj < 32; ++jj) {
                            if (visible(cc, jj)) m = fmaxf(m, __uint_as_float(vs[jj]));
                        }
                    }
                    const float m_s = (row_valid && !(kMask && m == -INFINITY)) ? m * a.scale_log2 : 0.f;
                    float l = 0.f, dot = 0.f;
#pragma unroll 1
                    for (int cc = 0; cc < 4; ++cc) {
                        if (!(warp_valid && 32 * cc < w_hi && 32 * cc + 32 > w_lo)) continue;
                        tmem_ld32(tmem_lane + C::kColS + 32 * cc, vs);
                        tmem_ld32(tmem_lane + C::kColDP + 32 * cc, vd);
#pragma unroll
                        for (int jj = 0; jj < 32; ++jj) {
                            float p = fast_exp2(__uint_as_float(vs[jj]) * a.scale_log2 - m_s);
                            const bool vis = visible(cc, jj);
                            p = vis ? p : 0.f;
                            l += p;
                            dot += vis ? p * __uint_as_float(vd[jj]) : 0.f;
                        }
                    }
                    const float inv_l = (row_valid && !(kMask && l == 0.f)) ? 1.f / l : 0.f;
                    const float delta = dot * inv_l;
                    const uint32_t rowP = sXP + (uint32_t)r * 128u, rowS = sdS + (uint32_t)r * 128u;
#pragma unroll 1
                    for (int cc = 0; cc < 4; ++cc) {
                        uint32_t pp[16], ps[16];
                        if (warp_valid && 32 * cc < w_hi && 32 * cc + 32 > w_lo) {
                            tmem_ld32(tmem_lane + C::kColS + 32 * cc, vs);
                            tmem_ld32(tmem_lane + C::kColDP + 32 * cc, vd);
#pragma unroll
                            for (int jj = 0; jj < 32; jj += 2) {
                                float pv[2], dv[2];
#pragma unroll
                                for (int e = 0; e < 2; ++e) {
                                    const bool vis = visible(cc, jj + e);
                                    float p = fast_exp2(__uint_as_float(vs[jj + e]) * a.scale_log2 - m_s) * inv_l;
                                    p = vis ? p : 0.f;
                                    pv[e] = p;
                                    dv[e] = vis ? p * (__uint_as_float(vd[jj + e]) - delta) * a.scale : 0.f;
                                }
                                pp[jj >> 1] = pack_bf16x2(pv[0], pv[1]);
                                ps[jj >> 1] = pack_bf16x2(dv[0], dv[1]);
                            }
                        } else {
#pragma unroll
                            for (int jj = 0; jj < 16; ++jj) { pp[jj] = 0u; ps[jj] = 0u; }
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

                // ---- G_i = P^T G (first hop: dV += P^T G), dQ = dS K, dK += dS^T Q
                if (tid == 0) {
                    tc_fence_after();
                    const uint32_t g_acc = tmem_base + (a.first_hop ? C::kColDV : C::kColS);
                    for (int kb = 0; kb < kblocks; ++kb) {
                        const uint32_t k_off = kb * 2048;                                  // 16 rows of 128 bytes
                        const uint32_t a_off = (kb >> 2) * kSlabBytes + (kb & 3) * 32;     // 16 columns of a K-major tile
                        // G_i[key, d] = sum_q P[q, key] G[q, d]
                        tc_mma_ss(g_acc, smem_desc_sw128(sXP + k_off, kSlabBytes, 1024),
                                  smem_desc_sw128(g_base + k_off, kSlabBytes, 1024), idesc_g,
                                  (kb > 0 || (a.first_hop && j > 0)) ? 1u : 0u);
                        // dQ[q, d] = sum_key dS[q, key] K[key, d]
                        tc_mma_ss(tmem_base + C::kColDP, smem_desc_sw128(sdS + a_off, 16, 1024),
                                  smem_desc_sw128(sK + k_off, kSlabBytes, 1024), idesc_dq, kb > 0);
                        // dK[key, d] += sum_q dS[q, key] Q[q, d]   (summed over the heads of the item)
                        tc_mma_ss(tmem_base + C::kColDK, smem_desc_sw128(sdS + k_off, kSlabBytes, 1024),
                                  smem_desc_sw128(q_base + k_off, kSlabBytes, 1024), idesc_g,
                                  (kb > 0 || j > 0) ? 1u : 0u);
                    }
                    tc_commit(o_done);
                    tc_commit(xp_free);                // the X / P slot may take the next head's X
                    if (last_head) tc_commit(k_free);
                }
                __syncwarp();
                ok = mbar_wait_abortable(o_done, par, 0x75, abort_flag);
                ok = wg_all(ok);
                if (!ok) break;
                tc_fence_after();

                // ---- epilogue: dQ (fp32, over this head's Q and G tiles) and G_i (bf16, over dS)
                if (kRope) stage_f32_unrotated(C::kColDP, q_base);
                else stage_f32(C::kColDP, q_base);
                if (!a.first_hop && warp_valid) {
                    uint32_t v[32];
#pragma unroll 1
                    for (int cc = 0; cc < D / 32; ++cc) {
                        tmem_ld32(tmem_lane + C::kColS + 32 * cc, v);
                        if (!row_valid) continue;
                        uint32_t pk[16];
#pragma unroll
                        for (int jj = 0; jj < 32; jj += 2)
                            pk[jj >> 1] = pack_bf16x2(__uint_as_float(v[jj]), __uint_as_float(v[jj + 1]));
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
                    for (int sl = 0; sl < D / 32; ++sl) {
                        if (a.accumulate)
                            tma_reduce_add_5d(&map_dq, q_base + sl * kSlabBytes, 32 * sl, 0, c.c_inner, c.c_outer, q_head);
                        else
                            tma_store_5d(&map_dq, q_base + sl * kSlabBytes, 32 * sl, 0, c.c_inner, c.c_outer, q_head);
                    }
                    if (!a.first_hop) {
#pragma unroll
                        for (int h = 0; h < kHalves; ++h)
                            tma_store_5d(&map_gout, sdS + h * kSlabBytes, 64 * h, 0, c.c_inner, c.c_outer, q_head);
                    }
                    if (last_head) tma_store_commit_and_wait_read();   // the staging space is reused right below
                    else asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
                if (last_head) {
                    // ---- once per item: dK (and, in the first hop, dV) of the whole group
                    wg_sync();                         // the staging space has been read out
                    tc_fence_after();
                    if (kRope) stage_f32_unrotated(C::kColDK, q_base);
                    else stage_f32(C::kColDK, q_base);
                    fence_proxy_async_smem();
                    tc_fence_before();
                    wg_sync();
                    if (tid == 0) {
#pragma unroll
                        for (int sl = 0; sl < D / 32; ++sl) {
                            if (a.accumulate)
                                tma_reduce_add_5d(&map_dk, q_base + sl * kSlabBytes, 32 * sl, 0, c.c_inner, c.c_outer, c.kv_head);
                            else
                                tma_store_5d(&map_dk, q_base + sl * kSlabBytes, 32 * sl, 0, c.c_inner, c.c_outer, c.kv_head);
                        }
                        tma_store_commit_and_wait_read();
                    }
                    if (a.first_hop) {
                        wg_sync();
                        tc_fence_after();
                        stage_f32(C::kColDV, q_base);
                        fence_proxy_async_smem();
                        tc_fence_before();
                        wg_sync();
                        if (tid == 0) {
#pragma unroll
                            for (int sl = 0; sl < D / 32; ++sl)
                                tma_store_5d(&map_dv, q_base + sl * kSlabBytes, 32 * sl, 0, c.c_inner, c.c_outer, c.kv_head);
                            tma_store_commit_and_wait_read();
                        }
                    }
                }
                if (tid == 0) {
                    if (last_head) mbar_arrive(qg_free(s));   // read out: this stage may take the head after next
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
template <typename TI, typename TO>
__global__ void group_sum_kernel(const TI *__restrict__ dout, TO *__restrict__ dv, long long per_head, int H, int H_kv,
                                 long long total_kv) {
    const int g = H / H_kv;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total_kv;
         i += (long long)gridDim.x * blockDim.x) {
        const long long bkv = i / per_head, rr = i % per_head;
        const long long b = bkv / H_kv, kvh = bkv % H_kv;
        float s = 0.f;
        for (int j = 0; j < g; ++j) {
            const TI x = dout[((b * H + kvh * g + j) * per_head) + rr];
            if constexpr (sizeof(TI) == 4) s += x;
            else s += __bfloat162float(x);
        }
        if constexpr (sizeof(TO) == 4) dv[i] = s;
        else dv[i] = __float2bfloat16_rn(s);
    }
}

template <int D>
int launch_bwd_d(const Problem &pb, const HopDesc &hd, const void *x, int x_heads, const void *g_in, void *g_out,
                 float *dq_acc, float *dk_acc, float *dv_acc, bool first_hop, bool accumulate) {
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
    a.accumulate = accumulate ? 1 : 0;
    a.window = pb.window[hd.hop];
    a.tiles_inner = hd.tiles_inner; a.tiles_outer = hd.tiles_outer;
    a.total_items = (long long)pb.B * pb.H_kv * hd.tiles_inner * hd.tiles_outer;
    a.scale = pb.scale;
    a.scale_log2 = pb.scale * 1.4426950408889634f;
    a.rope_log2_base = pb.rope_base > 0.f ? log2f(pb.rope_base) : 0.f;
    a.stride = (int)hd.stride;
    a.lens = pb.seq_lens;
    a.dmask = (pb.masks[hd.hop] && pb.masks_per_head) ? pb.dmask[hd.hop] : nullptr;
    if (pb.masks[hd.hop] && pb.masks_per_head && !a.dmask) return TA_ERR_INVALID_ARG;

    int dev = 0;
    const int num_sms = current_device_sms(&dev);
    constexpr size_t smem = BwdCfg<D>::kSmemBytes;
    static PerDeviceOnce configured;
    if (!configured.is_done(dev)) {
        const cudaFuncAttribute attr = cudaFuncAttributeMaxDynamicSharedMemorySize;
        if (cudaFuncSetAttribute(hop_tc_bwd_kernel<D, false, false>, attr, (int)smem) != cudaSuccess ||
            cudaFuncSetAttribute(hop_tc_bwd_kernel<D, true, false>, attr, (int)smem) != cudaSuccess ||
            cudaFuncSetAttribute(hop_tc_bwd_kernel<D, false, true>, attr, (int)smem) != cudaSuccess ||
            cudaFuncSetAttribute(hop_tc_bwd_kernel<D, true, true>, attr, (int)smem) != cudaSuccess)
            return TA_ERR_CUDA;
        configured.mark(dev);
    }
    const unsigned grid = (unsigned)(a.total_items < num_sms ? a.total_items : num_sms);
    if (pb.masks[hd.hop] || pb.seq_lens) {
        HopMask hm;                                  // explicit mask ^ causal flag ^ window, by value
        if (a.dmask) {
            memset(&hm, 0, sizeof(hm));              // per-head masks: read from device memory per head
        } else {
            const int rc = build_hop_mask(pb, hd, &hm);
            if (rc != TA_OK) return rc;
        }
        if (pb.rope_base > 0.f)
            return launch_kernel(hop_tc_bwd_kernel<D, true, true>, grid, kThreadsRope, smem, pb.stream, false, mq, mk, mx,
                                 mgi, mgo, mdq, mdk, mdv, a, hm);
        return launch_kernel(hop_tc_bwd_kernel<D, false, true>, grid, kThreads, smem, pb.stream, false, mq, mk, mx, mgi,
                             mgo, mdq, mdk, mdv, a, hm);
    }
    if (pb.rope_base > 0.f)
        return launch_kernel(hop_tc_bwd_kernel<D, true, false>, grid, kThreadsRope, smem, pb.stream, false, mq, mk, mx, mgi,
                             mgo, mdq, mdk, mdv, a, NoMask{});
    return launch_kernel(hop_tc_bwd_kernel<D, false, false>, grid, kThreads, smem, pb.stream, false, mq, mk, mx, mgi, mgo,
                         mdq, mdk, mdv, a, NoMask{});
}

}  // namespace

int launch_hop_tc_bwd(const Problem &pb, const HopDesc &hd, const void *x, int x_heads, const void *g_in,
                      void *g_out, float *dq_acc, float *dk_acc, float *dv_acc, bool first_hop, bool accumulate) {
    if (pb.D == 128)
        return launch_bwd_d<128>(pb, hd, x, x_heads, g_in, g_out, dq_acc, dk_acc, dv_acc, first_hop, accumulate);
    if (pb.D == 64)
        return launch_bwd_d<64>(pb, hd, x, x_heads, g_in, g_out, dq_acc, dk_acc, dv_acc, first_hop, accumulate);
    return TA_ERR_UNSUPPORTED;
}

int launch_f32_to_bf16(const float *src, void *dst, long long n, cudaStream_t stream) {
    if (n <= 0) return TA_OK;
    long long blocks = (n / 4 + 255) / 256;
    if (blocks > 148 * 32) blocks = 148 * 32;
    if (blocks < 1) blocks = 1;
    return launch_kernel(f32_to_bf16_kernel, (unsigned)blocks, 256, 0, stream, false, src, (__nv_bfloat16 *)dst, n);
}

int launch_group_sum(const void *dout, int dout_is_f32, void *dv, int dv_is_f32, int B, int H, int H_kv,
                     long long per_head, cudaStream_t stream) {
    const long long total = (long long)B * H_kv * per_head;
    long long blocks = (total + 255) / 256;
    if (blocks > 148 * 32) blocks = 148 * 32;
    const unsigned grid = (unsigned)blocks;
    if (dout_is_f32) {
        if (!dv_is_f32) return TA_ERR_UNSUPPORTED;     // fp32 tensors take fp32 gradients
        return launch_kernel(group_sum_kernel<float, float>, grid, 256, 0, stream, false, (const float *)dout, (float *)dv,
                             per_head, H, H_kv, total);
    }
    if (dv_is_f32)
        return launch_kernel(group_sum_kernel<__nv_bfloat16, float>, grid, 256, 0, stream, false,
                             (const __nv_bfloat16 *)dout, (float *)dv, per_head, H, H_kv, total);
    return launch_kernel(group_sum_kernel<__nv_bfloat16, __nv_bfloat16>, grid, 256, 0, stream, false,
                         (const __nv_bfloat16 *)dout, (__nv_bfloat16 *)dv, per_head, H, H_kv, total);
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
