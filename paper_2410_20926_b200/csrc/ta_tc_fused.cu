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
// Persistent, one CTA per SM, warp-specialised like the per-hop kernel:
//   warp 0      TMA producer: K once per work item (the query heads of a GQA group share it),
//               Q and the value tile X per head, into rings of shared memory
//   warp 1      MMA issuer: polls for whichever of S(t) = Q K^T or O(t, f) = P_f X has its
//               operands ready (two tiles are in flight, one per warpgroup)
//   warps 4-7   softmax + epilogue of the even tiles   } per tile: for each fused hop f, P_f from
//   warps 8-11  softmax + epilogue of the odd tiles    } S and the row's mask, then X <- O / rowsum
//   warp 2      TMA store of finished tiles; hands the X slot back to the producer
// Tensor memory: S x 2 (kept for all fused hops of its tile), P x 2 (bf16, A operand of the value
// MMA), O (x 2 at D = 64).  Every wait is bounded; when one expires the CTA raises a flag that
// ends all its roles, waits for its copies in flight, frees its TMEM and returns.
#include <cuda_bf16.h>

#include "ta_internal.h"
#include "ta_ptx.cuh"

namespace ta {
namespace {

constexpr int kTileRows = 128;
constexpr int kThreads = 384;
constexpr int kNK = 2, kNQ = 2;

struct FusedArgs {
    int block, rows, co, causal, g, H, H_kv, xin_is_kv, nf;
    int gi, hsplit;            // query heads per work item, items per GQA group
    int sub_n[TA_MAX_DIMS], sub_stride[TA_MAX_DIMS], sub_window[TA_MAX_DIMS];
    long long tiles_outer, total_items;
    float scale_log2;
    int x_f16;                 // the value tensor read holds fp16 (output of a preceding tensor-core hop), not bf16
};

template <int D>
struct FusedCfg {
    static constexpr int kHalves = D / 64;
    static constexpr uint32_t kSlabBytes = kTileRows * 128;
    static constexpr uint32_t kTileBytes = kHalves * kSlabBytes;
    static constexpr int kNX = D == 128 ? 2 : 4;                             // value-tile ring
    static constexpr uint32_t kOffK = 0;
    static constexpr uint32_t kOffQ = kOffK + kNK * kTileBytes;
    static constexpr uint32_t kOffX = kOffQ + kNQ * kTileBytes;
    static constexpr uint32_t kOffMask = kOffX + kNX * kTileBytes;          // [hop][128 rows][4 words]
    static constexpr uint32_t kMaskBytes = TA_MAX_DIMS * kTileRows * 16;
    static constexpr uint32_t kOffBar = kOffMask + kMaskBytes;
    static constexpr int kNumBars = 2 * kNK + 2 * kNQ + 3 * kNX + 2 + 2 + 2 + 2;
    static constexpr uint32_t kSmemBytes = kOffBar + kNumBars * 8 + 16 + 1024;
    static constexpr uint32_t kTmemCols = 512;
    // S: 2 x 128 | O: one buffer of 128 columns (D = 128) or two of 64 (D = 64) | P: 2 x 64
    static constexpr uint32_t kColS = 0, kColO = 256, kColP = 384;
    static constexpr int kNO = D == 64 ? 2 : 1;
};

struct FusedItem {
    int c_outer, kv_head, q_head0;
};
__device__ __forceinline__ FusedItem decode_fused_item(const FusedArgs &a, long long item) {
    FusedItem c;
    long long rest = item;
    const int hs = (int)(rest % a.hsplit); rest /= a.hsplit;
    c.c_outer = (int)(rest % a.tiles_outer) * a.co; rest /= a.tiles_outer;
    c.kv_head = (int)rest;
    c.q_head0 = (c.kv_head / a.H_kv) * a.H + (c.kv_head % a.H_kv) * a.g + hs * a.gi;
    return c;
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
hop_fused_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_xin, const __grid_constant__ CUtensorMap map_xout,
                 const FusedArgs a) {
    using C = FusedCfg<D>;
    constexpr int kHalves = C::kHalves;
    constexpr uint32_t kSlabBytes = C::kSlabBytes, kTileBytes = C::kTileBytes;
    constexpr int kNX = C::kNX, kNO = C::kNO;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t s0 = smem_u32(smem);
    const uint32_t sK = s0 + C::kOffK, sQ = s0 + C::kOffQ, sX = s0 + C::kOffX;
    uint32_t *masks = (uint32_t *)(smem + C::kOffMask);
    const uint32_t bar0 = s0 + C::kOffBar;
    auto k_full = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    auto k_free = [&](int i) { return bar0 + 8u * (uint32_t)(kNK + i); };
    auto q_full = [&](int i) { return bar0 + 8u * (uint32_t)(2 * kNK + i); };
    auto q_free = [&](int i) { return bar0 + 8u * (uint32_t)(2 * kNK + kNQ + i); };
    constexpr int kB0 = 2 * kNK + 2 * kNQ;
    auto x_full = [&](int i) { return bar0 + 8u * (uint32_t)(kB0 + i); };
    auto x_free = [&](int i) { return bar0 + 8u * (uint32_t)(kB0 + kNX + i); };
    auto out_full = [&](int i) { return bar0 + 8u * (uint32_t)(kB0 + 2 * kNX + i); };
    constexpr int kB1 = kB0 + 3 * kNX;
    auto s_full = [&](int i) { return bar0 + 8u * (uint32_t)(kB1 + i); };       // S(t) complete, per warpgroup
    auto p_full = [&](int i) { return bar0 + 8u * (uint32_t)(kB1 + 2 + i); };   // P_f written (4 warps)
    auto o_full = [&](int i) { return bar0 + 8u * (uint32_t)(kB1 + 4 + i); };   // O(t, f) complete
    auto o_free = [&](int i) { return bar0 + 8u * (uint32_t)(kB1 + 6 + i); };   // O read out (4 warps)
    uint32_t *tmem_slot = (uint32_t *)(smem + C::kOffBar + C::kNumBars * 8);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // ---- one-time setup
    for (uint32_t i = tid; i < C::kOffBar / 16; i += kThreads)
        ((uint4 *)smem)[i] = make_uint4(0, 0, 0, 0);   // rows a box never fills must stay finite
    if (tid == 0) {
        for (int i = 0; i < kNK; ++i) { mbar_init(k_full(i), 1); mbar_init(k_free(i), 1); }
        for (int i = 0; i < kNQ; ++i) { mbar_init(q_full(i), 1); mbar_init(q_free(i), 1); }
        for (int i = 0; i < kNX; ++i) { mbar_init(x_full(i), 1); mbar_init(x_free(i), 1); mbar_init(out_full(i), 4); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(s_full(i), 1); mbar_init(p_full(i), 4); mbar_init(o_full(i), 1); mbar_init(o_free(i), 4);
        }
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (tid < kTileRows && tid < a.rows) {
        // visibility of the tile's columns from row `tid` in each fused hop: the mode-f vector
        // through the row -- same block, every coordinate but the f-th equal (causal: up to its own)
        const int blk = tid / a.block, rr = tid % a.block;
        for (int f = 0; f < a.nf; ++f) {
            const int st = a.sub_stride[f], n = a.sub_n[f];
            const int coord = (rr / st) % n;
            const int first = blk * a.block + rr - coord * st;
            const int last = a.causal ? coord : n - 1;
            uint32_t *m = masks + ((size_t)f * kTileRows + tid) * 4;
            const int w = a.sub_window[f];              // sliding window along this dimension (0: none)
            for (int u = 0; u <= last; ++u) {
                if (w > 0 && (u <= coord - w || u >= coord + w)) continue;
                const int col = first + u * st;
                m[col >> 5] |= 1u << (col & 31);
            }
        }
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

    const long long my_items = (a.total_items - blockIdx.x + gridDim.x - 1) / gridDim.x;
    const uint32_t T = (uint32_t)(my_items * a.gi);
    const uint32_t slab_tx = (uint32_t)a.rows * 128u;

    if (warp == 0) {
        // =============================================================== TMA producer
        if (lane == 0) {
            uint32_t t = 0, it = 0;
            uint32_t armed = 0, last_par = 0;   // bit per barrier slot: k 0-1, q 2-3, x 4-7
            auto arm = [&](uint32_t bit, uint32_t parity) {
                armed |= bit;
                last_par = parity ? (last_par | bit) : (last_par & ~bit);
            };
            bool ok = true;
            bool prev_hop_done = false;
            for (long long item = blockIdx.x; ok && item < a.total_items; item += gridDim.x, ++it) {
                const FusedItem c = decode_fused_item(a, item);
                const int ks = it & 1;
                const uint32_t kpar = (it >> 1) & 1;
                ok = mbar_wait_abortable(k_free(ks), kpar ^ 1, 0x90, abort_flag);
                if (!ok) break;
                mbar_expect_tx(k_full(ks), kHalves * slab_tx);
                arm(1u << ks, kpar);
#pragma unroll
                for (int h = 0; h < kHalves; ++h)
                    tma_load_5d(sK + ks * kTileBytes + h * kSlabBytes, &map_k, k_full(ks), 64 * h, 0, 0, c.c_outer, c.kv_head);
                for (int j = 0; j < a.gi; ++j, ++t) {
                    const int q_head = c.q_head0 + j;
                    const int x_head = a.xin_is_kv ? c.kv_head : q_head;
                    const int qs = t & 1;
                    const uint32_t qpar = (t >> 1) & 1;
                    ok = mbar_wait_abortable(q_free(qs), qpar ^ 1, 0x91, abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(q_full(qs), kHalves * slab_tx);
                    arm(4u << qs, qpar);
#pragma unroll
                    for (int h = 0; h < kHalves; ++h)
                        tma_load_5d(sQ + qs * kTileBytes + h * kSlabBytes, &map_q, q_full(qs), 64 * h, 0, 0, c.c_outer, q_head);
                    const int xs = t % kNX;
                    const uint32_t xpar = (t / kNX) & 1;
                    ok = mbar_wait_abortable(x_free(xs), xpar ^ 1, 0x92, abort_flag);
                    if (!ok) break;
                    if (!prev_hop_done) {      // launched while the previous hop drains: its output is read from here on
                        griddep_wait();
                        prev_hop_done = true;
                    }
                    mbar_expect_tx(x_full(xs), kHalves * slab_tx);
                    arm(16u << xs, xpar);
#pragma unroll
                    for (int h = 0; h < kHalves; ++h)
                        tma_load_5d(sX + xs * kTileBytes + h * kSlabBytes, &map_xin, x_full(xs), 64 * h, 0, 0, c.c_outer, x_head);
                }
            }
            if (!ok) {
                // leaving early: let the copies already issued land (bounded)
                const unsigned long long t0 = globaltimer_ns();
                for (int slot = 0; slot < 4 + kNX; ++slot) {
                    if (!(armed & (1u << slot))) continue;
                    const uint32_t bar = slot < 2 ? k_full(slot) : (slot < 4 ? q_full(slot - 2) : x_full(slot - 4));
                    while (!mbar_try_wait(bar, (last_par >> slot) & 1u) && globaltimer_ns() - t0 < 10000000ull) {
                    }
                }
            }
        }
    } else if (warp == 1) {
        // =============================================================== MMA issuer
        // Two tiles are in flight, one per warpgroup ("chain" b = tile parity).  A chain is busy
        // from its S = Q K^T until the value MMA of its last fused hop has been issued.
        if (lane == 0) {
            constexpr uint32_t idesc_s = instr_desc(128, 0);
            // the value tile is fp16 from the second fused hop on (and from the first one when the hop
            // before this pass left fp16): the weights take its type
            constexpr uint32_t idesc_o_bf16 = instr_desc(D, 1), idesc_o_f16 = instr_desc_f16(D, 1);
            const int kblocks = (a.rows + 15) >> 4;
            uint32_t t1 = 0, it = 0, j = 0, tiles_done = 0;
            bool busy[2] = {false, false};
            uint32_t tile_of[2] = {0, 0}, hop_of[2] = {0, 0};   // chain: its tile and next fused hop
            uint32_t p_seen[2] = {0, 0};                        // phases of p_full(b) consumed
            uint32_t o_issued[2] = {0, 0};                      // value MMAs issued by chain b
            int last_user[2] = {-1, -1};                        // chain that last wrote each O buffer
            uint32_t idle = 0;
            unsigned long long idle_since = 0;
            while (tiles_done < T) {
                bool progressed = false;
                const int b1 = t1 & 1;
                if (t1 < T && !busy[b1]) {
                    const int ks = it & 1, qs = t1 & 1;
                    if ((j != 0 || mbar_test_wait(k_full(ks), (it >> 1) & 1)) && mbar_test_wait(q_full(qs), (t1 >> 1) & 1)) {
                        tc_fence_after();
                        const uint32_t q_base = sQ + qs * kTileBytes, k_base = sK + ks * kTileBytes;
#pragma unroll
                        for (int kb = 0; kb < D / 16; ++kb) {
                            const uint32_t off = (kb >> 2) * kSlabBytes + (kb & 3) * 32;
                            tc_mma_ss(tmem_base + C::kColS + b1 * 128, smem_desc_sw128(q_base + off, 16, 1024),
                                      smem_desc_sw128(k_base + off, 16, 1024), idesc_s, kb > 0);
                        }
                        tc_commit(s_full(b1));
                        tc_commit(q_free(qs));
                        if (++j == (uint32_t)a.gi) {
                            tc_commit(k_free(ks));
                            j = 0;
                            ++it;
                        }
                        busy[b1] = true;
                        tile_of[b1] = t1;
                        hop_of[b1] = 0;
                        ++t1;
                        progressed = true;
                    }
                }
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    const int b = (t1 + k) & 1;                 // the older tile first
                    if (!busy[b]) continue;
                    const uint32_t tile = tile_of[b];
                    const int xs = tile % kNX;
                    const int ob = kNO == 2 ? b : 0;
                    const int lu = last_user[ob];
                    if (!mbar_test_wait(p_full(b), p_seen[b] & 1)) continue;
                    if (hop_of[b] == 0 && !mbar_test_wait(x_full(xs), (tile / kNX) & 1)) continue;
                    if (lu >= 0 && !mbar_test_wait(o_free(lu), (o_issued[lu] - 1) & 1)) continue;
                    tc_fence_after();
                    // O[128 x D] = P_f[128 x rows] X[rows x D]; P from tensor memory, X MN-major from shared memory
                    const uint32_t d_tmem = tmem_base + C::kColO + (kNO == 2 ? 64 * b : 0);
                    const uint32_t p_tmem = tmem_base + C::kColP + 64 * b;
                    const uint32_t x_base = sX + xs * kTileBytes;
                    const uint32_t idesc_o = (hop_of[b] > 0 || a.x_f16) ? idesc_o_f16 : idesc_o_bf16;
                    for (int kb = 0; kb < kblocks; ++kb)
                        tc_mma_ts(d_tmem, p_tmem + kb * 8, smem_desc_sw128(x_base + kb * 2048, kSlabBytes, 1024), idesc_o,
                                  kb > 0);
                    tc_commit(o_full(b));
                    ++p_seen[b];
                    ++o_issued[b];
                    last_user[ob] = b;
                    if (++hop_of[b] == (uint32_t)a.nf) {
                        busy[b] = false;
                        ++tiles_done;
                    }
                    progressed = true;
                }
                if (progressed) {
                    idle = 0;
                    idle_since = 0;
                } else if (++idle < 1024) {
                    __nanosleep(40);
                } else {
                    idle = 0;
                    if (*abort_flag) break;
                    const unsigned long long now = globaltimer_ns();
                    if (idle_since == 0) idle_since = now;
                    if (now - idle_since > kWaitLimitNs) {
                        atomicCAS(&g_status_word, 0u, kErrWaitExpired | 0xA0u);
                        *abort_flag = 1u;
                        break;
                    }
                }
            }
        }
    } else if (warp == 2) {
        // =============================================================== TMA store
        if (lane == 0) {
            uint32_t t = 0;
            bool ok = true;
            for (long long item = blockIdx.x; ok && item < a.total_items; item += gridDim.x) {
                const FusedItem c = decode_fused_item(a, item);
                for (int j = 0; j < a.gi; ++j, ++t) {
                    const int xs = t % kNX;
                    ok = mbar_wait_abortable(out_full(xs), (t / kNX) & 1, 0xB0, abort_flag);
                    if (!ok) break;
#pragma unroll
                    for (int h = 0; h < kHalves; ++h)
                        tma_store_5d(&map_xout, sX + xs * kTileBytes + h * kSlabBytes, 64 * h, 0, 0, c.c_outer, c.q_head0 + j);
                    tma_store_commit_and_wait_read();
                    mbar_arrive(x_free(xs));
                }
            }
            tma_store_wait_all();
        }
    } else if (warp >= 4) {
        // =============================================================== softmax + epilogue
        const int b = (warp - 4) >> 2;                  // tile parity this warpgroup serves
        const int wq = warp & 3;                        // TMEM lane quarter of this warp
        const uint32_t tmem_lane = tmem_base + ((uint32_t)(wq * 32) << 16);
        const int r = wq * 32 + lane;                   // this thread's tile row = TMEM lane
        const bool row_valid = r < a.rows;
        // columns any row of this warp can see: the blocks its 32 rows belong to (causal: up to the row)
        const int w_lo = ((wq * 32) / a.block) * a.block;
        int w_hi = min(a.rows, ((wq * 32 + 31) / a.block + 1) * a.block);
        if (a.causal) w_hi = min(w_hi, wq * 32 + 32);
        const bool warp_valid = wq * 32 < a.rows;
        const int nchunks = (a.rows + 31) >> 5;
        const uint32_t s_col = tmem_lane + C::kColS + b * 128, p_col = tmem_lane + C::kColP + b * 64;
        const uint32_t o_col = tmem_lane + C::kColO + (kNO == 2 ? 64 * b : 0);

        bool ok = true;
        uint32_t o_seen = 0;                            // phases of o_full(b) consumed
        for (uint32_t t = b; ok && t < T; t += 2) {
            ok = mbar_wait_abortable(s_full(b), (t >> 1) & 1, 0xC0, abort_flag);
            ok = __all_sync(0xffffffffu, ok);           // keep the warp converged for the aligned TMEM ops
            if (!ok) break;
            tc_fence_after();
            const int xs = t % kNX;
            for (int f = 0; f < a.nf; ++f, ++o_seen) {
                // ---- softmax of this row over its mode-f vector; P (un-normalised, bf16) -> tensor memory
                const uint32_t *mword = masks + ((size_t)f * kTileRows + r) * 4;
                const bool x_f16 = f > 0 || a.x_f16 != 0;   // type of the value tile this hop multiplies
                const bool out_f16 = f + 1 < a.nf;          // between fused hops the tile is fp16; the last one writes bf16
                float m = -INFINITY;
                uint32_t v[32];
#pragma unroll 1
                for (int c = 0; c < nchunks; ++c) {
                    if (!(warp_valid && 32 * c < w_hi && 32 * c + 32 > w_lo)) continue;   // warp-uniform
                    tmem_ld32(s_col + 32 * c, v);
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
                        tmem_ld32(s_col + 32 * c, v);
                        const uint32_t bits = mword[c];
#pragma unroll
                        for (int jj = 0; jj < 32; jj += 2) {
                            float p0 = fast_exp2(__uint_as_float(v[jj]) * a.scale_log2 - m_scaled);
                            float p1 = fast_exp2(__uint_as_float(v[jj + 1]) * a.scale_log2 - m_scaled);
                            p0 = ((bits >> jj) & 1u) ? p0 : 0.f;
                            p1 = ((bits >> (jj + 1)) & 1u) ? p1 : 0.f;
                            uint32_t w;
                            if (x_f16) {
                                w = pack_f16x2(p0, p1);
                                sum += sum_f16x2(w);
                            } else {
                                w = pack_bf16x2(p0, p1);
                                sum += __uint_as_float(w << 16) + __uint_as_float(w & 0xFFFF0000u);
                            }
                            pk[jj >> 1] = w;
                        }
                    } else {
#pragma unroll
                        for (int jj = 0; jj < 16; ++jj) pk[jj] = 0u;
                    }
                    tmem_st16(p_col + 16 * c, pk);
                }
                tmem_st_wait();
                const float inv = row_valid ? 1.f / sum : 1.f;
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(p_full(b));

                // ---- X <- O / rowsum (bf16, in place in the value slot: the next fused hop's operand,
                // and after the last one the tile the store warp writes out)
                ok = mbar_wait_abortable(o_full(b), o_seen & 1, 0xC1, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                if (warp_valid) {
                    const uint32_t x_row = sX + xs * kTileBytes + (uint32_t)r * 128u;
#pragma unroll 1
                    for (int c = 0; c < D / 32; ++c) {
                        tmem_ld32(o_col + 32 * c, v);
                        uint32_t pk[16];
#pragma unroll
                        for (int jj = 0; jj < 32; jj += 2)
                            pk[jj >> 1] = out_f16 ? pack_f16x2(__uint_as_float(v[jj]) * inv, __uint_as_float(v[jj + 1]) * inv)
                                                  : pack_bf16x2(__uint_as_float(v[jj]) * inv, __uint_as_float(v[jj + 1]) * inv);
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
                fence_proxy_async_smem();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(o_free(b));
            }
            if (!ok) break;
            if (lane == 0) mbar_arrive(out_full(xs));
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
    a.x_f16 = hd.in_f16;
    for (int f = 0; f < TA_MAX_DIMS; ++f) {
        a.sub_n[f] = f < hd.nf ? hd.sub_n[f] : 1;
        a.sub_stride[f] = f < hd.nf ? hd.sub_stride[f] : 1;
        a.sub_window[f] = f < hd.nf ? pb.window[hd.sub_hop[f]] : 0;
    }
    int dev = 0;
    const int num_sms = current_device_sms(&dev);
    a.tiles_outer = hd.tiles_outer;
    // a work item = the gi query heads of a GQA group on one tile position (they share the K tile)
    const long long positions = (long long)pb.B * pb.H_kv * hd.tiles_outer;
    a.hsplit = 1;
    for (int d = 2; d <= a.g && positions * a.hsplit < 2ll * num_sms; ++d)
        if (a.g % d == 0) a.hsplit = d;
    a.gi = a.g / a.hsplit;
    a.total_items = positions * a.hsplit;
    a.scale_log2 = pb.scale * 1.4426950408889634f;
    constexpr size_t smem = FusedCfg<D>::kSmemBytes;
    auto kern = hop_fused_kernel<D>;
    static PerDeviceOnce configured;
    if (!configured.is_done(dev)) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return TA_ERR_CUDA;
        configured.mark(dev);
    }
    const unsigned grid = (unsigned)(a.total_items < num_sms ? a.total_items : num_sms);
    // after another hop of the same call: may start while that hop drains (see launch_hop_tc)
    const bool overlap = pb.pdl && a.total_items <= 32ll * num_sms;
    return launch_kernel(kern, grid, kThreads, smem, pb.stream, overlap, mq, mk, mxi, mxo, a);
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
