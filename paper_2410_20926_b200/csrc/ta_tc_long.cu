// Tensor-core kernel for one hop of tensorized attention over LONG segments (n_i > 128;
// ndims == 1 is ordinary attention over the whole sequence), bf16, head dim 64 or 128
// (Algorithm 1 loop body, Eq. 4; the softmax row no longer fits one tile, so it is taken
// block by block with a running maximum and sum -- "online" softmax in fp32).
//
// A work item is a pair of adjacent query tiles (2 x 128 consecutive positions) of one segment
// of one query head.  Their Q tiles stay in shared memory while the segment's keys go by ONCE in
// blocks of 128 (causal: up to each tile's diagonal block; with a window: only the blocks a
// tile can see); per tile c and key block j
//     S = Q_c K_j^T (tcgen05.mma, fp32 in TMEM)
//     m <- max(m, rowmax S),  alpha = 2^(m_old - m),  l <- alpha l + rowsum P,
//     P = 2^(S scale log2e - m)  (bf16, written back to TMEM over S)
//     O_c <- alpha O_c  (in TMEM, only when some row's maximum moved)   then   O_c += P X_j
// and finally O_c / l -> bf16 -> global memory (each thread owns one output row).  The two tiles
// belong to two softmax warpgroups that alternate on the tensor pipe: while one computes its
// softmax the MMAs of the other run.  Rows of the strided view are reached with the same rank-5
// TMA maps as the short-segment kernel (box = 128 positions of one segment); positions past n
// are zero-filled on load and skipped on store.  Several items read the value rows another item
// writes, so the hop is not in place: xin != xout.
//
// Persistent, one CTA per SM: warp 0 TMA producer (the Q pair per item, K_j / X_j into a
// two-stage ring shared by both tiles), warp 1 MMA issuer (polls for whichever of the two
// tiles' next MMA has its operands ready), warps 4-7 and 8-11 softmax / rescaling / epilogue of
// tile 0 and tile 1 (one TMEM lane = one query row per thread).  Every wait is bounded; when one
// expires the CTA raises a flag that ends all its roles, waits for its copies in flight, frees
// its TMEM and returns.
//
// Segments of a few tiles (n_i <= kSoloMaxN) take the kSolo instantiation instead: a work item is
// ONE query tile, a CTA has one chain (warps 4-7), single Q, K and X slots (96 KB at D = 128) and
// 256 TMEM columns, and TWO CTAs share an SM.  Such hops move about as many bytes per flop as the
// short-segment hops: what they need is loads in flight while a chain computes, and with a second
// CTA on the SM one CTA's loads run under the other's softmax and MMAs.
#include <cuda_bf16.h>
#include <stdlib.h>

#include "ta_internal.h"
#include "ta_ptx.cuh"

namespace ta {
namespace {

constexpr int kTileRows = 128;
constexpr int kThreads = 384;
constexpr int kNKV = 2;   // key / value block ring

struct LongArgs {
    int n, causal, g, H, H_kv, xin_is_kv, qblocks, qpairs;
    int window;                // 0, or w: keys within w positions of the query (blocks outside are skipped)
    long long stride, outer, total_items;
    long long row_stride, seg_outer_stride, head_stride;   // elements: between positions, outer blocks, heads
    float scale_log2;
    const int *lens;           // device, valid length per batch entry, or nullptr (kWindow variant only)
    int N;
    int pair_major;            // item numbering, see decode_long_item
    int tiles_per_item;        // 2: an item is a pair of query tiles; 1: a single tile (kSolo); qpairs counts items per segment
    // statistics pass of the backward: instead of the output rows, write per query row
    // (log2-sum-exp of the scaled scores, <G_t, O_t>) -- stats[q_head * N + token]; g = gradient
    // with respect to the hop's output, laid out like q
    float2 *stats;
    const __nv_bfloat16 *stats_g;
    // explicit mask of the dimension (kWindow variant only): bit matrix [n][mask_words] with the causal
    // flag and the window folded in, then per query block of 128 the range of key blocks it sees
    const uint32_t *mask_bits;
    int mask_words;
    int mask_heads;            // bit matrices (and range tables) behind mask_bits: 1 or H
};

constexpr int kSoloThreads = 256;
constexpr int kSoloMaxN = 1024;   // segments up to this length run one query tile per item, two CTAs per SM

template <int D, bool kSolo = false>
struct LongCfg {
    static constexpr int kHalves = D / 64;
    static constexpr int kChains = kSolo ? 1 : 2;
    static constexpr uint32_t kSlabBytes = kTileRows * 128;
    static constexpr uint32_t kTileBytes = kHalves * kSlabBytes;
    static constexpr uint32_t kOffQ = 0;                                   // the item's Q tiles
    // two chains: kNKV stages of (K block, X block); one chain: one K slot and one X slot (barrier
    // pair 0 is then K's, pair 1 X's)
    static constexpr uint32_t kOffKV = kOffQ + kChains * kTileBytes;
    static constexpr uint32_t kOffBar = kOffKV + (kSolo ? 1 : kNKV) * 2 * kTileBytes;
    static constexpr int kNumBars = 2 + 2 * kNKV + 6 + 1;
    static constexpr uint32_t kSmemBytes = kOffBar + kNumBars * 8 + 16 + 1024;
    static constexpr uint32_t kTmemCols = kSolo ? 256 : 512;
    // S_c at 128 c (P over its first 64 columns), then the O_c, 128 columns apart
    static constexpr uint32_t kColS = 0, kColO = 128 * kChains;
};

struct LongItem {
    int t0, inner, outer, q_head, kv_head;
    int ntiles;                // 1 or 2 query tiles (t0 and t0 + 128)
    int j0[2], je[2];          // key blocks [j0, je) of each tile (128 keys each)
    int keys_end[2];           // keys [.., keys_end) of each tile
    int jlo, jhi;              // union of the two ranges: the blocks the item loads
    int exist;                 // positions of the segment that are tokens (n without valid lengths)
};
// item -> (pair of query tiles, inner, outer, head).  Pairs of a segment are adjacent, later
// (longer, when causal) pairs first, so that the CTAs of one wave carry similar loads.
__device__ __forceinline__ LongItem decode_long_item(const LongArgs &a, long long item) {
    LongItem c;
    // Later (longer, when causal) pairs of query tiles first.  While the K and V of every head
    // together fit the L2, the pair is the slowest index: the numbering then runs from the longest
    // items to the shortest over the whole launch (see long_item_of_round), which evens out the
    // CTAs' loads.  Beyond that the pairs of a segment stay adjacent, so that a wave of CTAs works
    // on few heads and finds their K / V blocks in L2.
    int pb;
    long long rest;
    if (a.pair_major) {
        const long long per_pair = a.total_items / a.qpairs;
        pb = a.qpairs - 1 - (int)(item / per_pair);
        rest = item % per_pair;
    } else {
        pb = a.qpairs - 1 - (int)(item % a.qpairs);
        rest = item / a.qpairs;
    }
    c.inner = (int)(rest % a.stride); rest /= a.stride;
    c.outer = (int)(rest % a.outer); rest /= a.outer;
    c.q_head = (int)rest;                                          // b * H + h
    c.kv_head = (c.q_head / a.H) * a.H_kv + (c.q_head % a.H) / a.g;
    c.t0 = a.tiles_per_item * pb * kTileRows;
    c.ntiles = min(a.tiles_per_item, a.qblocks - a.tiles_per_item * pb);
    c.exist = a.n;
    if (a.lens != nullptr) {
        const long long len = min(max(__ldg(a.lens + c.q_head / a.H), 0), a.N);
        const long long first_token = (long long)c.outer * a.n * a.stride + c.inner;
        const long long left = (len - first_token + a.stride - 1) / a.stride;
        c.exist = len <= first_token ? 0 : (int)(left < a.n ? left : a.n);
    }
    int mask_lo = 0, mask_hi = 0;
    if (a.mask_bits != nullptr) {
        // (one range for the pair: the two tiles walk the same key blocks, as they do without a mask)
        const int mhead = a.mask_heads > 1 ? c.q_head % a.H : 0;
        const int *range = reinterpret_cast<const int *>(a.mask_bits + (size_t)a.mask_heads * a.n * a.mask_words) +
                           2 * ((size_t)mhead * a.qblocks + c.t0 / kTileRows);
        mask_lo = __ldg(range);
        mask_hi = __ldg(range + 1);
        if (c.ntiles == 2) {
            mask_lo = min(mask_lo, __ldg(range + 2));
            mask_hi = max(mask_hi, __ldg(range + 3));
        }
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int t0 = c.t0 + i * kTileRows;
        // keys any row of the tile can see: [first, keys_end)
        int first = 0;
        int keys_end = a.causal ? min(t0 + kTileRows, a.n) : a.n;
        if (a.window > 0) {
            first = max(0, t0 - a.window + 1);
            if (!a.causal) keys_end = min(a.n, t0 + kTileRows - 1 + a.window);
        }
        c.j0[i] = first / kTileRows;
        if (a.mask_bits != nullptr) {
            // key blocks before the first / after the last one the mask lets the item's query blocks see
            c.j0[i] = max(c.j0[i], mask_lo);
            keys_end = min(keys_end, mask_hi * kTileRows);
        }
        // padding keys are not visited, except that every tile keeps one block (its rows then see
        // nothing in it and come out as zeros), so that no role ever meets an empty chain
        keys_end = max(min(keys_end, c.exist), c.j0[i] * kTileRows + 1);
        c.keys_end[i] = keys_end;
        c.je[i] = (keys_end + kTileRows - 1) / kTileRows;
    }
    if (c.ntiles == 1) { c.j0[1] = c.je[1] = c.je[0]; }            // an absent tile has no blocks
    // no key block between the two tiles' ranges may be left to neither of them (the producer loads
    // the whole union): the second tile then walks such blocks too, seeing nothing in them
    if (c.ntiles == 2 && c.j0[1] > c.je[0]) c.j0[1] = c.je[0];
    c.jlo = c.j0[0];
    c.jhi = max(c.je[0], c.je[1]);
    return c;
}

// The item a CTA takes in its k-th round: the rounds run forth and back over the CTAs, so that the
// CTA that got the longest item of one round gets the shortest of the next.  -1: none in this round.
__device__ __forceinline__ long long long_item_of_round(const LongArgs &a, long long k) {
    const long long g = gridDim.x, b = blockIdx.x;
    const long long item = k * g + ((k & 1) ? g - 1 - b : b);
    return item < a.total_items ? item : -1;
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

template <int D, bool kWindow, bool kSolo>
__global__ void __launch_bounds__(kSolo ? kSoloThreads : kThreads, kSolo ? 2 : 1)
hop_long_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_xin, const __grid_constant__ CUtensorMap map_out,
                __nv_bfloat16 *__restrict__ xout, const LongArgs a) {
    using C = LongCfg<D, kSolo>;
    constexpr int kHalves = C::kHalves;
    constexpr uint32_t kSlabBytes = C::kSlabBytes, kTileBytes = C::kTileBytes;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t s0 = smem_u32(smem);
    auto sQ = [&](int c) { return s0 + C::kOffQ + (uint32_t)c * kTileBytes; };
    auto sKb = [&](int s) { return s0 + C::kOffKV + (uint32_t)s * 2 * kTileBytes; };
    auto sXb = [&](int s) { return s0 + C::kOffKV + (uint32_t)s * 2 * kTileBytes + kTileBytes; };
    const uint32_t bar0 = s0 + C::kOffBar;
    const uint32_t q_full = bar0, q_free = bar0 + 8;
    auto kv_full = [&](int i) { return bar0 + 8u * (uint32_t)(2 + i); };
    auto kv_free = [&](int i) { return bar0 + 8u * (uint32_t)(2 + kNKV + i); };
    constexpr int kB1 = 2 + 2 * kNKV;
    auto s_full = [&](int c) { return bar0 + 8u * (uint32_t)(kB1 + c); };        // S of tile c complete
    auto p_full = [&](int c) { return bar0 + 8u * (uint32_t)(kB1 + 2 + c); };    // P of tile c written (4 warps)
    auto pv_done = [&](int c) { return bar0 + 8u * (uint32_t)(kB1 + 4 + c); };   // value MMA of tile c complete
    const uint32_t out_full = bar0 + 8u * (uint32_t)(kB1 + 6);                   // kSolo: output tile staged (4 warps)
    uint32_t *tmem_slot = (uint32_t *)(smem + C::kOffBar + C::kNumBars * 8);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    for (uint32_t i = tid; i < C::kOffBar / 16; i += blockDim.x) ((uint4 *)smem)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) {
        for (int i = 0; i < C::kNumBars; ++i) {
            const uint32_t bar = bar0 + 8u * (uint32_t)i;
            mbar_init(bar, (bar == p_full(0) || bar == p_full(1) || bar == out_full) ? 4 : 1);   // one arrival per softmax warp
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
            uint32_t armed = 0, last_par = 0;        // bits: q 0, kv 1-2
            auto arm = [&](uint32_t bit, uint32_t parity) {
                armed |= bit;
                last_par = parity ? (last_par | bit) : (last_par & ~bit);
            };
            bool ok = true;
            for (long long round = 0; ok && round * gridDim.x < a.total_items; ++round, ++ic) {
                const long long item = long_item_of_round(a, round);
                if (item < 0) { --ic; continue; }
                const LongItem c = decode_long_item(a, item);
                const int x_head = a.xin_is_kv ? c.kv_head : c.q_head;
                ok = mbar_wait_abortable(q_free, (ic & 1) ^ 1, 0xD0, abort_flag);
                if (!ok) break;
                mbar_expect_tx(q_full, c.ntiles * kTileBytes);
                arm(1u, ic & 1);
                for (int i = 0; i < c.ntiles; ++i)
#pragma unroll
                    for (int h = 0; h < kHalves; ++h)
                        tma_load_5d(sQ(i) + h * kSlabBytes, &map_q, q_full, 64 * h, c.t0 + kTileRows * i, c.inner, c.outer, c.q_head);
                if constexpr (kSolo) {
                    // one K slot (barrier pair 0) and one X slot (pair 1), block after block
                    for (int j = c.jlo; j < c.jhi; ++j, ++g) {
                        const uint32_t par = g & 1;
                        ok = mbar_wait_abortable(kv_free(0), par ^ 1, 0xD1, abort_flag);
                        if (!ok) break;
                        mbar_expect_tx(kv_full(0), kTileBytes);
                        arm(2u, par);
#pragma unroll
                        for (int h = 0; h < kHalves; ++h)
                            tma_load_5d(sKb(0) + h * kSlabBytes, &map_k, kv_full(0), 64 * h, kTileRows * j, c.inner, c.outer, c.kv_head);
                        ok = mbar_wait_abortable(kv_free(1), par ^ 1, 0xD2, abort_flag);
                        if (!ok) break;
                        mbar_expect_tx(kv_full(1), kTileBytes);
                        arm(4u, par);
#pragma unroll
                        for (int h = 0; h < kHalves; ++h)
                            tma_load_5d(sXb(0) + h * kSlabBytes, &map_xin, kv_full(1), 64 * h, kTileRows * j, c.inner, c.outer, x_head);
                    }
                } else
                for (int j = c.jlo; j < c.jhi; ++j, ++g) {
                    const int st = g % kNKV;
                    const uint32_t par = (g / kNKV) & 1;
                    ok = mbar_wait_abortable(kv_free(st), par ^ 1, 0xD1, abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(kv_full(st), 2 * kTileBytes);
                    arm(2u << st, par);
#pragma unroll
                    for (int h = 0; h < kHalves; ++h)
                        tma_load_5d(sKb(st) + h * kSlabBytes, &map_k, kv_full(st), 64 * h, kTileRows * j, c.inner, c.outer, c.kv_head);
#pragma unroll
                    for (int h = 0; h < kHalves; ++h)
                        tma_load_5d(sXb(st) + h * kSlabBytes, &map_xin, kv_full(st), 64 * h, kTileRows * j, c.inner, c.outer, x_head);
                }
            }
            if (!ok) {
                const unsigned long long t0 = globaltimer_ns();
                for (int slot = 0; slot < 1 + kNKV; ++slot) {
                    if (!(armed & (1u << slot))) continue;
                    const uint32_t bar = slot == 0 ? q_full : kv_full(slot - 1);
                    while (!mbar_try_wait(bar, (last_par >> slot) & 1u) && globaltimer_ns() - t0 < 10000000ull) {
                    }
                }
            }
        }
    } else if (warp == 1) {
        // =============================================================== MMA issuer
        // Two chains (the item's two query tiles) share the key blocks.  Chain c alternates
        // S_c(j) = Q_c K_j^T and O_c += P_c(j) X_j; its single S buffer is free again once the
        // value MMA that reads P from it has been issued.  A key block's stage is released when
        // the last chain that uses the block has issued its value MMA.
        if (lane == 0) {
            constexpr uint32_t idesc_s = instr_desc(128, 0);
            constexpr uint32_t idesc_o = instr_desc(D, 1);
            uint32_t ic = 0, g0 = 0;
            uint32_t p_seen[2] = {0, 0};              // phases of p_full(c) consumed
            bool ok = true;
            for (long long round = 0; ok && round * gridDim.x < a.total_items; ++round, ++ic) {
                const long long item = long_item_of_round(a, round);
                if (item < 0) { --ic; continue; }
                const LongItem c = decode_long_item(a, item);
                ok = mbar_wait_abortable(q_full, ic & 1, 0xE0, abort_flag);
                if (!ok) break;
                if constexpr (kSolo) {
                    // one chain, in order: S(j), then O += P(j) X_j once the softmax warps have written P
                    for (int j = c.j0[0]; ok && j < c.je[0]; ++j, ++g0) {
                        const uint32_t par = g0 & 1;
                        ok = mbar_wait_abortable(kv_full(0), par, 0xE1, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
#pragma unroll
                        for (int kb = 0; kb < D / 16; ++kb) {
                            const uint32_t off = (kb >> 2) * kSlabBytes + (kb & 3) * 32;
                            tc_mma_ss(tmem_base + C::kColS, smem_desc_sw128(sQ(0) + off, 16, 1024),
                                      smem_desc_sw128(sKb(0) + off, 16, 1024), idesc_s, kb > 0);
                        }
                        tc_commit(s_full(0));
                        tc_commit(kv_free(0));
                        if (j == c.je[0] - 1) tc_commit(q_free);
                        ok = mbar_wait_abortable(p_full(0), p_seen[0] & 1, 0xE2, abort_flag);
                        if (!ok) break;
                        ++p_seen[0];
                        ok = mbar_wait_abortable(kv_full(1), par, 0xE3, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        const int keys = min(kTileRows, c.keys_end[0] - kTileRows * j);
                        const int kblocks = (keys + 15) >> 4;
                        for (int kb = 0; kb < kblocks; ++kb)
                            tc_mma_ts(tmem_base + C::kColO, tmem_base + C::kColS + kb * 8,
                                      smem_desc_sw128(sXb(0) + kb * 2048, kSlabBytes, 1024), idesc_o,
                                      (kb > 0 || j > c.j0[0]) ? 1u : 0u);
                        tc_commit(pv_done(0));
                        // (the X slot of a tile's last block takes the output tile next: the store thread frees it)
                        if (j < c.je[0] - 1) tc_commit(kv_free(1));
                    }
                    continue;
                }
                int js[2] = {c.j0[0], c.j0[1]};       // next block whose S is to be issued
                int jp[2] = {c.j0[0], c.j0[1]};       // next block whose value MMA is to be issued
                bool q_released = false;
                uint32_t idle = 0;
                unsigned long long idle_since = 0;
                while (jp[0] < c.je[0] || jp[1] < c.je[1]) {
                    bool progressed = false;
#pragma unroll
                    for (int ch = 0; ch < 2; ++ch) {
                        // ---- S_ch(js)
                        if (js[ch] < c.je[ch] && js[ch] == jp[ch]) {
                            const uint32_t g = g0 + (uint32_t)(js[ch] - c.jlo);
                            const int st = g % kNKV;
                            if (mbar_test_wait(kv_full(st), (g / kNKV) & 1)) {
                                tc_fence_after();
#pragma unroll
                                for (int kb = 0; kb < D / 16; ++kb) {
                                    const uint32_t off = (kb >> 2) * kSlabBytes + (kb & 3) * 32;
                                    tc_mma_ss(tmem_base + C::kColS + ch * 128, smem_desc_sw128(sQ(ch) + off, 16, 1024),
                                              smem_desc_sw128(sKb(st) + off, 16, 1024), idesc_s, kb > 0);
                                }
                                tc_commit(s_full(ch));
                                ++js[ch];
                                progressed = true;
                            }
                        }
                        // ---- O_ch += P_ch(jp) X_jp
                        if (jp[ch] < js[ch] && mbar_test_wait(p_full(ch), p_seen[ch] & 1)) {
                            const int j = jp[ch];
                            const uint32_t g = g0 + (uint32_t)(j - c.jlo);
                            const int st = g % kNKV;
                            tc_fence_after();
                            const int keys = min(kTileRows, c.keys_end[ch] - kTileRows * j);
                            const int kblocks = (keys + 15) >> 4;
                            for (int kb = 0; kb < kblocks; ++kb)
                                tc_mma_ts(tmem_base + C::kColO + ch * 128, tmem_base + C::kColS + ch * 128 + kb * 8,
                                          smem_desc_sw128(sXb(st) + kb * 2048, kSlabBytes, 1024), idesc_o,
                                          (kb > 0 || j > c.j0[ch]) ? 1u : 0u);
                            tc_commit(pv_done(ch));
                            ++p_seen[ch];
                            ++jp[ch];
                            // release the key block once the other chain is past it (or never uses it)
                            const int o = ch ^ 1;
                            if (!(j >= c.j0[o] && j < c.je[o]) || jp[o] > j) tc_commit(kv_free(st));
                            progressed = true;
                        }
                    }
                    if (!q_released && js[0] == c.je[0] && js[1] == c.je[1]) {
                        tc_commit(q_free);            // every S of this item has been issued
                        q_released = true;
                    }
                    if (progressed) {
                        idle = 0;
                        idle_since = 0;
                    } else if (++idle < 1024) {
                        __nanosleep(20);
                    } else {
                        idle = 0;
                        if (*abort_flag) { ok = false; break; }
                        const unsigned long long now = globaltimer_ns();
                        if (idle_since == 0) idle_since = now;
                        if (now - idle_since > kWaitLimitNs) {
                            atomicCAS(&g_status_word, 0u, kErrWaitExpired | 0xE5u);
                            *abort_flag = 1u;
                            ok = false;
                            break;
                        }
                    }
                }
                g0 += (uint32_t)(c.jhi - c.jlo);
            }
        }
    } else if (kSolo && warp == 2) {
        // =============================================================== TMA store of finished tiles (kSolo)
        // The softmax warps stage the output tile in the X slot of the tile's last key block; the
        // slot goes back to the producer once the store has read it.
        if (lane == 0) {
            uint32_t ic = 0;
            bool ok = true;
            for (long long round = 0; ok && round * gridDim.x < a.total_items; ++round) {
                const long long item = long_item_of_round(a, round);
                if (item < 0) continue;
                const LongItem c = decode_long_item(a, item);
                ok = mbar_wait_abortable(out_full, ic & 1, 0xC0, abort_flag);
                if (!ok) break;
                ++ic;
                if (a.stats == nullptr) {
#pragma unroll
                    for (int h = 0; h < kHalves; ++h)
                        tma_store_5d(&map_out, sXb(0) + h * kSlabBytes, 64 * h, c.t0, c.inner, c.outer, c.q_head);
                    tma_store_commit_and_wait_read();
                }
                mbar_arrive(kv_free(1));
            }
            tma_store_wait_all();
        }
    } else if (warp >= 4) {
        // =============================================================== softmax, rescaling, epilogue
        const int ch = kSolo ? 0 : (warp - 4) >> 2;     // which of the item's query tiles
        const int wq = warp & 3;                        // TMEM lane quarter of this warp
        const uint32_t tmem_lane = tmem_base + ((uint32_t)(wq * 32) << 16);
        const int r = wq * 32 + lane;                   // this thread's query row of the tile
        const uint32_t s_col = tmem_lane + C::kColS + ch * 128;
        const uint32_t o_col = tmem_lane + C::kColO + ch * 128;

        bool ok = true;
        uint32_t blocks_seen = 0;                       // key blocks this chain has processed (all items)
        for (long long round = 0; ok && round * gridDim.x < a.total_items; ++round) {
            const long long item = long_item_of_round(a, round);
            if (item < 0) continue;
            const LongItem c = decode_long_item(a, item);
            if (ch >= c.ntiles) continue;
            const int t = c.t0 + kTileRows * ch + r;    // position of this row in the segment
            const bool row_valid = t < a.n;
            const int keys_end = c.keys_end[ch];
            float m_run = -INFINITY, l_run = 0.f;       // running maximum (scaled, log2 domain) and sum
            for (int j = c.j0[ch]; j < c.je[ch]; ++j, ++blocks_seen) {
                const int u0 = kTileRows * j;
                const int keys = min(kTileRows, keys_end - u0);            // key columns of this block
                // columns any row of this warp can see in this block (warp-uniform)
                const bool diag = a.causal && u0 == c.t0 + kTileRows * ch;
                const int w_hi = diag ? min(keys, wq * 32 + 32) : keys;
                // this row: columns [c_lo, c_hi) of the block
                int c_hi = !row_valid ? 0 : (diag ? min(keys, r + 1) : keys);
                int c_lo = 0;                           // stays a compile-time 0 without a window
                if (kWindow) {
                    if (a.window > 0) {
                        c_lo = max(0, t - a.window + 1 - u0);
                        if (!a.causal) c_hi = min(c_hi, t + a.window - u0);
                    }
                    c_hi = t < c.exist ? min(c_hi, c.exist - u0) : 0;     // valid length: padding keys, padding rows
                }
                // explicit mask: this row's 128 bits over the block's keys (all ones without a mask)
                uint4 mrow = make_uint4(~0u, ~0u, ~0u, ~0u);
                if (kWindow && a.mask_bits != nullptr && row_valid)
                    mrow = __ldg(reinterpret_cast<const uint4 *>(
                        a.mask_bits + ((size_t)(a.mask_heads > 1 ? c.q_head % a.H : 0) * a.n + t) * a.mask_words + 4 * j));
                auto mask_word = [&](int cc) { return cc == 0 ? mrow.x : (cc == 1 ? mrow.y : (cc == 2 ? mrow.z : mrow.w)); };
                const int nchunks = (keys + 31) >> 5;

                ok = mbar_wait_abortable(s_full(ch), blocks_seen & 1, 0xF4, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();

                // 32-column chunks every row of this warp sees completely need no per-element masks (all
                // of a block below the diagonal; in the diagonal block the chunks left of the warp's own)
                uint32_t my_full = 0;
                if (!kWindow) {
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc)
                        if (32 * cc + 32 <= c_hi) my_full |= 1u << cc;
                }
                const uint32_t full_bits = kWindow ? 0u : __reduce_and_sync(0xffffffffu, my_full);
                // (with two chains per CTA a block every row sees completely -- most blocks of a long
                // segment -- has loops of its own: measured 11 % faster there, and 9 % slower with one)
                const bool full_w = !kSolo && full_bits == 0xFu;
                float bm = -INFINITY;
                uint32_t v[32];
                if (full_w) {
#pragma unroll 1
                    for (int cc = 0; cc < 4; ++cc) {
                        tmem_ld32(s_col + 32 * cc, v);
                        float b0 = fmaxf(__uint_as_float(v[0]), __uint_as_float(v[1]));
                        float b1 = fmaxf(__uint_as_float(v[2]), __uint_as_float(v[3]));
#pragma unroll
                        for (int jj = 4; jj < 32; jj += 4) {
                            b0 = fmaxf(b0, fmaxf(__uint_as_float(v[jj]), __uint_as_float(v[jj + 1])));
                            b1 = fmaxf(b1, fmaxf(__uint_as_float(v[jj + 2]), __uint_as_float(v[jj + 3])));
                        }
                        bm = fmaxf(bm, fmaxf(b0, b1));
                    }
                } else
#pragma unroll 1
                for (int cc = 0; cc < nchunks; ++cc) {
                    if (32 * cc >= w_hi) continue;          // warp-uniform
                    tmem_ld32(s_col + 32 * cc, v);
                    if ((full_bits >> cc) & 1u) {
                        float b0 = fmaxf(__uint_as_float(v[0]), __uint_as_float(v[1]));
                        float b1 = fmaxf(__uint_as_float(v[2]), __uint_as_float(v[3]));
#pragma unroll
                        for (int jj = 4; jj < 32; jj += 4) {
                            b0 = fmaxf(b0, fmaxf(__uint_as_float(v[jj]), __uint_as_float(v[jj + 1])));
                            b1 = fmaxf(b1, fmaxf(__uint_as_float(v[jj + 2]), __uint_as_float(v[jj + 3])));
                        }
                        bm = fmaxf(bm, fmaxf(b0, b1));
                    } else {
                        const uint32_t mw = kWindow ? mask_word(cc) : ~0u;
#pragma unroll
                        for (int jj = 0; jj < 32; ++jj)
                            if (32 * cc + jj >= c_lo && 32 * cc + jj < c_hi && ((mw >> jj) & 1u))
                                bm = fmaxf(bm, __uint_as_float(v[jj]));
                    }
                }
                // (with a window a row may see nothing in a block: the running maximum then stays -inf
                // until its first visible key, and the reference below keeps the arithmetic finite)
                const float m_new = fmaxf(m_run, bm * a.scale_log2);
                const float m_ref = m_new == -INFINITY ? 0.f : m_new;
                const float alpha = m_run == -INFINITY ? 1.f : fast_exp2(m_run - m_ref);

                // ---- O <- alpha O, once the previous block's value MMA has completed
                if (j > c.j0[ch]) {
                    ok = mbar_wait_abortable(pv_done(ch), (blocks_seen - 1) & 1, 0xF5, abort_flag);
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

                // ---- P (un-normalised, bf16) over the S columns already consumed
                // (over a chunk without masks the row sum is taken over the fp32 weights: the rounding of
                // P averages out; elsewhere over the rounded weights)
                float sum = 0.f, sum1 = 0.f;
                if (full_w) {
#pragma unroll 1
                    for (int cc = 0; cc < 4; ++cc) {
                        uint32_t pk[16];
                        tmem_ld32(s_col + 32 * cc, v);
#pragma unroll
                        for (int jj = 0; jj < 32; jj += 2) {
                            const float p0 = fast_exp2(fmaf(__uint_as_float(v[jj]), a.scale_log2, -m_ref));
                            const float p1 = fast_exp2(fmaf(__uint_as_float(v[jj + 1]), a.scale_log2, -m_ref));
                            pk[jj >> 1] = pack_bf16x2(p0, p1);
                            sum += p0;
                            sum1 += p1;
                        }
                        tmem_st16(s_col + 16 * cc, pk);
                    }
                } else
#pragma unroll 1
                for (int cc = 0; cc < nchunks; ++cc) {
                    uint32_t pk[16];
                    if (32 * cc >= w_hi) {
#pragma unroll
                        for (int jj = 0; jj < 16; ++jj) pk[jj] = 0u;
                    } else if ((full_bits >> cc) & 1u) {
                        tmem_ld32(s_col + 32 * cc, v);
#pragma unroll
                        for (int jj = 0; jj < 32; jj += 2) {
                            const float p0 = fast_exp2(fmaf(__uint_as_float(v[jj]), a.scale_log2, -m_ref));
                            const float p1 = fast_exp2(fmaf(__uint_as_float(v[jj + 1]), a.scale_log2, -m_ref));
                            pk[jj >> 1] = pack_bf16x2(p0, p1);
                            sum += p0;
                            sum1 += p1;
                        }
                    } else {
                        tmem_ld32(s_col + 32 * cc, v);
                        const uint32_t mw = kWindow ? mask_word(cc) : ~0u;
#pragma unroll
                        for (int jj = 0; jj < 32; jj += 2) {
                            const int col = 32 * cc + jj;
                            float p0 = fast_exp2(__uint_as_float(v[jj]) * a.scale_log2 - m_ref);
                            float p1 = fast_exp2(__uint_as_float(v[jj + 1]) * a.scale_log2 - m_ref);
                            p0 = (col >= c_lo && col < c_hi && ((mw >> jj) & 1u)) ? p0 : 0.f;
                            p1 = (col + 1 >= c_lo && col + 1 < c_hi && ((mw >> (jj + 1)) & 1u)) ? p1 : 0.f;
                            const uint32_t w = pack_bf16x2(p0, p1);
                            pk[jj >> 1] = w;
                            sum += __uint_as_float(w << 16) + __uint_as_float(w & 0xFFFF0000u);
                        }
                    }
                    tmem_st16(s_col + 16 * cc, pk);
                }
                sum += sum1;
                tmem_st_wait();
                l_run = l_run * alpha + sum;
                m_run = m_new;
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(p_full(ch));
            }
            if (!ok) break;

            // ---- epilogue: O / l -> bf16 -> this thread's output row in global memory
            ok = mbar_wait_abortable(pv_done(ch), (blocks_seen - 1) & 1, 0xF6, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            if (a.stats != nullptr) {
                const float inv = (row_valid && l_run > 0.f) ? 1.f / l_run : 0.f;
                const long long row_off = (long long)c.q_head * a.head_stride + (long long)c.outer * a.seg_outer_stride +
                                          (long long)t * a.row_stride + (long long)c.inner * D;
                const __nv_bfloat16 *grow = a.stats_g + row_off;
                float dot = 0.f;
                uint32_t v[32];
#pragma unroll 1
                for (int cc = 0; cc < D / 32; ++cc) {
                    tmem_ld32(o_col + 32 * cc, v);
                    if (row_valid) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const uint4 w = __ldg(reinterpret_cast<const uint4 *>(grow + 32 * cc + 8 * i));
                            const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                dot = fmaf(__uint_as_float(ws[e] << 16), __uint_as_float(v[8 * i + 2 * e]), dot);
                                dot = fmaf(__uint_as_float(ws[e] & 0xFFFF0000u), __uint_as_float(v[8 * i + 2 * e + 1]), dot);
                            }
                        }
                    }
                }
                if (row_valid)
                    a.stats[row_off / D] = make_float2(l_run > 0.f ? m_run + log2f(l_run) : INFINITY, dot * inv);
            } else if constexpr (kSolo) {
                // O / l -> bf16 -> the X slot (swizzled box layout) -> store thread
                const float inv = (row_valid && l_run > 0.f) ? 1.f / l_run : 0.f;
                const uint32_t x_row = sXb(0) + (uint32_t)r * 128u;
                uint32_t v[32];
#pragma unroll 1
                for (int cc = 0; cc < D / 32; ++cc) {
                    tmem_ld32(o_col + 32 * cc, v);
                    uint32_t pk[16];
#pragma unroll
                    for (int jj = 0; jj < 32; jj += 2)
                        pk[jj >> 1] = pack_bf16x2(__uint_as_float(v[jj]) * inv, __uint_as_float(v[jj + 1]) * inv);
                    const uint32_t slab = x_row + (uint32_t)(cc >> 1) * kSlabBytes;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint32_t chunk = (uint32_t)(((cc & 1) * 4 + i) ^ (r & 7));
                        st_shared_v4(slab + chunk * 16, pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
                    }
                }
                fence_proxy_async_smem();
            } else {
                const float inv = (row_valid && l_run > 0.f) ? 1.f / l_run : 0.f;
                __nv_bfloat16 *dst = xout + (long long)c.q_head * a.head_stride + (long long)c.outer * a.seg_outer_stride +
                                     (long long)t * a.row_stride + (long long)c.inner * D;
                uint32_t v[32];
#pragma unroll 1
                for (int cc = 0; cc < D / 32; ++cc) {
                    tmem_ld32(o_col + 32 * cc, v);      // whole warp; rows past n discard it
                    if (row_valid) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            uint4 w;
                            w.x = pack_bf16x2(__uint_as_float(v[8 * i]) * inv, __uint_as_float(v[8 * i + 1]) * inv);
                            w.y = pack_bf16x2(__uint_as_float(v[8 * i + 2]) * inv, __uint_as_float(v[8 * i + 3]) * inv);
                            w.z = pack_bf16x2(__uint_as_float(v[8 * i + 4]) * inv, __uint_as_float(v[8 * i + 5]) * inv);
                            w.w = pack_bf16x2(__uint_as_float(v[8 * i + 6]) * inv, __uint_as_float(v[8 * i + 7]) * inv);
                            *reinterpret_cast<uint4 *>(dst + 32 * cc + 8 * i) = w;
                        }
                    }
                }
            }
            tc_fence_before();
            if constexpr (kSolo) {
                __syncwarp();
                if (lane == 0) mbar_arrive(out_full);
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 3) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::kTmemCols) : "memory");
    }
}

// Longest segment that runs one query tile per item (env TA_LONG_SOLO_MAX_N overrides, for measurements)
int solo_max_n() {
    static const int v = [] {
        const char *e = getenv("TA_LONG_SOLO_MAX_N");
        return e ? atoi(e) : kSoloMaxN;
    }();
    return v;
}

template <int D>
int launch_long_d(const Problem &pb, const HopDesc &hd, const void *xin, int xin_heads, void *xout, void *stats = nullptr,
                  const void *stats_g = nullptr) {
    CUtensorMap mq, mk, mxi;
    int rc;
    // box: 128 positions of one segment (positions past n are zero-filled / clipped)
    if ((rc = make_view_map(&mq, pb.q, pb.B * pb.H, pb.N, D, hd, 2, kTileRows, 1, 1)) != TA_OK) return rc;
    if ((rc = make_view_map(&mk, pb.k, pb.B * pb.H_kv, pb.N, D, hd, 2, kTileRows, 1, 1)) != TA_OK) return rc;
    if ((rc = make_view_map(&mxi, xin, pb.B * xin_heads, pb.N, D, hd, 2, kTileRows, 1, 1)) != TA_OK) return rc;
    // (the statistics pass writes no output rows: its map is never used)
    CUtensorMap mo = mq;
    if (xout && (rc = make_view_map(&mo, xout, pb.B * pb.H, pb.N, D, hd, 2, kTileRows, 1, 1)) != TA_OK) return rc;

    LongArgs a;
    a.n = hd.n; a.causal = pb.causal; a.g = pb.H / pb.H_kv; a.H = pb.H; a.H_kv = pb.H_kv;
    a.xin_is_kv = xin_heads != pb.H ? 1 : 0;
    a.tiles_per_item = long_tiles_per_item(hd.n);
    const bool solo = a.tiles_per_item == 1;
    a.qblocks = (hd.n + kTileRows - 1) / kTileRows;
    a.qpairs = (a.qblocks + a.tiles_per_item - 1) / a.tiles_per_item;
    a.stride = hd.stride; a.outer = hd.outer;
    a.total_items = (long long)pb.B * pb.H * hd.outer * hd.stride * a.qpairs;
    a.row_stride = hd.stride * (long long)D;
    a.seg_outer_stride = (long long)hd.n * hd.stride * D;
    a.head_stride = (long long)pb.N * D;
    a.window = pb.window[hd.hop];
    a.scale_log2 = pb.scale * 1.4426950408889634f;
    a.lens = pb.seq_lens;
    a.N = pb.N;
    // K and V of all heads (bf16) against the 126 MB L2
    a.pair_major = 2ull * pb.B * pb.H_kv * pb.N * D * 2 <= (96ull << 20) ? 1 : 0;
    a.stats = (float2 *)stats;
    a.stats_g = (const __nv_bfloat16 *)stats_g;
    a.mask_bits = pb.masks[hd.hop] ? pb.dmask[hd.hop] : nullptr;
    a.mask_words = pb.dmask_words[hd.hop];
    a.mask_heads = pb.masks_per_head ? pb.H : 1;
    if (pb.masks[hd.hop] && !a.mask_bits) return TA_ERR_INVALID_ARG;

    int dev = 0;
    const int num_sms = current_device_sms(&dev);
    constexpr size_t smem = LongCfg<D>::kSmemBytes, smem_solo = LongCfg<D, true>::kSmemBytes;
    static PerDeviceOnce configured;
    if (!configured.is_done(dev)) {
        const auto dyn = cudaFuncAttributeMaxDynamicSharedMemorySize;
        const auto carve = cudaFuncAttributePreferredSharedMemoryCarveout;
        if (cudaFuncSetAttribute(hop_long_kernel<D, false, false>, dyn, (int)smem) != cudaSuccess ||
            cudaFuncSetAttribute(hop_long_kernel<D, true, false>, dyn, (int)smem) != cudaSuccess ||
            cudaFuncSetAttribute(hop_long_kernel<D, false, true>, dyn, (int)smem_solo) != cudaSuccess ||
            cudaFuncSetAttribute(hop_long_kernel<D, true, true>, dyn, (int)smem_solo) != cudaSuccess ||
            cudaFuncSetAttribute(hop_long_kernel<D, false, true>, carve, 100) != cudaSuccess ||
            cudaFuncSetAttribute(hop_long_kernel<D, true, true>, carve, 100) != cudaSuccess)
            return TA_ERR_CUDA;
        configured.mark(dev);
    }
    const bool windowed = a.window > 0 || a.lens != nullptr || a.mask_bits != nullptr;
    if (solo) {
        // two CTAs per SM
        const unsigned grid = (unsigned)(a.total_items < 2LL * num_sms ? a.total_items : 2LL * num_sms);
        if (windowed)
            return launch_kernel(hop_long_kernel<D, true, true>, grid, kSoloThreads, smem_solo, pb.stream, false, mq, mk,
                                 mxi, mo, (__nv_bfloat16 *)xout, a);
        return launch_kernel(hop_long_kernel<D, false, true>, grid, kSoloThreads, smem_solo, pb.stream, false, mq, mk, mxi, mo,
                             (__nv_bfloat16 *)xout, a);
    }
    const unsigned grid = (unsigned)(a.total_items < num_sms ? a.total_items : num_sms);
    if (windowed)
        return launch_kernel(hop_long_kernel<D, true, false>, grid, kThreads, smem, pb.stream, false, mq, mk, mxi, mo,
                             (__nv_bfloat16 *)xout, a);
    return launch_kernel(hop_long_kernel<D, false, false>, grid, kThreads, smem, pb.stream, false, mq, mk, mxi, mo,
                         (__nv_bfloat16 *)xout, a);
}

}  // namespace

// Tensorized positional encoding (Section 3.2) for a long-segment hop: dst = src with every row
// rotated by its coordinate along the hop's dimension (feature c paired with c + D/2, angle
// position * base^(-2c/D)).  A long hop re-reads each K block once per pair of query tiles, so
// rotating inside the pipeline would repeat the work n / 256 times; one elementwise pass over Q
// and K costs two reads and writes of them against a hop whose time grows with n.  The angle is
// reduced modulo 2 pi in double precision (positions reach 10^5, where an fp32 product is off by
// milliradians).
namespace {
__global__ void rope_copy_kernel(const __nv_bfloat16 *__restrict__ src, __nv_bfloat16 *__restrict__ dst,
                                 long long pairs, int N, int D, long long stride, int n, double log2_base) {
    const int half = D >> 1;
    for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < pairs;
         idx += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(idx % half);
        const long long row = idx / half;                       // head * N + token
        const long long token = row % N;
        const int pos = (int)((token / stride) % n);
        const double theta = exp2(-2.0 * (double)c / (double)D * log2_base);
        const double angle = fmod((double)pos * theta, 6.283185307179586476925);
        float sn, cs;
        sincosf((float)angle, &sn, &cs);
        const long long o = row * D + c;
        const float x1 = __bfloat162float(src[o]), x2 = __bfloat162float(src[o + half]);
        dst[o] = __float2bfloat16_rn(x1 * cs - x2 * sn);
        dst[o + half] = __float2bfloat16_rn(x2 * cs + x1 * sn);
    }
}
}  // namespace

// dst (fp32) = or += the transposed rotation of src (fp32): gradients with respect to rotated
// vectors turned back to gradients with respect to the un-rotated ones.
namespace {
__global__ void rope_unrotate_add_kernel(const float *__restrict__ src, float *__restrict__ dst, long long pairs, int N,
                                         int D, long long stride, int n, double log2_base, int accumulate) {
    const int half = D >> 1;
    for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < pairs;
         idx += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(idx % half);
        const long long row = idx / half;
        const long long token = row % N;
        const int pos = (int)((token / stride) % n);
        const double theta = exp2(-2.0 * (double)c / (double)D * log2_base);
        const double angle = fmod((double)pos * theta, 6.283185307179586476925);
        float sn, cs;
        sincosf((float)angle, &sn, &cs);
        const long long o = row * D + c;
        const float x1 = src[o], x2 = src[o + half];
        const float y1 = x1 * cs + x2 * sn, y2 = x2 * cs - x1 * sn;
        dst[o] = accumulate ? dst[o] + y1 : y1;
        dst[o + half] = accumulate ? dst[o + half] + y2 : y2;
    }
}
unsigned rope_blocks(long long pairs) { return (unsigned)(pairs / 256 + 1 < 148 * 32 ? pairs / 256 + 1 : 148 * 32); }
}  // namespace

// Rotated bf16 copies of q and k for hop `hd` in a pooled buffer (*pooled, stream-ordered), followed
// by `extra_bytes` of scratch (*extra).
int rope_rotated_copies(const Problem &pb, const HopDesc &hd, const void **rq_out, const void **rk_out,
                        size_t extra_bytes, void **extra, void **pooled) {
    const size_t tq = (size_t)pb.B * pb.H * pb.N * pb.D, tkv = (size_t)pb.B * pb.H_kv * pb.N * pb.D;
    const size_t q_bytes = (tq * 2 + 255) & ~(size_t)255, k_bytes = (tkv * 2 + 255) & ~(size_t)255;
    void *buf = nullptr;
    int rc = pool_alloc(q_bytes + k_bytes + extra_bytes, pb.stream, &buf);
    if (rc != TA_OK) return rc;
    *pooled = buf;
    __nv_bfloat16 *rq = (__nv_bfloat16 *)buf, *rk = (__nv_bfloat16 *)((char *)buf + q_bytes);
    const double log2_base = log2((double)pb.rope_base);
    const long long pq = (long long)(tq / 2), pk = (long long)(tkv / 2);
    rc = launch_kernel(rope_copy_kernel, rope_blocks(pq), 256, 0, pb.stream, false, (const __nv_bfloat16 *)pb.q, rq, pq,
                       pb.N, pb.D, (long long)hd.stride, hd.n, log2_base);
    if (rc != TA_OK) return rc;
    rc = launch_kernel(rope_copy_kernel, rope_blocks(pk), 256, 0, pb.stream, false, (const __nv_bfloat16 *)pb.k, rk, pk,
                       pb.N, pb.D, (long long)hd.stride, hd.n, log2_base);
    if (rc != TA_OK) return rc;
    *rq_out = rq;
    *rk_out = rk;
    if (extra) *extra = (char *)buf + q_bytes + k_bytes;
    return TA_OK;
}

int rope_unrotate_add(const Problem &pb, const HopDesc &hd, const float *src, float *dst, int heads, bool accumulate) {
    const long long pairs = (long long)pb.B * heads * pb.N * pb.D / 2;
    return launch_kernel(rope_unrotate_add_kernel, rope_blocks(pairs), 256, 0, pb.stream, false, src, dst, pairs, pb.N,
                         pb.D, (long long)hd.stride, hd.n, log2((double)pb.rope_base), accumulate ? 1 : 0);
}

int long_tiles_per_item(int n) { return n <= solo_max_n() ? 1 : 2; }

int launch_hop_tc_long(const Problem &pb, const HopDesc &hd, const void *xin, int xin_heads, void *xout) {
    if (xin == xout) return TA_ERR_INVALID_ARG;
    if (pb.D != 128 && pb.D != 64) return TA_ERR_UNSUPPORTED;
    Problem hop = pb;
    void *pooled = nullptr;
    if (pb.rope_base > 0.f) {
        const int rc = rope_rotated_copies(pb, hd, &hop.q, &hop.k, 0, nullptr, &pooled);
        if (rc != TA_OK) {
            pool_free(pooled, pb.stream);
            return rc;
        }
        hop.rope_base = 0.f;
    }
    const int rc = pb.D == 128 ? launch_long_d<128>(hop, hd, xin, xin_heads, xout)
                               : launch_long_d<64>(hop, hd, xin, xin_heads, xout);
    pool_free(pooled, pb.stream);
    return rc;
}

// The backward's statistics pass over a long-segment hop (no positional encoding): same pipeline,
// per query row (log2-sum-exp of the scaled scores, <G_t, O_t>) instead of the output.
int launch_hop_tc_long_stats(const Problem &pb, const HopDesc &hd, const void *xin, int xin_heads, const void *g,
                             void *stats) {
    if (pb.rope_base > 0.f || !stats || !g) return TA_ERR_INVALID_ARG;
    if (pb.D == 128) return launch_long_d<128>(pb, hd, xin, xin_heads, nullptr, stats, g);
    if (pb.D == 64) return launch_long_d<64>(pb, hd, xin, xin_heads, nullptr, stats, g);
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
