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
// in fp32 registers (tcgen05.ld), un-normalised weights rounded to bf16 and written back to
// tensor memory over S (tcgen05.st)  ->  O = P X (tcgen05.mma with the A operand in TMEM, fp32
// accumulator in TMEM)  ->  O / rowsum -> bf16 -> shared memory (over the X tile)  ->  TMA store
// to the same strided rows.  Because a tile owns whole segments, the value tensor is updated
// in place.  Shared memory holds only operand tiles: K x 2, Q x 2, X x 3 (D = 128).
//
// The kernel is persistent (one CTA per SM) and warp-specialised, so that the HBM traffic of
// the next tiles overlaps the arithmetic of the current one:
//   warp 0      TMA producer: K tile of a work item (shared by the query heads of a GQA group
//               that the item covers), then Q and X tiles per head, into rings of shared memory
//   warp 1      MMA issuer: S(t) as soon as Q(t), K are in; O(t-1) once P(t-1), X(t-1) are
//   warps 4-7   softmax + epilogue of the even tiles   } each warp owns 32 TMEM lanes (rows);
//   warps 8-11  softmax + epilogue of the odd tiles    } S and O are double-buffered in TMEM
//   warp 2      TMA store of finished tiles; hands the X slot back to the producer
//   warps 12-19 (only with the tensorized positional encoding, Section 3.2) rotate the K and Q
//               tiles in place in shared memory by the rows' coordinate along the hop's
//               dimension (RoPE, feature c paired with c + D/2) before the MMA issuer sees them
// Every wait is an mbarrier wait with a time limit; when one expires the CTA raises a flag that
// ends all its roles, waits for its copies in flight, frees its TMEM and returns.
#include <cuda_bf16.h>

#include <cstring>
#include <mutex>

#include "ta_internal.h"
#include "ta_ptx.cuh"
#include "ta_rope.cuh"
#include "ta_mask.cuh"

namespace ta {

namespace {

constexpr int kTileRows = 128;
constexpr int kThreads = 384;        // without the positional encoding
constexpr int kThreadsRope = 640;    // + two warpgroups that rotate Q and K tiles
constexpr int kNK = 2;   // K ring (one slot per work item)
constexpr int kNQ = 2;   // Q ring (one slot per tile)

template <int D>
struct PipeCfg {
    static constexpr int kHalves = D / 64;                     // 64-column (128-byte) slabs per row
    static constexpr uint32_t kSlabBytes = kTileRows * 128;    // one [128 rows][64 cols] bf16 slab
    static constexpr uint32_t kTileBytes = kHalves * kSlabBytes;
    static constexpr int kNX = D == 128 ? 3 : 6;               // X ring (value tile in, output tile out)
    static constexpr uint32_t kOffK = 0;
    static constexpr uint32_t kOffQ = kOffK + kNK * kTileBytes;
    static constexpr uint32_t kOffX = kOffQ + kNQ * kTileBytes;
    static constexpr uint32_t kOffBar = kOffX + kNX * kTileBytes;
    static constexpr int kNumBars = 2 * kNK + 2 * kNQ + 3 * kNX + 2 + 2 + 2 + kNK + kNQ;
    static constexpr uint32_t kSmemBytes = kOffBar + kNumBars * 8 + 16 + 1024 /*alignment slack*/;
    // S: 2 x 128 fp32 columns (P, bf16, is written over the first 64 columns of its S), O: 2 x 128
    static constexpr uint32_t kTmemCols = 512;
    static constexpr uint32_t kColS = 0, kColO = 256;
};

struct TcArgs {
    int n, rows, ci, co, causal, g, H, H_kv, xin_is_kv;
    int gi, hsplit;            // query heads per work item, items per GQA group (gi * hsplit == g)
    long long tiles_inner, tiles_outer, total_items;
    int window;                // 0, or w: keys within w positions of the query along the hop's dimension
    float scale_log2;
    float rope_log2_base;      // log2 of the RoPE base (rotating variant only)
    int stride;                // token stride of the hop's dimension
    const int *lens;           // device, one valid length per batch entry, or nullptr (masked variant only)
    int x_f16, out_f16;        // the value tensor read / written holds fp16 (an intermediate of a hop chain), not bf16
    const uint32_t *dmask;     // masked variant, masks that differ per head: [H][n][4] words in device memory
                               // (causal flag and window folded in); nullptr: the mask is the kernel parameter
};

struct ItemCoord {
    int c_inner, c_outer, kv_head, q_head0;
};
// item -> (head chunk of the group, inner tile, outer tile, kv head, batch); the head chunks of
// a GQA group are adjacent so that their common K (and V) tile is hot in L2.
__device__ __forceinline__ ItemCoord decode_item(const TcArgs &a, long long item) {
    ItemCoord c;
    long long rest = item;
    const int hs = (int)(rest % a.hsplit); rest /= a.hsplit;
    c.c_inner = (int)(rest % a.tiles_inner) * a.ci; rest /= a.tiles_inner;
    c.c_outer = (int)(rest % a.tiles_outer) * a.co; rest /= a.tiles_outer;
    c.kv_head = (int)rest;                                      // b * H_kv + kvh
    c.q_head0 = (c.kv_head / a.H_kv) * a.H + (c.kv_head % a.H_kv) * a.g + hs * a.gi;
    return c;
}

// ----------------------------------------------------------------------------- the kernel
template <int D, bool kRope, bool kMask>
__global__ void __launch_bounds__(kRope ? kThreadsRope : kThreads, 1)
hop_pipe_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_xin, const __grid_constant__ CUtensorMap map_xout,
                const TcArgs a, const __grid_constant__ typename MaskArg<kMask>::type hop_mask) {
    using C = PipeCfg<D>;
    constexpr int kHalves = C::kHalves;
    constexpr uint32_t kSlabBytes = C::kSlabBytes, kTileBytes = C::kTileBytes;
    constexpr int kNX = C::kNX;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t s0 = smem_u32(smem);
    const uint32_t sK = s0 + C::kOffK, sQ = s0 + C::kOffQ, sX = s0 + C::kOffX;
    const uint32_t bar0 = s0 + C::kOffBar;
    // barrier indices
    auto k_full = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    auto k_free = [&](int i) { return bar0 + 8u * (uint32_t)(kNK + i); };
    auto q_full = [&](int i) { return bar0 + 8u * (uint32_t)(2 * kNK + i); };
    auto q_free = [&](int i) { return bar0 + 8u * (uint32_t)(2 * kNK + kNQ + i); };
    constexpr int kB0 = 2 * kNK + 2 * kNQ;
    auto x_full = [&](int i) { return bar0 + 8u * (uint32_t)(kB0 + i); };
    auto x_free = [&](int i) { return bar0 + 8u * (uint32_t)(kB0 + kNX + i); };
    auto out_full = [&](int i) { return bar0 + 8u * (uint32_t)(kB0 + 2 * kNX + i); };
    constexpr int kB1 = kB0 + 3 * kNX;
    auto s_full = [&](int i) { return bar0 + 8u * (uint32_t)(kB1 + i); };
    auto o_full = [&](int i) { return bar0 + 8u * (uint32_t)(kB1 + 2 + i); };
    auto p_full = [&](int i) { return bar0 + 8u * (uint32_t)(kB1 + 4 + i); };
    auto k_rot = [&](int i) { return bar0 + 8u * (uint32_t)(kB1 + 6 + i); };          // rotated K ready
    auto q_rot = [&](int i) { return bar0 + 8u * (uint32_t)(kB1 + 6 + kNK + i); };    // rotated Q ready
    uint32_t *tmem_slot = (uint32_t *)(smem + C::kOffBar + C::kNumBars * 8);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // ---- one-time setup
    for (uint32_t i = tid; i < C::kOffBar / 16; i += blockDim.x)
        ((uint4 *)smem)[i] = make_uint4(0, 0, 0, 0);   // rows a box never fills must stay finite
    if (tid == 0) {
        for (int i = 0; i < kNK; ++i) { mbar_init(k_full(i), 1); mbar_init(k_free(i), 1); }
        for (int i = 0; i < kNQ; ++i) { mbar_init(q_full(i), 1); mbar_init(q_free(i), 1); }
        for (int i = 0; i < kNX; ++i) { mbar_init(x_full(i), 1); mbar_init(x_free(i), 1); mbar_init(out_full(i), 4); }
        for (int i = 0; i < 2; ++i) { mbar_init(s_full(i), 1); mbar_init(o_full(i), 1); mbar_init(p_full(i), 4); }
        for (int i = 0; i < kNK; ++i) mbar_init(k_rot(i), 8);
        for (int i = 0; i < kNQ; ++i) mbar_init(q_rot(i), 8);
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
    // every CTA of this (persistent, fully resident) grid is running: the next hop's kernel may be
    // scheduled on SMs as they drain; it touches nothing this hop writes before its own wait
    if (tid == 0) griddep_launch_dependents();

    // tiles this CTA processes: its work items (round robin over the grid) x gi heads each
    const long long my_items = (a.total_items - blockIdx.x + gridDim.x - 1) / gridDim.x;
    const uint32_t T = (uint32_t)(my_items * a.gi);
    const uint32_t slab_tx = (uint32_t)a.rows * 128u;

    if (warp == 0) {
        // =============================================================== TMA producer
        if (lane == 0) {
            uint32_t t = 0, it = 0;
            // slots armed so far and the parity of the last phase armed on each (k 0-1, q 2-3, x 4-7)
            uint32_t armed = 0, last_par = 0;
            auto arm = [&](uint32_t bit, uint32_t parity) {
                armed |= bit;
                last_par = parity ? (last_par | bit) : (last_par & ~bit);
            };
            bool ok = true;
            bool prev_hop_done = false;   // Q and K are inputs of the call; the value tensor is the previous hop's output
            for (long long item = blockIdx.x; ok && item < a.total_items; item += gridDim.x, ++it) {
                const ItemCoord c = decode_item(a, item);
                const int ks = it & 1;
                const uint32_t kpar = (it >> 1) & 1;
                ok = mbar_wait_abortable(k_free(ks), kpar ^ 1, 0x10, abort_flag);
                if (!ok) break;
                mbar_expect_tx(k_full(ks), kHalves * slab_tx);
                arm(1u << ks, kpar);
#pragma unroll
                for (int h = 0; h < kHalves; ++h)
                    tma_load_5d(sK + ks * kTileBytes + h * kSlabBytes, &map_k, k_full(ks), 64 * h, 0, c.c_inner, c.c_outer, c.kv_head);
                for (int j = 0; j < a.gi; ++j, ++t) {
                    const int q_head = c.q_head0 + j;
                    const int x_head = a.xin_is_kv ? c.kv_head : q_head;
                    const int qs = t & 1;
                    const uint32_t qpar = (t >> 1) & 1;
                    ok = mbar_wait_abortable(q_free(qs), qpar ^ 1, 0x11, abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(q_full(qs), kHalves * slab_tx);
                    arm(4u << qs, qpar);
#pragma unroll
                    for (int h = 0; h < kHalves; ++h)
                        tma_load_5d(sQ + qs * kTileBytes + h * kSlabBytes, &map_q, q_full(qs), 64 * h, 0, c.c_inner, c.c_outer, q_head);
                    const int xs = t % kNX;
                    const uint32_t xpar = (t / kNX) & 1;
                    ok = mbar_wait_abortable(x_free(xs), xpar ^ 1, 0x12, abort_flag);
                    if (!ok) break;
                    if (!prev_hop_done) {
                        griddep_wait();
                        prev_hop_done = true;
                    }
                    mbar_expect_tx(x_full(xs), kHalves * slab_tx);
                    arm(16u << xs, xpar);
#pragma unroll
                    for (int h = 0; h < kHalves; ++h)
                        tma_load_5d(sX + xs * kTileBytes + h * kSlabBytes, &map_xin, x_full(xs), 64 * h, 0, c.c_inner, c.c_outer, x_head);
                }
            }
            if (!ok) {
                // leaving early: let the copies already issued land (bounded) before the CTA's
                // shared memory is released
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
        if (lane == 0) {
            constexpr uint32_t idesc_s = instr_desc(128, 0);
            const uint32_t idesc_o = a.x_f16 ? instr_desc_f16(D, 1) : instr_desc(D, 1);   // P has the type of X
            const int kblocks = (a.rows + 15) >> 4;
            bool ok = true;
            auto issue_o = [&](uint32_t u) -> bool {
                // O(u)[128 x D] = P[128 x rows] X[rows x D]; P from tensor memory (16 keys = 8
                // columns per instruction), X rows are keys (MN-major B operand)
                const int xs = u % kNX;
                if (!mbar_wait_abortable(p_full(u & 1), (u >> 1) & 1, 0x21, abort_flag)) return false;
                if (!mbar_wait_abortable(x_full(xs), (u / kNX) & 1, 0x22, abort_flag)) return false;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + C::kColO + (u & 1) * 128;
                const uint32_t p_tmem = tmem_base + C::kColS + (u & 1) * 128;
                const uint32_t x_base = sX + xs * kTileBytes;
                for (int kb = 0; kb < kblocks; ++kb)
                    tc_mma_ts(d_tmem, p_tmem + kb * 8, smem_desc_sw128(x_base + kb * 2048, kSlabBytes, 1024), idesc_o,
                              kb > 0);
                tc_commit(o_full(u & 1));
                return true;
            };
            uint32_t it = 0, j = 0;
            for (uint32_t t = 0; ok && t < T; ++t) {
                const int ks = it & 1, qs = t & 1;
                if (j == 0) ok = mbar_wait_abortable(kRope ? k_rot(ks) : k_full(ks), (it >> 1) & 1, 0x23, abort_flag);
                if (ok) ok = mbar_wait_abortable(kRope ? q_rot(qs) : q_full(qs), (t >> 1) & 1, 0x24, abort_flag);
                if (!ok) break;
                tc_fence_after();
                // S(t)[128 x 128] = Q[128 x D] K^T : D/16 instructions of K = 16.  Its buffer last
                // held P(t-2), the operand of O(t-2), which was issued earlier and executes first.
                const uint32_t q_base = sQ + qs * kTileBytes, k_base = sK + ks * kTileBytes;
#pragma unroll
                for (int kb = 0; kb < D / 16; ++kb) {
                    const uint32_t off = (kb >> 2) * kSlabBytes + (kb & 3) * 32;
                    tc_mma_ss(tmem_base + C::kColS + (t & 1) * 128, smem_desc_sw128(q_base + off, 16, 1024),
                              smem_desc_sw128(k_base + off, 16, 1024), idesc_s, kb > 0);
                }
                tc_commit(s_full(t & 1));
                tc_commit(q_free(qs));
                if (++j == (uint32_t)a.gi) {
                    tc_commit(k_free(ks));
                    j = 0;
                    ++it;
                }
                if (t > 0) ok = issue_o(t - 1);
            }
            if (ok && T > 0) issue_o(T - 1);
        }
    } else if (warp == 2) {
        // =============================================================== TMA store
        if (lane == 0) {
            uint32_t t = 0;
            bool ok = true;
            for (long long item = blockIdx.x; ok && item < a.total_items; item += gridDim.x) {
                const ItemCoord c = decode_item(a, item);
                for (int j = 0; j < a.gi; ++j, ++t) {
                    const int xs = t % kNX;
                    ok = mbar_wait_abortable(out_full(xs), (t / kNX) & 1, 0x30, abort_flag);
                    if (!ok) break;
#pragma unroll
                    for (int h = 0; h < kHalves; ++h)
                        tma_store_5d(&map_xout, sX + xs * kTileBytes + h * kSlabBytes, 64 * h, 0, c.c_inner, c.c_outer, c.q_head0 + j);
                    tma_store_commit_and_wait_read();
                    mbar_arrive(x_free(xs));
                }
            }
            tma_store_wait_all();
        }
    } else if (kRope && warp >= 12) {
        // =============================================================== RoPE on the K and Q tiles
        RopeRotator<D> rot;
        rot.init(tid - 12 * 32, a.n, a.rows, a.rope_log2_base);
        bool ok = true;
        uint32_t t = 0, it = 0;
        for (long long item = blockIdx.x; ok && item < a.total_items; item += gridDim.x, ++it) {
            const int ks = it & 1;
            ok = mbar_wait_abortable(k_full(ks), (it >> 1) & 1, 0x50, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            rot.rotate(sK + ks * kTileBytes);
            if (lane == 0) mbar_arrive(k_rot(ks));
            for (int j = 0; j < a.gi; ++j, ++t) {
                const int qs = t & 1;
                ok = mbar_wait_abortable(q_full(qs), (t >> 1) & 1, 0x51, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                rot.rotate(sQ + qs * kTileBytes);
                if (lane == 0) mbar_arrive(q_rot(qs));
            }
        }
    } else if (warp >= 4) {
        // =============================================================== softmax + epilogue
        const int b = (warp - 4) >> 2;                  // tile parity this warpgroup serves
        const int wq = warp & 3;                        // TMEM lane quarter of this warp
        const uint32_t tmem_lane = tmem_base + ((uint32_t)(wq * 32) << 16);
        const int r = wq * 32 + lane;                   // this thread's tile row = TMEM lane
        const int seg = r / a.n;
        const bool row_valid = r < a.rows;
        int c_lo = seg * a.n;
        int c_hi = a.causal ? r + 1 : c_lo + a.n;       // visible key columns [c_lo, c_hi)
        if (a.window > 0) {                             // sliding window along the hop's dimension
            c_lo = max(c_lo, r - a.window + 1);
            if (!a.causal) c_hi = min(c_hi, r + a.window);
        }
        // columns any row of this warp needs (warp-uniform)
        const int w_lo = ((wq * 32) / a.n) * a.n;
        int w_hi = min(a.rows, ((wq * 32 + 31) / a.n + 1) * a.n);
        if (a.causal) w_hi = min(w_hi, wq * 32 + 32);
        // explicit mask (already combined with the causal flag and the window): this row's bits
        // over the tile's key columns
        uint32_t mrow[4];
        tile_row_mask(hop_mask, row_valid ? r % a.n : 0, seg * a.n, mrow);
        if (kMask && !row_valid) mrow[0] = mrow[1] = mrow[2] = mrow[3] = 0u;
        const bool warp_valid = wq * 32 < a.rows;
        const int nchunks = (a.rows + 31) >> 5;         // 32-column chunks of P the MMA reads
        const uint32_t s_col = tmem_lane + C::kColS + b * 128, o_col = tmem_lane + C::kColO + b * 128;

        bool ok = true;
        for (uint32_t t = b; t < T; t += 2) {
            const uint32_t par = (t >> 1) & 1;
            // valid length: only the first `exist` positions of this row's segment are tokens
            // (flat index below the batch entry's length); a padding row sees nothing
            uint32_t mt[4] = {mrow[0], mrow[1], mrow[2], mrow[3]};
            if (kMask && a.dmask != nullptr) {
                // this tile's query head has a mask of its own
                const ItemCoord c = decode_item(a, (long long)blockIdx.x + (long long)(t / (uint32_t)a.gi) * gridDim.x);
                const int head = (c.q_head0 + (int)(t % (uint32_t)a.gi)) % a.H;
                tile_row_mask(a.dmask + (size_t)head * a.n * 4, row_valid ? r % a.n : 0, seg * a.n, mt);
                if (!row_valid) mt[0] = mt[1] = mt[2] = mt[3] = 0u;
            }
            if (kMask && a.lens != nullptr) {
                const ItemCoord c = decode_item(a, (long long)blockIdx.x + (long long)(t / (uint32_t)a.gi) * gridDim.x);
                const int len = __ldg(a.lens + c.kv_head / a.H_kv);
                const long long first = (long long)(c.c_outer + seg / a.ci) * a.n * a.stride + (c.c_inner + seg % a.ci);
                const long long left = ((long long)len - first + a.stride - 1) / a.stride;
                const int exist = len <= first ? 0 : (int)(left < a.n ? left : a.n);
                const int limit = (r % a.n) < exist ? seg * a.n + exist : 0;      // columns below it exist
#pragma unroll
                for (int cch = 0; cch < 4; ++cch) {
                    const int nb = limit - 32 * cch;
                    mt[cch] &= nb >= 32 ? 0xffffffffu : (nb <= 0 ? 0u : ((1u << nb) - 1u));
                }
            }
            ok = mbar_wait_abortable(s_full(b), par, 0x40, abort_flag);
            ok = __all_sync(0xffffffffu, ok);           // keep the warp converged for the aligned TMEM ops
            if (!ok) break;
            tc_fence_after();

            // ---- softmax over the row's visible columns; P (un-normalised, bf16) -> tensor memory,
            // two keys per 32-bit column, over the S columns already consumed
            float m = -INFINITY;
            uint32_t v[32];
#pragma unroll 1
            for (int c = 0; c < nchunks; ++c) {
                if (!(warp_valid && 32 * c < w_hi && 32 * c + 32 > w_lo)) continue;   // warp-uniform
                tmem_ld32(s_col + 32 * c, v);
#pragma unroll
                for (int jj = 0; jj < 32; ++jj) {
                    const int col = 32 * c + jj;
                    const float s = __uint_as_float(v[jj]);
                    const bool vis = kMask ? ((mask_chunk(mt, c) >> jj) & 1u) != 0 : (col >= c_lo && col < c_hi);
                    if (vis) m = fmaxf(m, s);
                }
            }
            // (a padding row of the masked variant has seen nothing: keep the arithmetic finite)
            const float m_scaled = (row_valid && !(kMask && m == -INFINITY)) ? m * a.scale_log2 : 0.f;
            float sum = 0.f;
#pragma unroll 1
            for (int c = 0; c < nchunks; ++c) {
                uint32_t pk[16];
                if (warp_valid && 32 * c < w_hi && 32 * c + 32 > w_lo) {
                    tmem_ld32(s_col + 32 * c, v);
#pragma unroll
                    for (int jj = 0; jj < 32; jj += 2) {
                        const int col = 32 * c + jj;
                        float p0 = fast_exp2(__uint_as_float(v[jj]) * a.scale_log2 - m_scaled);
                        float p1 = fast_exp2(__uint_as_float(v[jj + 1]) * a.scale_log2 - m_scaled);
                        if (kMask) {
                            const uint32_t bits = mask_chunk(mt, c);
                            p0 = ((bits >> jj) & 1u) ? p0 : 0.f;
                            p1 = ((bits >> (jj + 1)) & 1u) ? p1 : 0.f;
                        } else {
                            p0 = (row_valid && col >= c_lo && col < c_hi) ? p0 : 0.f;
                            p1 = (row_valid && col + 1 >= c_lo && col + 1 < c_hi) ? p1 : 0.f;
                        }
                        uint32_t w;
                        if (a.x_f16) {          // uniform: the weights take the type of the value tile
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
                tmem_st16(s_col + 16 * c, pk);
            }
            tmem_st_wait();
            const float inv = row_valid ? (kMask ? (sum > 0.f ? 1.f / sum : 0.f) : 1.f / sum) : 1.f;
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(p_full(b));

            // ---- epilogue: O / rowsum -> bf16 -> X slot (same swizzled box layout) -> store warp
            const int xs = t % kNX;
            ok = mbar_wait_abortable(o_full(b), par, 0x42, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            if (warp_valid) {
                const uint32_t x_row = sX + xs * kTileBytes + (uint32_t)r * 128u;
#pragma unroll 1
                for (int c = 0; c < D / 32; ++c) {
                    tmem_ld32(o_col + 32 * c, v);       // whole warp; rows beyond `rows` discard it
                    uint32_t pk[16];
#pragma unroll
                    for (int jj = 0; jj < 32; jj += 2)
                        pk[jj >> 1] = a.out_f16 ? pack_f16x2(__uint_as_float(v[jj]) * inv, __uint_as_float(v[jj + 1]) * inv)
                                                : pack_bf16x2(__uint_as_float(v[jj]) * inv, __uint_as_float(v[jj + 1]) * inv);
                    const uint32_t slab = x_row + (uint32_t)(c >> 1) * kSlabBytes;
                    if (row_valid) {
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

typedef CUresult (*CtxGetCurrentFn)(CUcontext *);
bool thread_has_context() {
    static CtxGetCurrentFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuCtxGetCurrent", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (CtxGetCurrentFn)p;
    });
    CUcontext ctx = nullptr;
    return fn && fn(&ctx) == CUDA_SUCCESS && ctx != nullptr;
}

}  // namespace

// Rank-5 map of one tensor [heads][N][D] seen through hop `hd`: dims (D, t, inner, outer, head),
// box (128 bytes of D, n, ci, co, 1), 128-byte swizzle.  elem = 2 (bf16) or 4 (fp32).
int make_hop_map(CUtensorMap *map, const void *base, int heads_total, int N, int D, const HopDesc &hd, int elem) {
    return make_view_map(map, base, heads_total, N, D, hd, elem, hd.n, hd.ci, hd.co);
}

int make_view_map(CUtensorMap *map, const void *base, int heads_total, int N, int D, const HopDesc &hd, int elem,
                  int box_t, int box_inner, int box_outer) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) {
        tl_last_cuda_error = -1000;
        return TA_ERR_CUDA;
    }
    const cuuint64_t e = (cuuint64_t)elem;
    cuuint64_t gdim[5] = {(cuuint64_t)D, (cuuint64_t)hd.n, (cuuint64_t)hd.stride, (cuuint64_t)hd.outer,
                          (cuuint64_t)heads_total};
    cuuint64_t gstr[4] = {(cuuint64_t)hd.stride * D * e, (cuuint64_t)D * e, (cuuint64_t)hd.n * hd.stride * D * e,
                          (cuuint64_t)N * D * e};
    cuuint32_t box[5] = {(cuuint32_t)(128 / elem), (cuuint32_t)box_t, (cuuint32_t)box_inner, (cuuint32_t)box_outer, 1u};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    // The encoder is a driver call and needs a context current on this host thread; a thread whose
    // first CUDA activity is this library (its caller's streams and buffers may all come from
    // pools filled by other threads) has none until a runtime call binds the primary context.
    // (Asked of the driver each time rather than remembered: the bind itself is not allowed
    // inside a stream capture, and a capturing thread always has a context.)
    if (!thread_has_context()) cudaFree(nullptr);
    CUresult r = enc(map, elem == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 5,
                     const_cast<void *>(base), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r == CUDA_ERROR_INVALID_CONTEXT) {   // e.g. the thread's context was popped since: bind and retry once
        cudaFree(nullptr);
        r = enc(map, elem == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 5,
                const_cast<void *>(base), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
    if (r != CUDA_SUCCESS) {
        tl_last_cuda_error = -1000 - (int)r;   // a driver (CUresult) code, not a runtime one
        return TA_ERR_CUDA;
    }
    return TA_OK;
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

    int dev = 0;
    const int num_sms = current_device_sms(&dev);
    TcArgs a;
    a.n = hd.n; a.rows = hd.rows; a.ci = hd.ci; a.co = hd.co; a.causal = pb.causal;
    a.g = pb.H / pb.H_kv; a.H = pb.H; a.H_kv = pb.H_kv; a.xin_is_kv = xin_heads != pb.H ? 1 : 0;
    a.tiles_inner = hd.tiles_inner; a.tiles_outer = hd.tiles_outer;
    // A work item covers gi query heads of one GQA group on one tile position (they share the
    // K tile); groups are split across items only when there are too few items to fill the GPU.
    const long long positions = (long long)pb.B * pb.H_kv * hd.tiles_inner * hd.tiles_outer;
    a.hsplit = 1;
    for (int d = 2; d <= a.g && positions * a.hsplit < 2ll * num_sms; ++d)
        if (a.g % d == 0) a.hsplit = d;
    a.gi = a.g / a.hsplit;
    a.total_items = positions * a.hsplit;
    a.window = pb.window[hd.hop];
    a.scale_log2 = pb.scale * 1.4426950408889634f;
    a.rope_log2_base = pb.rope_base > 0.f ? log2f(pb.rope_base) : 0.f;
    a.stride = (int)hd.stride;
    a.lens = pb.seq_lens;
    a.x_f16 = hd.in_f16;
    a.out_f16 = hd.out_f16;
    a.dmask = (pb.masks[hd.hop] && pb.masks_per_head) ? pb.dmask[hd.hop] : nullptr;
    if (pb.masks[hd.hop] && pb.masks_per_head && !a.dmask) return TA_ERR_INVALID_ARG;

    constexpr size_t smem = PipeCfg<D>::kSmemBytes;
    const unsigned grid = (unsigned)(a.total_items < num_sms ? a.total_items : num_sms);
    static PerDeviceOnce configured;
    if (!configured.is_done(dev)) {
        const cudaFuncAttribute attr = cudaFuncAttributeMaxDynamicSharedMemorySize;
        if (cudaFuncSetAttribute(hop_pipe_kernel<D, false, false>, attr, (int)smem) != cudaSuccess ||
            cudaFuncSetAttribute(hop_pipe_kernel<D, true, false>, attr, (int)smem) != cudaSuccess ||
            cudaFuncSetAttribute(hop_pipe_kernel<D, false, true>, attr, (int)smem) != cudaSuccess ||
            cudaFuncSetAttribute(hop_pipe_kernel<D, true, true>, attr, (int)smem) != cudaSuccess)
            return TA_ERR_CUDA;
        configured.mark(dev);
    }
    // A hop that follows another hop kernel of the same call is launched with programmatic stream
    // serialization: its CTAs may start on SMs the previous hop has left and fetch their first K and
    // Q tiles (inputs of the call) while that hop drains; they wait for it before touching the
    // value tensor.  The saving is a fixed few microseconds per hop boundary (3.5 % of a 0.4 ms
    // call), so it is used for short hops only: on hops of more than 32 work items per CTA it
    // measured within noise, and slightly negative on the 128k-token shape.
    const bool overlap = pb.pdl && a.total_items <= 32ll * num_sms;
    if (pb.masks[hd.hop] || pb.seq_lens) {
        HopMask hm;                                  // explicit mask ^ causal flag ^ window, by value
        if (a.dmask) {
            // per-head masks live in device memory; the parameter only says "everything visible"
            // (the kernel replaces it per tile)
            memset(&hm, 0, sizeof(hm));
        } else {
            const int rc = build_hop_mask(pb, hd, &hm);
            if (rc != TA_OK) return rc;
        }
        if (pb.rope_base > 0.f)
            return launch_kernel(hop_pipe_kernel<D, true, true>, grid, kThreadsRope, smem, pb.stream, overlap, mq, mk, mxi,
                                 mxo, a, hm);
        return launch_kernel(hop_pipe_kernel<D, false, true>, grid, kThreads, smem, pb.stream, overlap, mq, mk, mxi, mxo, a,
                             hm);
    }
    if (pb.rope_base > 0.f)
        return launch_kernel(hop_pipe_kernel<D, true, false>, grid, kThreadsRope, smem, pb.stream, overlap, mq, mk, mxi, mxo,
                             a, NoMask{});
    return launch_kernel(hop_pipe_kernel<D, false, false>, grid, kThreads, smem, pb.stream, overlap, mq, mk, mxi, mxo, a,
                         NoMask{});
}

}  // namespace

int launch_hop_tc(const Problem &pb, const HopDesc &hd, const void *xin, int xin_heads, void *xout) {
    if (hd.nf > 1) return launch_hop_tc_fused(pb, hd, xin, xin_heads, xout);
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
