// Two consecutive hops of tensorized attention (Algorithm 1, loop iterations i and i+1) in ONE
// launch, ordered so that the second hop finds the first hop's output still in the L2 cache.
//
// Hops i and i+1 over adjacent dimensions are both closed over a "block": the contiguous run of
// n_i * s_i tokens that share every coordinate slower than dimension i.  Such a block is far
// larger than one SM's shared memory on long sequences (32 x 32 tokens x 256 B = 256 KB per head
// at 32k, 1 MB at 128k), so the two hops cannot be fused on chip; launched one after the other,
// every tile of the value tensor goes to HBM and comes back.  Here one persistent grid walks a
// single sequence of work items in which the hop-(i+1) tiles of a block follow the hop-i tiles of
// the same block by a fixed, short distance (`lag` blocks):
//
//     A(0) A(1) .. A(lag-1) | A(lag) B(0) | A(lag+1) B(1) | ... | B(units-lag) .. B(units-1)
//
// A(u) = the hop-i tiles of unit u, B(u) = its hop-(i+1) tiles; a unit is one block of one KV
// head (with the query heads of its group).  The bytes written and read between A(u) and B(u)
// stay far below the L2 capacity, so B(u) reads the value rows, and Q and K a second time, from
// L2, and overwrites lines that are still dirty there: HBM sees Q, K, the value tensor in and the
// value tensor out once for the two hops.
//
// Correctness does not depend on the cache: a B item waits on a counter in global memory that the
// A items of its unit (and head chunk) increment after their TMA stores have completed.  The CTAs
// claim the items of the sequence in order from a grid-wide counter (whichever CTA is ready takes
// the next one), so a B item only ever waits for items that were claimed earlier, by CTAs that are
// running, and A items wait for nobody: every wait ends, whatever the number of CTAs resident.
// The waits are bounded all the same.  The per-tile pipeline (TMA producer, MMA issuer, two softmax /
// epilogue warpgroups, store warp; S, P and O in tensor memory) is the one of the one-hop kernel.
#include <cuda_bf16.h>

#include <cstdlib>

#include "ta_internal.h"
#include "ta_ptx.cuh"

namespace ta {

namespace {

constexpr int kTileRows = 128;
constexpr int kThreads = 416;   // 13 warps: two producers, MMA issuer, two store warps, two softmax warpgroups
constexpr int kNK = 2;   // K ring (one slot per work item)
constexpr int kNQ = 2;   // Q ring (one slot per tile)

template <int D>
struct PairCfg {
    static constexpr int kHalves = D / 64;                     // 64-column (128-byte) slabs per row
    static constexpr uint32_t kSlabBytes = kTileRows * 128;
    static constexpr uint32_t kTileBytes = kHalves * kSlabBytes;
    static constexpr int kNX = D == 128 ? 3 : 6;               // value-tile ring
    static constexpr uint32_t kOffK = 0;
    static constexpr uint32_t kOffQ = kOffK + kNK * kTileBytes;
    static constexpr uint32_t kOffX = kOffQ + kNQ * kTileBytes;
    static constexpr uint32_t kOffBar = kOffX + kNX * kTileBytes;
    static constexpr int kNumBars = 2 * kNK + 2 * kNQ + 3 * kNX + 6 + 16 /*item ring*/;
    static constexpr uint32_t kSmemBytes = kOffBar + kNumBars * 8 + 16 + 16 * 4 + 1024 /*alignment slack*/;
    static constexpr uint32_t kTmemCols = 512;                 // S x 2 (P over S), O x 2
    static constexpr uint32_t kColS = 0, kColO = 256;
};

struct PhaseArgs {
    int n, rows, ci, co, window, xin_is_kv;
    int x_f16, out_f16;     // the value tensor read / written by this phase holds fp16, not bf16
    uint32_t tiles_inner;   // tiles along the hop's inner extent
    uint32_t items;         // work items of one unit in this phase
};

struct PairArgs {
    PhaseArgs ph[2];        // [0] = hop i ("A"), [1] = hop i+1 ("B")
    int causal, g, H, H_kv, gi, hsplit;
    int n_a;                // segment length of phase A: B's outer index = block * n_a + position along A
    uint32_t blocks;        // blocks per head (= outer extent of phase A)
    uint32_t units;         // B * H_kv * blocks
    uint32_t lag;           // units between A(u) and B(u) in the sequence (<= units)
    uint32_t total;         // positions of the sequence = units * (items A + items B)
    uint32_t flag_target;   // hop-A tiles per (unit, head chunk) = ph[0].tiles_inner * gi
    float scale_log2;
    unsigned int *flags;    // [units * hsplit] completion counters, zero when the kernel starts
    unsigned int *next_pos; // next unclaimed position of the sequence, zero when the kernel starts
};

struct PairItem {
    int phase, c_inner, c_outer, kv_head, q_head0;
    uint32_t flag;          // index of the (unit, head chunk) counter
};

// phase of sequence position p (one division)
__device__ __forceinline__ int phase_of(const PairArgs &a, uint32_t p) {
    const uint32_t ia = a.ph[0].items, ib = a.ph[1].items;
    const uint32_t pro = a.lag * ia;
    if (p < pro) return 0;
    const uint32_t q = p - pro, mid = (a.units - a.lag) * (ia + ib);
    if (q >= mid) return 1;
    return (q % (ia + ib)) < ia ? 0 : 1;
}

__device__ __forceinline__ PairItem decode_pos(const PairArgs &a, uint32_t p) {
    const uint32_t ia = a.ph[0].items, ib = a.ph[1].items;
    const uint32_t pro = a.lag * ia;
    uint32_t unit, idx;
    PairItem it;
    if (p < pro) {
        it.phase = 0; unit = p / ia; idx = p % ia;
    } else {
        const uint32_t q = p - pro, mid = (a.units - a.lag) * (ia + ib);
        if (q < mid) {
            const uint32_t step = q / (ia + ib), w = q % (ia + ib);
            if (w < ia) { it.phase = 0; unit = a.lag + step; idx = w; }
            else        { it.phase = 1; unit = step; idx = w - ia; }
        } else {
            const uint32_t r = q - mid;
            it.phase = 1; unit = a.units - a.lag + r / ib; idx = r % ib;
        }
    }
    const uint32_t hs = idx % (uint32_t)a.hsplit, rest = idx / (uint32_t)a.hsplit;
    it.kv_head = (int)(unit / a.blocks);                        // b * H_kv + kvh
    const uint32_t block = unit % a.blocks;
    if (it.phase == 0) {
        it.c_inner = (int)rest * a.ph[0].ci;
        it.c_outer = (int)block;
    } else {
        const uint32_t ti = rest % a.ph[1].tiles_inner, to = rest / a.ph[1].tiles_inner;
        it.c_inner = (int)ti * a.ph[1].ci;
        it.c_outer = (int)block * a.n_a + (int)to * a.ph[1].co;
    }
    it.q_head0 = (it.kv_head / a.H_kv) * a.H + (it.kv_head % a.H_kv) * a.g + (int)hs * a.gi;
    it.flag = unit * (uint32_t)a.hsplit + hs;
    return it;
}

__device__ __forceinline__ unsigned int ld_acquire_gpu(const unsigned int *p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_gpu_add(unsigned int *p, unsigned int v) {
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// orders accesses made through the async proxy (TMA) against those of the generic proxy
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

// Bounded wait until *flag >= target (another CTA's stores have completed); gives up when the
// CTA's abort flag is raised or the time limit passes (then raises it and records the error word).
__device__ __noinline__ bool wait_flag(const unsigned int *flag, unsigned int target, uint32_t where,
                                       volatile uint32_t *abort_flag) {
    if (ld_acquire_gpu(flag) >= target) return true;
    const unsigned long long t0 = globaltimer_ns();
    for (;;) {
        for (int i = 0; i < 16; ++i) {
            if (ld_acquire_gpu(flag) >= target) return true;
            __nanosleep(64);
        }
        if (*abort_flag) return false;
        if (globaltimer_ns() - t0 > kWaitLimitNs) {
            atomicCAS(&g_status_word, 0u, kErrWaitExpired | where);
            *abort_flag = 1u;
            return false;
        }
    }
}

// Row constants of a softmax thread for one phase (its tile row never changes, but the segment
// length -- hence the visible key columns -- differs between the two hops).
struct RowConst {
    int c_lo, c_hi, w_lo, w_hi, nchunks, row_valid, warp_valid;
};
__device__ __forceinline__ RowConst row_const(const PhaseArgs &p, int causal, int wq, int r) {
    RowConst c;
    const int seg = r / p.n;
    c.row_valid = r < p.rows;
    c.c_lo = seg * p.n;
    c.c_hi = causal ? r + 1 : c.c_lo + p.n;
    if (p.window > 0) {
        c.c_lo = max(c.c_lo, r - p.window + 1);
        if (!causal) c.c_hi = min(c.c_hi, r + p.window);
    }
    c.w_lo = ((wq * 32) / p.n) * p.n;
    c.w_hi = min(p.rows, ((wq * 32 + 31) / p.n + 1) * p.n);
    if (causal) c.w_hi = min(c.w_hi, wq * 32 + 32);
    c.warp_valid = wq * 32 < p.rows;
    c.nchunks = (p.rows + 31) >> 5;
    return c;
}

// ----------------------------------------------------------------------------- the kernel
constexpr int kRing = 16;                    // item ring: far more than the items a CTA has in flight
constexpr uint32_t kNoItem = 0xFFFFFFFFu;

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
hop_pair_kernel(const __grid_constant__ CUtensorMap map_qa, const __grid_constant__ CUtensorMap map_ka,
                const __grid_constant__ CUtensorMap map_xin_a, const __grid_constant__ CUtensorMap map_xout_a,
                const __grid_constant__ CUtensorMap map_qb, const __grid_constant__ CUtensorMap map_kb,
                const __grid_constant__ CUtensorMap map_xb, const PairArgs a) {
    using C = PairCfg<D>;
    constexpr int kHalves = C::kHalves;
    constexpr uint32_t kSlabBytes = C::kSlabBytes, kTileBytes = C::kTileBytes;
    constexpr int kNX = C::kNX;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t s0 = smem_u32(smem);
    const uint32_t sK = s0 + C::kOffK, sQ = s0 + C::kOffQ, sX = s0 + C::kOffX;
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
    auto s_full = [&](int i) { return bar0 + 8u * (uint32_t)(kB1 + i); };
    auto o_full = [&](int i) { return bar0 + 8u * (uint32_t)(kB1 + 2 + i); };
    auto p_full = [&](int i) { return bar0 + 8u * (uint32_t)(kB1 + 4 + i); };
    auto item_full = [&](int i) { return bar0 + 8u * (uint32_t)(kB1 + 6 + i); };
    uint32_t *tmem_slot = (uint32_t *)(smem + C::kOffBar + C::kNumBars * 8);
    volatile uint32_t *abort_flag = tmem_slot + 1;
    volatile uint32_t *item_pos = tmem_slot + 2;      // [kRing] sequence positions claimed by this CTA

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // ---- one-time setup
    for (uint32_t i = tid; i < C::kOffBar / 16; i += blockDim.x)
        ((uint4 *)smem)[i] = make_uint4(0, 0, 0, 0);   // rows a box never fills must stay finite
    if (tid == 0) {
        for (int i = 0; i < kNK; ++i) { mbar_init(k_full(i), 1); mbar_init(k_free(i), 1); }
        for (int i = 0; i < kNQ; ++i) { mbar_init(q_full(i), 1); mbar_init(q_free(i), 1); }
        for (int i = 0; i < kNX; ++i) { mbar_init(x_full(i), 1); mbar_init(x_free(i), 1); mbar_init(out_full(i), 4); }
        for (int i = 0; i < 2; ++i) { mbar_init(s_full(i), 1); mbar_init(o_full(i), 1); mbar_init(p_full(i), 4); }
        for (int i = 0; i < kRing; ++i) mbar_init(item_full(i), 1);
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
    if (tid == 0) griddep_launch_dependents();

    // The CTA's it-th item: the position the K/Q producer claimed for it from the grid-wide counter
    // (kNoItem when the sequence is exhausted or the CTA is shutting down).
    auto item_of = [&](uint32_t it, uint32_t where) -> uint32_t {
        if (!mbar_wait_abortable(item_full(it % kRing), (it / kRing) & 1, where, abort_flag)) return kNoItem;
        return item_pos[it % kRing];
    };

    if (warp == 0) {
        // =============================================================== claims items; TMA producer of K and Q
        // (inputs of the call: never wait for another CTA, so they run ahead of the value tiles)
        if (lane == 0) {
            uint32_t t = 0;
            uint32_t armed = 0, last_par = 0;
            auto arm = [&](uint32_t bit, uint32_t parity) {
                armed |= bit;
                last_par = parity ? (last_par | bit) : (last_par & ~bit);
            };
            bool ok = true;
            for (uint32_t it = 0; ok; ++it) {
                // Items are claimed in sequence order by whichever CTA is ready for one: a B item
                // only ever waits for items claimed before it, by CTAs that are running.
                const uint32_t pos = atomicAdd(a.next_pos, 1u);
                item_pos[it % kRing] = pos < a.total ? pos : kNoItem;
                mbar_arrive(item_full(it % kRing));
                if (pos >= a.total) break;
                const PairItem c = decode_pos(a, pos);
                const uint32_t slab_tx = (uint32_t)a.ph[c.phase].rows * 128u;
                const CUtensorMap *mk = c.phase ? &map_kb : &map_ka;
                const CUtensorMap *mq = c.phase ? &map_qb : &map_qa;
                const int ks = it & 1;
                const uint32_t kpar = (it >> 1) & 1;
                ok = mbar_wait_abortable(k_free(ks), kpar ^ 1, 0x10, abort_flag);
                if (!ok) break;
                mbar_expect_tx(k_full(ks), kHalves * slab_tx);
                arm(1u << ks, kpar);
#pragma unroll
                for (int h = 0; h < kHalves; ++h)
                    tma_load_5d(sK + ks * kTileBytes + h * kSlabBytes, mk, k_full(ks), 64 * h, 0, c.c_inner, c.c_outer, c.kv_head);
                for (int j = 0; j < a.gi; ++j, ++t) {
                    const int qs = t % kNQ;
                    const uint32_t qpar = (t / kNQ) & 1;
                    ok = mbar_wait_abortable(q_free(qs), qpar ^ 1, 0x11, abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(q_full(qs), kHalves * slab_tx);
                    arm(4u << qs, qpar);
#pragma unroll
                    for (int h = 0; h < kHalves; ++h)
                        tma_load_5d(sQ + qs * kTileBytes + h * kSlabBytes, mq, q_full(qs), 64 * h, 0, c.c_inner, c.c_outer, c.q_head0 + j);
                }
            }
            if (!ok) {
                // leaving early: let the copies already issued land (bounded) before the CTA's
                // shared memory is released
                const unsigned long long t0 = globaltimer_ns();
                for (int slot = 0; slot < 2 + kNQ; ++slot) {
                    if (!(armed & (1u << slot))) continue;
                    const uint32_t bar = slot < 2 ? k_full(slot) : q_full(slot - 2);
                    while (!mbar_try_wait(bar, (last_par >> slot) & 1u) && globaltimer_ns() - t0 < 10000000ull) {
                    }
                }
            }
        }
    } else if (warp == 3) {
        // =============================================================== TMA producer: value tiles
        if (lane == 0) {
            uint32_t t = 0;
            uint32_t armed = 0, last_par = 0;
            bool ok = true;
            bool prev_hop_done = false;   // the value tensor may be the previous kernel's output
            for (uint32_t it = 0; ok; ++it) {
                const uint32_t pos = item_of(it, 0x14);
                if (pos == kNoItem) break;
                const PairItem c = decode_pos(a, pos);
                const PhaseArgs &ph = a.ph[c.phase];
                const uint32_t slab_tx = (uint32_t)ph.rows * 128u;
                const CUtensorMap *mx = c.phase ? &map_xb : &map_xin_a;
                for (int j = 0; j < a.gi; ++j, ++t) {
                    const int x_head = ph.xin_is_kv ? c.kv_head : c.q_head0 + j;
                    const int xs = t % kNX;
                    const uint32_t xpar = (t / kNX) & 1;
                    ok = mbar_wait_abortable(x_free(xs), xpar ^ 1, 0x12, abort_flag);
                    if (!ok) break;
                    if (!prev_hop_done) {
                        griddep_wait();
                        prev_hop_done = true;
                    }
                    if (c.phase == 1 && j == 0) {
                        // the rows of this item's tiles are outputs of the A items of its unit
                        ok = wait_flag(a.flags + c.flag, a.flag_target, 0x13, abort_flag);
                        if (!ok) break;
                        fence_proxy_async_all();
                    }
                    mbar_expect_tx(x_full(xs), kHalves * slab_tx);
                    armed |= 1u << xs;
                    last_par = xpar ? (last_par | (1u << xs)) : (last_par & ~(1u << xs));
#pragma unroll
                    for (int h = 0; h < kHalves; ++h)
                        tma_load_5d(sX + xs * kTileBytes + h * kSlabBytes, mx, x_full(xs), 64 * h, 0, c.c_inner, c.c_outer, x_head);
                }
            }
            if (!ok) {
                const unsigned long long t0 = globaltimer_ns();
                for (int slot = 0; slot < kNX; ++slot) {
                    if (!(armed & (1u << slot))) continue;
                    while (!mbar_try_wait(x_full(slot), (last_par >> slot) & 1u) && globaltimer_ns() - t0 < 10000000ull) {
                    }
                }
            }
        }
    } else if (warp == 1) {
        // =============================================================== MMA issuer
        // S(t) = Q K^T one tile ahead of O(t-1) = P X.  K and Q come from a producer of their own
        // that runs ahead of the value tiles, so the wait for Q(t) is short and does not hold back O(t-1).
        if (lane == 0) {
            constexpr uint32_t idesc_s = instr_desc(128, 0);
            bool ok = true;
            auto issue_o = [&](uint32_t u, int kblocks, int f16) -> bool {
                const uint32_t idesc_o = f16 ? instr_desc_f16(D, 1) : instr_desc(D, 1);   // P has the type of X
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
            uint32_t t = 0;
            int kblocks = 0, kblocks_prev = 0;      // key blocks of 16 rows of tile t / tile t-1
            int f16 = 0, f16_prev = 0;              // type of their value tile
            for (uint32_t it = 0; ok; ++it) {
                const uint32_t pos = item_of(it, 0x26);
                if (pos == kNoItem) break;
                const PhaseArgs &ph = a.ph[phase_of(a, pos)];
                const int ks = it & 1;
                for (int j = 0; ok && j < a.gi; ++j, ++t) {
                    const int qs = t % kNQ;
                    kblocks_prev = kblocks;
                    f16_prev = f16;
                    kblocks = (ph.rows + 15) >> 4;
                    f16 = ph.x_f16;
                    if (j == 0) ok = mbar_wait_abortable(k_full(ks), (it >> 1) & 1, 0x23, abort_flag);
                    if (ok) ok = mbar_wait_abortable(q_full(qs), (t / kNQ) & 1, 0x24, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t q_base = sQ + qs * kTileBytes, k_base = sK + ks * kTileBytes;
#pragma unroll
                    for (int kb = 0; kb < D / 16; ++kb) {
                        const uint32_t off = (kb >> 2) * kSlabBytes + (kb & 3) * 32;
                        tc_mma_ss(tmem_base + C::kColS + (t & 1) * 128, smem_desc_sw128(q_base + off, 16, 1024),
                                  smem_desc_sw128(k_base + off, 16, 1024), idesc_s, kb > 0);
                    }
                    tc_commit(s_full(t & 1));
                    tc_commit(q_free(qs));
                    if (j == a.gi - 1) tc_commit(k_free(ks));
                    if (t > 0) ok = issue_o(t - 1, kblocks_prev, f16_prev);
                }
            }
            if (ok && t > 0) issue_o(t - 1, kblocks, f16);
        }
    } else if (warp == 2 || warp == 12) {
        // =============================================================== TMA store
        // Two store threads, one for the even and one for the odd tiles: a hop-A tile has to be
        // complete in global memory (not merely read out of shared memory) before its unit's
        // counter may say so, and that takes about a tile's time; the other thread stores the
        // next tile meanwhile.
        if (lane == 0) {
            const uint32_t mine = warp == 2 ? 0u : 1u;
            uint32_t t = 0;
            bool ok = true;
            for (uint32_t it = 0; ok; ++it) {
                const uint32_t pos = item_of(it, 0x31);
                if (pos == kNoItem) break;
                const PairItem c = decode_pos(a, pos);
                const CUtensorMap *mo = c.phase ? &map_xb : &map_xout_a;
                for (int j = 0; j < a.gi; ++j, ++t) {
                    if ((t & 1u) != mine) continue;
                    const int xs = t % kNX;
                    ok = mbar_wait_abortable(out_full(xs), (t / kNX) & 1, 0x30, abort_flag);
                    if (!ok) break;
#pragma unroll
                    for (int h = 0; h < kHalves; ++h)
                        tma_store_5d(mo, sX + xs * kTileBytes + h * kSlabBytes, 64 * h, 0, c.c_inner, c.c_outer, c.q_head0 + j);
                    tma_store_commit_and_wait_read();
                    mbar_arrive(x_free(xs));
                    if (c.phase == 0) {
                        tma_store_wait_all();
                        fence_proxy_async_all();
                        __threadfence();
                        red_release_gpu_add(a.flags + c.flag, 1u);
                    }
                }
            }
            tma_store_wait_all();
        }
    } else if (warp >= 4 && warp < 12) {
        // =============================================================== softmax + epilogue
        const int b = (warp - 4) >> 2;                  // tile parity this warpgroup serves
        const int wq = warp & 3;                        // TMEM lane quarter of this warp
        const uint32_t tmem_lane = tmem_base + ((uint32_t)(wq * 32) << 16);
        const int r = wq * 32 + lane;                   // this thread's tile row = TMEM lane
        const RowConst rc0 = row_const(a.ph[0], a.causal, wq, r), rc1 = row_const(a.ph[1], a.causal, wq, r);
        const uint32_t s_col = tmem_lane + C::kColS + b * 128, o_col = tmem_lane + C::kColO + b * 128;

        bool ok = true;
        uint32_t t = 0;
        for (uint32_t it = 0; ok; ++it) {
            uint32_t pos = item_of(it, 0x43);
            pos = __shfl_sync(0xffffffffu, pos, 0);     // one answer per warp (the aligned TMEM ops need it converged)
            if (pos == kNoItem) break;
            const int phase = phase_of(a, pos);
            const int c_lo = phase ? rc1.c_lo : rc0.c_lo, c_hi = phase ? rc1.c_hi : rc0.c_hi;
            const int w_lo = phase ? rc1.w_lo : rc0.w_lo, w_hi = phase ? rc1.w_hi : rc0.w_hi;
            const int nchunks = phase ? rc1.nchunks : rc0.nchunks;
            const bool row_valid = (phase ? rc1.row_valid : rc0.row_valid) != 0;
            const bool warp_valid = (phase ? rc1.warp_valid : rc0.warp_valid) != 0;
            const bool x_f16 = a.ph[phase].x_f16 != 0, out_f16 = a.ph[phase].out_f16 != 0;
            for (int j = 0; ok && j < a.gi; ++j, ++t) {
                if ((t & 1u) != (uint32_t)b) continue;
                const uint32_t par = (t >> 1) & 1;
                ok = mbar_wait_abortable(s_full(b), par, 0x40, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();

                float m = -INFINITY;
                uint32_t v[32];
#pragma unroll 1
                for (int c = 0; c < nchunks; ++c) {
                    if (!(warp_valid && 32 * c < w_hi && 32 * c + 32 > w_lo)) continue;   // warp-uniform
                    tmem_ld32(s_col + 32 * c, v);
#pragma unroll
                    for (int jj = 0; jj < 32; ++jj) {
                        const int col = 32 * c + jj;
                        if (col >= c_lo && col < c_hi) m = fmaxf(m, __uint_as_float(v[jj]));
                    }
                }
                const float m_scaled = row_valid ? m * a.scale_log2 : 0.f;
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
                            p0 = (row_valid && col >= c_lo && col < c_hi) ? p0 : 0.f;
                            p1 = (row_valid && col + 1 >= c_lo && col + 1 < c_hi) ? p1 : 0.f;
                            uint32_t w;
                            if (x_f16) {            // uniform: the weights take the type of the value tile
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
                const float inv = row_valid ? 1.f / sum : 1.f;
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(p_full(b));

                const int xs = t % kNX;
                ok = mbar_wait_abortable(o_full(b), par, 0x42, abort_flag);
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
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 3) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::kTmemCols) : "memory");
    }
}

template <int D>
int launch_pair_d(const Problem &pb, const HopDesc &ha, const HopDesc &hb, const void *xin, int xin_heads, void *out,
                  unsigned int *flags) {
    CUtensorMap mqa, mka, mxia, mxoa, mqb, mkb, mxb;
    int rc;
    if ((rc = make_hop_map(&mqa, pb.q, pb.B * pb.H, pb.N, D, ha, 2)) != TA_OK) return rc;
    if ((rc = make_hop_map(&mka, pb.k, pb.B * pb.H_kv, pb.N, D, ha, 2)) != TA_OK) return rc;
    if ((rc = make_hop_map(&mxia, xin, pb.B * xin_heads, pb.N, D, ha, 2)) != TA_OK) return rc;
    if ((rc = make_hop_map(&mxoa, out, pb.B * pb.H, pb.N, D, ha, 2)) != TA_OK) return rc;
    if ((rc = make_hop_map(&mqb, pb.q, pb.B * pb.H, pb.N, D, hb, 2)) != TA_OK) return rc;
    if ((rc = make_hop_map(&mkb, pb.k, pb.B * pb.H_kv, pb.N, D, hb, 2)) != TA_OK) return rc;
    if ((rc = make_hop_map(&mxb, out, pb.B * pb.H, pb.N, D, hb, 2)) != TA_OK) return rc;

    int dev = 0;
    const int num_sms = current_device_sms(&dev);
    PairArgs a;
    PairGeometry geo;
    if (!pair_geometry(pb.B, pb.H, pb.H_kv, ha, hb, num_sms, &geo)) return TA_ERR_INVALID_ARG;
    const HopDesc *hd[2] = {&ha, &hb};
    for (int p = 0; p < 2; ++p) {
        a.ph[p].n = hd[p]->n; a.ph[p].rows = hd[p]->rows; a.ph[p].ci = hd[p]->ci; a.ph[p].co = hd[p]->co;
        a.ph[p].window = pb.window[hd[p]->hop];
        a.ph[p].tiles_inner = (uint32_t)hd[p]->tiles_inner;
        a.ph[p].x_f16 = hd[p]->in_f16;
        a.ph[p].out_f16 = hd[p]->out_f16;
    }
    a.ph[0].xin_is_kv = xin_heads != pb.H ? 1 : 0;
    a.ph[1].xin_is_kv = 0;
    a.ph[0].items = geo.items_a;
    a.ph[1].items = geo.items_b;
    a.causal = pb.causal; a.g = pb.H / pb.H_kv; a.H = pb.H; a.H_kv = pb.H_kv;
    a.hsplit = geo.hsplit; a.gi = a.g / a.hsplit;
    a.n_a = ha.n;
    a.blocks = (uint32_t)ha.outer;
    a.units = geo.units;
    a.lag = geo.lag;
    a.total = geo.total;
    a.flag_target = (uint32_t)ha.tiles_inner * (uint32_t)a.gi;
    a.scale_log2 = pb.scale * 1.4426950408889634f;
    a.flags = flags;
    a.next_pos = flags + (size_t)geo.units * geo.hsplit;

    constexpr size_t smem = PairCfg<D>::kSmemBytes;
    auto kern = hop_pair_kernel<D>;
    static PerDeviceOnce configured;
    if (!configured.is_done(dev)) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return TA_ERR_CUDA;
        configured.mark(dev);
    }
    // Completion counters and the claim counter start at zero.  No CTA ever waits for an item that
    // is not already claimed by a running CTA, so the grid needs no co-residency guarantee.
    const unsigned grid = (unsigned)(a.total < (uint32_t)num_sms ? a.total : (uint32_t)num_sms);
    const cudaError_t e = cudaMemsetAsync(flags, 0, geo.flag_bytes, pb.stream);
    if (e != cudaSuccess) return cuda_fail(e);
    return launch_kernel(kern, grid, kThreads, smem, pb.stream, false, mqa, mka, mxia, mxoa, mqb, mkb, mxb, a);
}

}  // namespace

// Host geometry of a pair launch (also used by the planner to size the counters and to decide
// whether the pair is worth fusing).  Returns false when the two hops cannot run as a pair.
bool pair_geometry(int B, int H, int H_kv, const HopDesc &ha, const HopDesc &hb, int num_sms, PairGeometry *geo) {
    if (ha.path != PATH_TC || hb.path != PATH_TC || ha.nf > 1 || hb.nf > 1) return false;
    if (ha.stride != (long long)hb.n * hb.stride) return false;          // adjacent dimensions
    if (ha.co != 1) return false;                                        // an A tile lies inside one block
    if (ha.n % hb.co != 0) return false;                                 // a B tile lies inside one block
    const int g = H / H_kv;
    // An item covers the query heads of a whole GQA group on one tile position: they share the K
    // tile.  (One head per item keeps fewer bytes between A(u) and B(u) but loads K once per tile;
    // it measured slower at every lag.)
    geo->hsplit = 1;
    const long long tiles_b = (long long)(ha.n / hb.co) * hb.tiles_inner;
    const long long ia = ha.tiles_inner * geo->hsplit, ib = tiles_b * geo->hsplit;
    const long long units = (long long)B * H_kv * ha.outer;
    const long long total = units * (ia + ib);
    if (total >= (1ll << 31) || units * geo->hsplit >= (1ll << 30)) return false;
    geo->items_a = (uint32_t)ia;
    geo->items_b = (uint32_t)ib;
    geo->units = (uint32_t)units;
    geo->total = (uint32_t)total;
    // B(u) follows A(u) by about one and a half times as many items as there are CTAs.  The CTAs
    // hold that many consecutive items in flight (one being computed, the next ones prefetched), and
    // an A item's counter is incremented only when its last store has completed, so a B item that
    // follows its A items more closely finds them unfinished and stalls its CTA (measured at 32k
    // tokens: a third of this distance doubles the time).  A longer distance pushes the rows out of
    // the L2 before the B items read them.
    long long lag = (3ll * num_sms / 2 + (ia + ib) - 1) / (ia + ib);
    // Tuning knob for measurements: TA_PAIR_LAG_UNITS=<n> in the environment overrides the distance.
    if (const char *env = getenv("TA_PAIR_LAG_UNITS")) {
        const long long v = atoll(env);
        if (v >= 1) lag = v;
    }
    if (lag < 1) lag = 1;
    if (lag > units) lag = units;
    geo->lag = (uint32_t)lag;
    geo->flag_bytes = ((size_t)units * geo->hsplit + 1) * sizeof(unsigned int);   // counters + the claim counter
    // bytes touched between A(u) and B(u): Q, K, value in and out of `lag` units
    const double unit_bytes = (double)ha.n * ha.stride * 128.0 /*D<=128 bf16 upper bound*/ * 2.0 * (3.0 * g + 1.0);
    geo->window_bytes = unit_bytes * (double)lag;
    return true;
}

int launch_hop_tc_pair(const Problem &pb, const HopDesc &ha, const HopDesc &hb, const void *xin, int xin_heads,
                       void *out, void *flags) {
    if (!flags || pb.rope_base > 0.f || pb.seq_lens || pb.masks[ha.hop] || pb.masks[hb.hop]) return TA_ERR_INVALID_ARG;
    if (pb.D == 128) return launch_pair_d<128>(pb, ha, hb, xin, xin_heads, out, (unsigned int *)flags);
    if (pb.D == 64) return launch_pair_d<64>(pb, ha, hb, xin, xin_heads, out, (unsigned int *)flags);
    return TA_ERR_UNSUPPORTED;
}

int read_status_tc_pair(unsigned int *word) {
    if (cudaMemcpyFromSymbol(word, g_status_word, sizeof(*word)) != cudaSuccess) return TA_ERR_CUDA;
    if (*word != 0) {
        unsigned int z = 0;
        cudaMemcpyToSymbol(g_status_word, &z, sizeof(z));
    }
    return TA_OK;
}

}  // namespace ta
