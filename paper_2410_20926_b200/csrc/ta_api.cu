// C ABI of libta_b200.so: argument validation, the host-side hop planner and the launch loop
// of Algorithm 1 (one hop per tensor dimension, first dimension first).
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <vector>

#include "ta_internal.h"

namespace ta {

static std::atomic<unsigned long long> g_launches{0};
thread_local int tl_last_cuda_error = 0;
void count_launch(unsigned n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

int validate_shape(int B, int H, int H_kv, int N, int D, const int *dims, int ndims, int dtype) {
    if (!dims || B <= 0 || H <= 0 || H_kv <= 0 || N <= 0 || D <= 0) return TA_ERR_INVALID_ARG;
    if (ndims < 1 || ndims > TA_MAX_DIMS) return TA_ERR_INVALID_ARG;
    long long prod = 1;
    for (int i = 0; i < ndims; ++i) {
        if (dims[i] < 1) return TA_ERR_INVALID_ARG;
        prod *= dims[i];
        if (prod > (1ll << 40)) return TA_ERR_SHAPE;
    }
    if (prod != N || H % H_kv != 0) return TA_ERR_SHAPE;
    if (dtype != TA_DTYPE_BF16 && dtype != TA_DTYPE_F32) return TA_ERR_UNSUPPORTED;
    if (D > TA_MAX_HEAD_DIM) return TA_ERR_UNSUPPORTED;
    return TA_OK;
}

// A pair launch pays only while what is touched between the two hops of a unit stays in L2.
constexpr double kPairWindowLimitBytes = 160.0 * 1024 * 1024;

static bool tc_eligible(int D, int dtype, unsigned flags) {
    return dtype == TA_DTYPE_BF16 && (D == 64 || D == 128) && !(flags & TA_FLAG_NO_TENSOR_CORE);
}

// Packs whole segments into a 128-row tile: ci consecutive `inner` positions, then co
// consecutive `outer` positions (co only when the inner extent is exhausted, and only if it
// divides the outer extent so that a tile never straddles two heads).
static void tile_packing(HopDesc &h) {
    const int cap = 128 / h.n;                       // segments per tile
    h.ci = (int)(h.stride < cap ? h.stride : cap);
    int co = cap / h.ci;
    if (h.ci < h.stride) co = 1;
    if (co > h.outer) co = (int)h.outer;
    while (co > 1 && h.outer % co != 0) --co;
    h.co = co;
    h.rows = h.ci * h.co * h.n;
    h.tiles_inner = (h.stride + h.ci - 1) / h.ci;
    h.tiles_outer = (h.outer + h.co - 1) / h.co;
}

int build_plan(int B, int H, int H_kv, int N, int D, const int *dims, int ndims, int dtype,
               unsigned flags, int hop_begin, int hop_end, Plan *plan) {
    int rc = validate_shape(B, H, H_kv, N, D, dims, ndims, dtype);
    if (rc != TA_OK) return rc;
    if (flags & ~(unsigned)(TA_FLAG_NO_TENSOR_CORE | TA_FLAG_NO_HOP_FUSION | TA_FLAG_SAVE_HOPS | TA_FLAG_NO_HOP_OVERLAP |
                            TA_FLAG_PAIR_HOPS | TA_FLAG_BF16_INTERMEDIATES | kPlanAllowPairs))
        return TA_ERR_UNSUPPORTED;
    if (hop_begin == 0 && hop_end == 0) hop_end = ndims;
    if (hop_begin < 0 || hop_end > ndims || hop_begin > hop_end) return TA_ERR_INVALID_ARG;
    memset(plan, 0, sizeof(*plan));
    for (int i = hop_begin; i < hop_end; ++i) {
        if (dims[i] == 1) continue;  // softmax over one element: identity hop
        HopDesc &h = plan->hops[plan->nhops++];
        h.hop = i;
        h.n = dims[i];
        h.stride = 1;
        for (int l = i + 1; l < ndims; ++l) h.stride *= dims[l];
        h.outer = (long long)N / ((long long)h.n * h.stride);
        h.path = PATH_SIMT;
        if (tc_eligible(D, dtype, flags)) {
            if (h.n <= 128) h.path = PATH_TC;
            else h.path = PATH_TC_LONG;
        }
        if (h.path == PATH_TC) tile_packing(h);
    }
    // Hop fusion: the longest run of trailing dimensions i0..ndims-1 whose product is at most one
    // 128-row tile (all of them in the requested hop range and on the tensor-core path) becomes one
    // pass over contiguous blocks -- Q, K and the value tensor are read once for all those hops.
    if (!(flags & (TA_FLAG_NO_HOP_FUSION | TA_FLAG_SAVE_HOPS)) && hop_end == ndims && plan->nhops >= 2) {
        long long block = 1;
        int first = plan->nhops;                     // index in plan->hops of the first fused hop
        for (int j = plan->nhops - 1; j >= 0; --j) {
            const HopDesc &h = plan->hops[j];
            if (h.path != PATH_TC || (long long)h.n * h.stride > 128) break;
            block = (long long)h.n * h.stride;       // = prod(dims[h.hop ..])
            first = j;
        }
        const int nf = plan->nhops - first;
        if (nf >= 2) {
            HopDesc f = plan->hops[first];
            f.nf = nf;
            for (int j = 0; j < nf; ++j) {
                f.sub_n[j] = plan->hops[first + j].n;
                f.sub_stride[j] = (int)plan->hops[first + j].stride;
                f.sub_hop[j] = plan->hops[first + j].hop;
            }
            f.n = (int)block;
            f.stride = 1;
            f.outer = (long long)N / block;
            tile_packing(f);
            // Measured on B200: at D = 128 the fused pass is faster than the passes it replaces
            // (HBM-bound either way, fewer bytes); at D = 64 a tile carries half the bytes, the
            // fused pass is bound by its softmax / epilogue chain instead and only pays when the
            // problem is so small that the launches themselves dominate.
            const long long tiles = (long long)B * H * f.tiles_inner * f.tiles_outer;
            if (D == 128 || tiles <= 2ll * current_device_sms(nullptr)) {
                plan->hops[first] = f;
                plan->nhops = first + 1;
            }
        }
    }
    const size_t tensor_bytes = (size_t)B * H * N * D * elem_bytes(dtype);
    const int nh = plan->nhops;
    if (nh == 0) return TA_OK;
    const int first_src = hop_begin > 0 ? BUF_OUT : BUF_V;
    if (flags & TA_FLAG_SAVE_HOPS) {
        // X_{j+1} of hop j goes to save slot j (buffer id 3 + j); the last hop writes `out`.
        for (int j = 0; j < nh; ++j) {
            plan->hops[j].src = j == 0 ? first_src : 3 + (j - 1);
            plan->hops[j].dst = j == nh - 1 ? BUF_OUT : 3 + j;
        }
        plan->save_bytes = (size_t)(nh - 1) * tensor_bytes;
        if (plan->hops[0].src == plan->hops[0].dst && plan->hops[0].path != PATH_TC) {
            // one hop with hop_begin > 0 on a kernel that cannot update in place: the caller's
            // `out` is first copied to scratch
            plan->hops[0].src = BUF_SCRATCH;
            plan->need_scratch = true;
            plan->scratch_bytes = tensor_bytes;
        }
        return TA_OK;
    }
    // The tensor-core kernel updates in place; the generic kernel needs src != dst.  Assign
    // buffers from the last hop (which must land in `out`) backwards.
    int dst = BUF_OUT;
    for (int j = nh - 1; j >= 0; --j) {
        HopDesc &h = plan->hops[j];
        h.dst = dst;
        if (j == 0) {
            h.src = first_src;
        } else {
            h.src = h.path == PATH_TC ? dst : (dst == BUF_OUT ? BUF_SCRATCH : BUF_OUT);
            dst = h.src;
        }
    }
    if (plan->hops[0].path != PATH_TC && plan->hops[0].src == plan->hops[0].dst) {
        // only reachable with hop_begin > 0: the caller's `out` is first copied to scratch
        plan->hops[0].src = BUF_SCRATCH;
    }
    for (int j = 0; j < nh; ++j)
        if (plan->hops[j].src == BUF_SCRATCH || plan->hops[j].dst == BUF_SCRATCH) plan->need_scratch = true;
    if (plan->need_scratch) plan->scratch_bytes = tensor_bytes;
    // The value tensor between two tensor-core hops (the second may be a fused pass) is stored as fp16.
    if (!(flags & TA_FLAG_BF16_INTERMEDIATES)) {
        for (int j = 0; j + 1 < nh; ++j) {
            HopDesc &ha = plan->hops[j], &hb = plan->hops[j + 1];
            if (ha.path == PATH_TC && hb.path == PATH_TC && ha.nf <= 1 && ha.dst == hb.src) {
                ha.out_f16 = 1;
                hb.in_f16 = 1;
            }
        }
    }
    // Pairs of adjacent tensor-core hops whose common block exceeds one SM's shared memory: one
    // L2-ordered launch per pair (ta_tc_pair.cu), chosen from the last hop backwards (the later
    // hops move the most bytes: value tensor in and out with all H heads).
    if ((flags & (kPlanAllowPairs | TA_FLAG_PAIR_HOPS)) && !(flags & (TA_FLAG_NO_HOP_FUSION | TA_FLAG_SAVE_HOPS))) {
        const int sms = current_device_sms(nullptr);
        for (int j = nh - 2; j >= 0; --j) {
            HopDesc &ha = plan->hops[j];
            const HopDesc &hb = plan->hops[j + 1];
            PairGeometry geo;
            if (hb.pair || hb.src != BUF_OUT || hb.dst != BUF_OUT || ha.dst != BUF_OUT ||
                (ha.src != BUF_OUT && ha.src != BUF_V))
                continue;
            if (!pair_geometry(B, H, H_kv, ha, hb, sms, &geo)) continue;
            if (geo.window_bytes > kPairWindowLimitBytes) continue;
            ha.pair = 1;
            if (geo.flag_bytes > plan->flag_bytes) plan->flag_bytes = (geo.flag_bytes + 255) & ~(size_t)255;
            --j;   // the hop before a pair's first hop may not be the second hop of another pair
        }
    }
    return TA_OK;
}

int current_device_sms(int *dev) {
    static std::atomic<int> cache[64];
    int d = 0;
    if (cudaGetDevice(&d) != cudaSuccess) d = 0;
    if (dev) *dev = d;
    int n = (d >= 0 && d < 64) ? cache[d].load(std::memory_order_relaxed) : 0;
    if (n > 0) return n;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, d) != cudaSuccess || n <= 0) n = 148;
    if (d >= 0 && d < 64) cache[d].store(n, std::memory_order_relaxed);
    return n;
}

int build_hop_mask(const Problem &pb, const HopDesc &hd, HopMask *hm) {
    const int n = hd.n;
    if (n > 128) return TA_ERR_UNSUPPORTED;
    const unsigned char *m = pb.masks[hd.hop];
    const int w = pb.window[hd.hop];
    memset(hm, 0, sizeof(*hm));
    for (int t = 0; t < n; ++t) {
        bool any = false;
        for (int u = 0; u < n; ++u) {
            if (pb.causal && u > t) continue;
            if (w > 0 && (t - u >= w || u - t >= w)) continue;
            if (m && !m[(size_t)t * n + u]) continue;
            hm->bits[t][u >> 5] |= 1u << (u & 31);
            any = true;
        }
        if (!any) return TA_ERR_INVALID_ARG;
    }
    return TA_OK;
}

int upload_long_masks(Problem *pb, const Plan &plan, void **pooled) {
    *pooled = nullptr;
    const int mh = pb->masks_per_head ? pb->H : 1;              // matrices per masked dimension
    auto on_device = [&](const HopDesc &h) { return h.nf <= 1 && pb->masks[h.hop] && (h.n > 128 || pb->masks_per_head); };
    size_t total_words = 0;
    for (int j = 0; j < plan.nhops; ++j) {
        const HopDesc &h = plan.hops[j];
        if (!on_device(h)) continue;
        const size_t words = (size_t)((h.n + 127) / 128) * 4, qblocks = (size_t)(h.n + 127) / 128;
        total_words += (size_t)mh * ((size_t)h.n * words + 2 * qblocks);
        total_words = (total_words + 3) & ~(size_t)3;
    }
    if (total_words == 0) return TA_OK;
    std::vector<uint32_t> host(total_words, 0u);
    struct Placed { int hop; size_t off; int words; };
    std::vector<Placed> placed;
    size_t off = 0;
    for (int j = 0; j < plan.nhops; ++j) {
        const HopDesc &h = plan.hops[j];
        if (!on_device(h)) continue;
        const int n = h.n, words = ((n + 127) / 128) * 4, qblocks = (n + 127) / 128;
        const int w = pb->window[h.hop];
        uint32_t *bits0 = host.data() + off;
        int *ranges0 = (int *)(bits0 + (size_t)mh * n * words);
        for (int hh = 0; hh < mh; ++hh) {
            const unsigned char *m = pb->masks[h.hop] + (size_t)hh * n * n;
            uint32_t *bits = bits0 + (size_t)hh * n * words;
            int *ranges = ranges0 + (size_t)hh * 2 * qblocks;
            for (int qb = 0; qb < qblocks; ++qb) { ranges[2 * qb] = qblocks; ranges[2 * qb + 1] = 0; }
            for (int t = 0; t < n; ++t) {
                bool any = false;
                for (int u = 0; u < n; ++u) {
                    if (pb->causal && u > t) break;
                    if (w > 0 && (t - u >= w || u - t >= w)) continue;
                    if (!m[(size_t)t * n + u]) continue;
                    bits[(size_t)t * words + (u >> 5)] |= 1u << (u & 31);
                    any = true;
                    int &lo = ranges[2 * (t / 128)], &hi = ranges[2 * (t / 128) + 1];
                    if (u / 128 < lo) lo = u / 128;
                    if (u / 128 + 1 > hi) hi = u / 128 + 1;
                }
                if (!any) return TA_ERR_INVALID_ARG;
            }
        }
        placed.push_back({h.hop, off, words});
        off += (size_t)mh * ((size_t)n * words + 2 * (size_t)qblocks);
        off = (off + 3) & ~(size_t)3;
    }
    void *dev = nullptr;
    int rc = pool_alloc(total_words * sizeof(uint32_t), pb->stream, &dev);
    if (rc != TA_OK) return rc;
    *pooled = dev;
    // (pageable source: the runtime stages it before the call returns, so `host` may go away)
    const cudaError_t e = cudaMemcpyAsync(dev, host.data(), total_words * sizeof(uint32_t), cudaMemcpyHostToDevice, pb->stream);
    if (e != cudaSuccess) return cuda_fail(e);
    for (const Placed &pl : placed) {
        pb->dmask[pl.hop] = (const uint32_t *)dev + pl.off;
        pb->dmask_words[pl.hop] = pl.words;
    }
    return TA_OK;
}

int take_masks(Problem *pb, const Plan &plan, const int *window, const unsigned char *const *hop_masks, int ndims) {
    for (int i = 0; i < TA_MAX_DIMS; ++i) {
        pb->dmask[i] = nullptr;
        pb->dmask_words[i] = 0;
        pb->window[i] = (window && i < ndims) ? window[i] : 0;
        pb->masks[i] = (hop_masks && i < ndims) ? hop_masks[i] : nullptr;
        if (pb->window[i] < 0) return TA_ERR_INVALID_ARG;
    }
    // every masked hop is checked before anything is launched
    for (int j = 0; j < plan.nhops; ++j) {
        const HopDesc &h = plan.hops[j];
        if (h.nf > 1 || !pb->masks[h.hop] || h.n > 128 || pb->masks_per_head) continue;   // those: upload_long_masks
        HopMask hm;
        const int rc = build_hop_mask(*pb, h, &hm);
        if (rc != TA_OK) return rc;
    }
    return TA_OK;
}

// ---------------------------------------------------------------------------------------
// Device memory the library takes by itself.
//  * Scratch of a call that was given no workspace (second value buffer, rotated Q / K copies,
//    completion counters): stream-ordered allocations from a memory pool the library creates per
//    device.  An allocation belongs to one call on one stream and goes back in stream order, so
//    calls on different streams or host threads never share it, nothing is freed while a kernel
//    may still use it, and there is no device-wide synchronisation.
//  * Staging memory of ta_forward_host: one grow-only arena (calls are serialised by a lock).
// ---------------------------------------------------------------------------------------
static std::mutex g_pool_mutex;
static cudaMemPool_t g_pools[64] = {};

int pool_alloc(size_t bytes, cudaStream_t stream, void **ptr) {
    *ptr = nullptr;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= 64) return TA_ERR_TOO_LARGE;
    cudaMemPool_t pool;
    {
        std::lock_guard<std::mutex> lock(g_pool_mutex);
        if (!g_pools[dev]) {
            cudaMemPoolProps props = {};
            props.allocType = cudaMemAllocationTypePinned;
            props.handleTypes = cudaMemHandleTypeNone;
            props.location.type = cudaMemLocationTypeDevice;
            props.location.id = dev;
            if ((e = cudaMemPoolCreate(&g_pools[dev], &props)) != cudaSuccess) {
                g_pools[dev] = nullptr;
                return cuda_fail(e);
            }
            // keep freed memory in the pool (the next call takes it back without a driver round trip)
            unsigned long long keep = ~0ull;
            cudaMemPoolSetAttribute(g_pools[dev], cudaMemPoolAttrReleaseThreshold, &keep);
        }
        pool = g_pools[dev];
    }
    if ((e = cudaMallocFromPoolAsync(ptr, bytes ? bytes : 256, pool, stream)) != cudaSuccess) {
        *ptr = nullptr;
        return cuda_fail(e);
    }
    return TA_OK;
}

void pool_free(void *ptr, cudaStream_t stream) {
    if (ptr) cudaFreeAsync(ptr, stream);
}

struct Arena {
    void *ptr = nullptr;
    size_t bytes = 0;
    int device = -1;
    int reserve(size_t need) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return TA_ERR_CUDA;
        if (ptr && dev == device && bytes >= need) return TA_OK;
        if (ptr) {
            cudaDeviceSynchronize();
            cudaFree(ptr);
            ptr = nullptr;
            bytes = 0;
        }
        if (cudaMalloc(&ptr, need) != cudaSuccess) {
            ptr = nullptr;
            return TA_ERR_CUDA;
        }
        bytes = need;
        device = dev;
        return TA_OK;
    }
    void release() {
        if (ptr) cudaFree(ptr);
        ptr = nullptr;
        bytes = 0;
        device = -1;
    }
};
static std::mutex g_arena_mutex;
static Arena g_staging;

// Copy engine of ta_forward_host: uploads and downloads run on two streams of their own and
// the staging memory has two sets, so that the upload of one call overlaps the kernels and the
// download of the previous one (PCIe is full duplex).  Inside a call the (batch, KV head) pairs
// are independent, so a large call is cut into up to kHostGroups groups of them that follow one
// another through upload, kernels and download: the kernels and the download of a group run
// under the upload of the next ones, and a single call costs little more than its upload.
constexpr int kHostGroups = 16;
struct HostPipe {
    bool ready = false;
    int device = -1;
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t in_done[2][kHostGroups] = {}, k_done[2][kHostGroups] = {}, out_done[2] = {};
    bool used[2] = {false, false};
    unsigned turn = 0;
    int init() {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return TA_ERR_CUDA;
        if (ready && dev == device) return TA_OK;
        if (ready) destroy();
        if (cudaStreamCreateWithFlags(&s_in, cudaStreamNonBlocking) != cudaSuccess ||
            cudaStreamCreateWithFlags(&s_out, cudaStreamNonBlocking) != cudaSuccess)
            return TA_ERR_CUDA;
        for (int i = 0; i < 2; ++i) {
            if (cudaEventCreateWithFlags(&out_done[i], cudaEventDisableTiming) != cudaSuccess) return TA_ERR_CUDA;
            for (int g = 0; g < kHostGroups; ++g)
                if (cudaEventCreateWithFlags(&in_done[i][g], cudaEventDisableTiming) != cudaSuccess ||
                    cudaEventCreateWithFlags(&k_done[i][g], cudaEventDisableTiming) != cudaSuccess)
                    return TA_ERR_CUDA;
        }
        used[0] = used[1] = false;
        turn = 0;
        device = dev;
        ready = true;
        return TA_OK;
    }
    void destroy() {
        if (!ready) return;
        cudaStreamDestroy(s_in);
        cudaStreamDestroy(s_out);
        for (int i = 0; i < 2; ++i) {
            cudaEventDestroy(out_done[i]);
            for (int g = 0; g < kHostGroups; ++g) {
                cudaEventDestroy(in_done[i][g]);
                cudaEventDestroy(k_done[i][g]);
            }
        }
        ready = false;
        device = -1;
    }
};
static HostPipe g_host_pipe;
static std::mutex g_host_mutex;   // ta_forward_host calls, one at a time; taken before g_arena_mutex

static int check_arch() {
    static std::atomic<int> cached[64];   // 0 = unknown, 1 = compute capability 10.x, 2 = another
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return TA_ERR_CUDA;
    }
    const bool slot = dev >= 0 && dev < 64;
    const int c = slot ? cached[dev].load(std::memory_order_relaxed) : 0;
    if (c != 0) return c == 1 ? TA_OK : TA_ERR_ARCH;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
        cudaGetLastError();
        return TA_ERR_CUDA;
    }
    if (slot) cached[dev].store(major == 10 ? 1 : 2, std::memory_order_relaxed);
    return major == 10 ? TA_OK : TA_ERR_ARCH;
}

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static bool overlaps(const void *a, size_t a_bytes, const void *b, size_t b_bytes) {
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
    return a0 < b0 + b_bytes && b0 < a0 + a_bytes;
}

static int forward_impl(const ta_params &p);

// A bf16 problem whose head dim has no tensor-core kernel, run on zero-padded copies (ta_pad.cu).
// Everything lives in one stream-ordered allocation: [q'][k'][v'][out'][workspace of the padded call].
// With TA_FLAG_SAVE_HOPS the saved hop inputs are copied back, unpadded, into the caller's workspace.
static int forward_padded(const ta_params &p) {
    const int DP = padded_dim(p.D);
    Plan plan_u, plan_p;
    int rc = build_plan(p.B, p.H, p.H_kv, p.N, p.D, p.dims, p.ndims, p.dtype, p.flags, p.hop_begin, p.hop_end, &plan_u);
    if (rc != TA_OK) return rc;
    if (!aligned16(p.q) || !aligned16(p.k) || !aligned16(p.v) || !aligned16(p.out)) return TA_ERR_ALIGNMENT;
    if (p.workspace && (reinterpret_cast<uintptr_t>(p.workspace) & 255u)) return TA_ERR_ALIGNMENT;
    const size_t tq = (size_t)p.B * p.H * p.N, tkv = (size_t)p.B * p.H_kv * p.N;     // rows
    const size_t tensor_u = tq * p.D * 2, kv_u = tkv * p.D * 2;
    if ((p.flags & TA_FLAG_SAVE_HOPS) && plan_u.save_bytes && !p.workspace) return TA_ERR_WORKSPACE;
    if (p.workspace && p.workspace_bytes < plan_u.scratch_bytes + plan_u.save_bytes + plan_u.flag_bytes)
        return TA_ERR_WORKSPACE;
    if (overlaps(p.out, tensor_u, p.q, tensor_u) || overlaps(p.out, tensor_u, p.k, kv_u) ||
        overlaps(p.out, tensor_u, p.v, kv_u))
        return TA_ERR_INVALID_ARG;
    // (the plan the padded call will build: same flags as forward_impl derives)
    bool any_mask = false;
    if (p.hop_masks)
        for (int i = 0; i < p.ndims; ++i) any_mask = any_mask || p.hop_masks[i] != nullptr;
    const unsigned fusion_off = (p.rope_base > 0.f || p.seq_lens || any_mask) ? (unsigned)TA_FLAG_NO_HOP_FUSION : 0u;
    rc = build_plan(p.B, p.H, p.H_kv, p.N, DP, p.dims, p.ndims, p.dtype, p.flags | fusion_off, p.hop_begin, p.hop_end,
                    &plan_p);
    if (rc != TA_OK) return rc;
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    const size_t q_bytes = up(tq * DP * 2), kv_bytes = up(tkv * DP * 2);
    const size_t ws_bytes = plan_p.scratch_bytes + plan_p.save_bytes + plan_p.flag_bytes;
    cudaStream_t stream = (cudaStream_t)p.stream;
    void *pooled = nullptr;
    if ((rc = pool_alloc(2 * q_bytes + 2 * kv_bytes + ws_bytes, stream, &pooled)) != TA_OK) return rc;
    PooledGuard guard{pooled, stream};
    char *qp = (char *)pooled, *kp = qp + q_bytes, *vp = kp + kv_bytes, *outp = vp + kv_bytes, *wsp = outp + q_bytes;
    if ((rc = launch_pad_rows(p.q, qp, (long long)tq, p.D, DP, 2, stream)) != TA_OK) return rc;
    if ((rc = launch_pad_rows(p.k, kp, (long long)tkv, p.D, DP, 2, stream)) != TA_OK) return rc;
    if ((rc = launch_pad_rows(p.v, vp, (long long)tkv, p.D, DP, 2, stream)) != TA_OK) return rc;
    // a call that starts after the first hop reads its value tensor from `out`
    if (p.hop_begin > 0 && (rc = launch_pad_rows(p.out, outp, (long long)tq, p.D, DP, 2, stream)) != TA_OK) return rc;
    ta_params p2 = p;
    p2.q = qp; p2.k = kp; p2.v = vp; p2.out = outp;
    p2.D = DP;
    p2.softmax_scale = p.softmax_scale != 0.f ? p.softmax_scale : 1.0f / sqrtf((float)p.D);
    if (p.rope_base > 0.f) p2.rope_base = padded_rope_base(p.rope_base, p.D, DP);
    p2.workspace = ws_bytes ? wsp : nullptr;
    p2.workspace_bytes = ws_bytes;
    if ((rc = forward_impl(p2)) != TA_OK) return rc;
    if ((rc = launch_unpad_rows(outp, p.out, (long long)tq, p.D, DP, 2, stream)) != TA_OK) return rc;
    if (p.flags & TA_FLAG_SAVE_HOPS) {
        const size_t slots = plan_p.save_bytes / (tq * DP * 2);
        for (size_t i = 0; i < slots; ++i) {
            rc = launch_unpad_rows(wsp + plan_p.scratch_bytes + i * tq * DP * 2,
                                   (char *)p.workspace + plan_u.scratch_bytes + i * tensor_u, (long long)tq, p.D, DP, 2,
                                   stream);
            if (rc != TA_OK) return rc;
        }
    }
    return TA_OK;
}

static int forward_impl(const ta_params &p) {
    if (!p.q || !p.k || !p.v || !p.out) return TA_ERR_INVALID_ARG;
    if (pad_eligible(p.D, p.dtype, p.flags) && p.ndims >= 1 && p.ndims <= TA_MAX_DIMS &&
        !(p.rope_base > 0.f && ((p.D & 1) || padded_rope_base(p.rope_base, p.D, padded_dim(p.D)) == 0.f))) {
        bool hops = false;
        const int he = (p.hop_begin == 0 && p.hop_end == 0) ? p.ndims : p.hop_end;
        for (int i = p.hop_begin; i >= 0 && i < he && i < p.ndims; ++i) hops = hops || p.dims[i] > 1;
        if (hops) return forward_padded(p);
    }
    if (p.rope_base < 0.f || !(p.rope_base == p.rope_base)) return TA_ERR_INVALID_ARG;
    if (p.rope_base > 0.f && (p.D & 1)) return TA_ERR_UNSUPPORTED;
    if (p.window && p.ndims >= 1 && p.ndims <= TA_MAX_DIMS)
        for (int i = 0; i < p.ndims; ++i)
            if (p.window[i] < 0) return TA_ERR_INVALID_ARG;
    Plan plan;
    // the positional encoding gives every hop its own rotated Q and K: nothing to share, no fusion
    bool any_mask = false;
    if (p.hop_masks && p.ndims >= 1 && p.ndims <= TA_MAX_DIMS)
        for (int i = 0; i < p.ndims; ++i) any_mask = any_mask || p.hop_masks[i] != nullptr;
    const unsigned plan_flags = p.flags | (p.rope_base > 0.f ? (unsigned)TA_FLAG_NO_HOP_FUSION : 0u) |
                                (any_mask ? (unsigned)TA_FLAG_NO_HOP_FUSION : 0u) |
                                (p.seq_lens ? (unsigned)TA_FLAG_NO_HOP_FUSION : 0u);
    int rc = build_plan(p.B, p.H, p.H_kv, p.N, p.D, p.dims, p.ndims, p.dtype, plan_flags, p.hop_begin,
                        p.hop_end, &plan);
    if (rc != TA_OK) return rc;
    if (!aligned16(p.q) || !aligned16(p.k) || !aligned16(p.v) || !aligned16(p.out)) return TA_ERR_ALIGNMENT;
    if (p.workspace && (reinterpret_cast<uintptr_t>(p.workspace) & 255u)) return TA_ERR_ALIGNMENT;
    const size_t tensor_bytes = (size_t)p.B * p.H * p.N * p.D * elem_bytes(p.dtype);
    const size_t kv_bytes = tensor_bytes / p.H * p.H_kv;
    const size_t need = plan.scratch_bytes + plan.save_bytes + plan.flag_bytes;
    if ((p.flags & TA_FLAG_SAVE_HOPS) && plan.save_bytes && !p.workspace) return TA_ERR_WORKSPACE;
    if (p.workspace && p.workspace_bytes < need) return TA_ERR_WORKSPACE;
    if (overlaps(p.out, tensor_bytes, p.q, tensor_bytes) || overlaps(p.out, tensor_bytes, p.k, kv_bytes) ||
        overlaps(p.out, tensor_bytes, p.v, kv_bytes))
        return TA_ERR_INVALID_ARG;
    rc = check_arch();
    if (rc != TA_OK) return rc;

    Problem pb;
    pb.q = p.q; pb.k = p.k; pb.v = p.v; pb.out = p.out;
    pb.B = p.B; pb.H = p.H; pb.H_kv = p.H_kv; pb.N = p.N; pb.D = p.D;
    for (int i = 0; i < p.ndims; ++i) pb.dims[i] = p.dims[i];
    pb.ndims = p.ndims; pb.causal = p.causal ? 1 : 0; pb.dtype = p.dtype;
    pb.scale = p.softmax_scale != 0.f ? p.softmax_scale : 1.0f / sqrtf((float)p.D);
    pb.rope_base = p.rope_base;
    pb.seq_lens = p.seq_lens;
    pb.masks_per_head = (any_mask && p.masks_per_head) ? 1 : 0;
    pb.pdl = 0;
    if ((rc = take_masks(&pb, plan, p.window, p.hop_masks, p.ndims)) != TA_OK) return rc;
    pb.flags = p.flags; pb.hop_begin = p.hop_begin; pb.hop_end = p.hop_end;
    pb.stream = (cudaStream_t)p.stream;

    if (plan.nhops == 0) {
        if (p.hop_begin > 0) return TA_OK;  // value tensor already in `out`
        return launch_broadcast_kv(pb);
    }
    // scratch of this call: the caller's workspace, else a stream-ordered allocation handed back
    // (in stream order) when the last hop has been enqueued
    char *ws = (char *)p.workspace;
    void *pooled = nullptr;
    if (!ws && need) {
        if ((rc = pool_alloc(need, pb.stream, &pooled)) != TA_OK) return rc;
        ws = (char *)pooled;
    }
    auto buffer = [&](int id) -> void * {
        if (id == BUF_V) return const_cast<void *>(p.v);
        if (id == BUF_OUT) return p.out;
        if (id == BUF_SCRATCH) return ws;
        return ws + plan.scratch_bytes + (size_t)(id - 3) * tensor_bytes;
    };
    void *flags = ws ? ws + plan.scratch_bytes + plan.save_bytes : nullptr;
    void *pooled_masks = nullptr;
    rc = upload_long_masks(&pb, plan, &pooled_masks);

    if (rc == TA_OK && p.hop_begin > 0 && plan.hops[0].src == BUF_SCRATCH) {
        const cudaError_t e = cudaMemcpyAsync(ws, p.out, tensor_bytes, cudaMemcpyDeviceToDevice, pb.stream);
        if (e != cudaSuccess) rc = cuda_fail(e);
    }
    for (int j = 0; rc == TA_OK && j < plan.nhops; ++j) {
        const HopDesc &h = plan.hops[j];
        const void *xin = buffer(h.src);
        const int xin_heads = h.src == BUF_V ? p.H_kv : p.H;
        void *xout = buffer(h.dst);
        pb.pdl = (j > 0 && !(p.flags & TA_FLAG_NO_HOP_OVERLAP)) ? 1 : 0;   // follows a hop kernel of this call
        if (h.pair) {
            rc = launch_hop_tc_pair(pb, h, plan.hops[j + 1], xin, xin_heads, xout, flags);
            ++j;
            continue;
        }
        rc = h.path == PATH_TC        ? launch_hop_tc(pb, h, xin, xin_heads, xout)
             : h.path == PATH_TC_LONG ? launch_hop_tc_long(pb, h, xin, xin_heads, xout)
                                      : launch_hop_simt(pb, h, xin, xin_heads, xout);
    }
    pool_free(pooled_masks, pb.stream);
    pool_free(pooled, pb.stream);
    return rc;
}

}  // namespace ta

using namespace ta;

// Result of an entry point: remembers which CUDA error stands behind a TA_ERR_CUDA.
static int finish(int rc) {
    if (rc == TA_ERR_CUDA && tl_last_cuda_error == 0) tl_last_cuda_error = (int)cudaPeekAtLastError();
    return rc;
}

extern "C" {

int ta_last_cuda_error(void) { return tl_last_cuda_error; }

int ta_forward_ex(const ta_params *p) {
    if (!p || p->struct_bytes != sizeof(ta_params)) return TA_ERR_INVALID_ARG;
    tl_last_cuda_error = 0;
    return finish(forward_impl(*p));
}

static int forward_simple(const void *q, const void *k, const void *v, void *out, int B, int H, int H_kv,
                          int N, int D, const int *dims, int ndims, int causal, int dtype,
                          ta_stream_t stream) {
    ta_params p;
    memset(&p, 0, sizeof(p));
    p.struct_bytes = sizeof(p);
    p.q = q; p.k = k; p.v = v; p.out = out;
    p.B = B; p.H = H; p.H_kv = H_kv; p.N = N; p.D = D;
    p.dims = dims; p.ndims = ndims; p.causal = causal; p.dtype = dtype;
    p.stream = stream;
    tl_last_cuda_error = 0;
    return finish(forward_impl(p));
}

int ta_forward(const void *q, const void *k, const void *v, void *out, int B, int H, int H_kv, int N, int D,
               const int *dims, int ndims, int causal, ta_stream_t stream) {
    return forward_simple(q, k, v, out, B, H, H_kv, N, D, dims, ndims, causal, TA_DTYPE_BF16, stream);
}

int ta_forward_f32(const void *q, const void *k, const void *v, void *out, int B, int H, int H_kv, int N,
                   int D, const int *dims, int ndims, int causal, ta_stream_t stream) {
    return forward_simple(q, k, v, out, B, H, H_kv, N, D, dims, ndims, causal, TA_DTYPE_F32, stream);
}

size_t ta_workspace_bytes(int B, int H, int H_kv, int N, int D, const int *dims, int ndims, int dtype,
                          int mode) {
    Plan plan;
    unsigned flags = (mode == TA_WS_FORWARD_SAVE ? TA_FLAG_SAVE_HOPS : 0u) | kPlanAllowPairs;
    if (build_plan(B, H, H_kv, N, D, dims, ndims, dtype, flags, 0, 0, &plan) != TA_OK) return 0;
    if (mode == TA_WS_BACKWARD) return backward_workspace_bytes(B, H, H_kv, N, D, dims, ndims, dtype, TA_DTYPE_BF16, false);
    if (mode == TA_WS_BACKWARD_F32_GRADS)
        return backward_workspace_bytes(B, H, H_kv, N, D, dims, ndims, dtype, TA_DTYPE_F32, false);
    return plan.scratch_bytes + plan.save_bytes + plan.flag_bytes;
}

int ta_forward_host(const void *qh, const void *kh, const void *vh, void *outh, int B, int H, int H_kv, int N,
                    int D, const int *dims, int ndims, int causal, int dtype, ta_stream_t stream) {
    if (!qh || !kh || !vh || !outh) return TA_ERR_INVALID_ARG;
    int rc = validate_shape(B, H, H_kv, N, D, dims, ndims, dtype);
    if (rc != TA_OK) return rc;
    rc = check_arch();
    if (rc != TA_OK) return rc;
    const size_t e = elem_bytes(dtype);
    const size_t qb = (size_t)B * H * N * D * e, kb = (size_t)B * H_kv * N * D * e;
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    const size_t set_bytes = 2 * up(qb) + 2 * up(kb);
    // one call at a time enqueues into the pipe (a lock of its own: the forward pass below takes
    // the arena lock when it needs the library's scratch tensor)
    std::lock_guard<std::mutex> lock(g_host_mutex);
    HostPipe &hp = g_host_pipe;
    if ((rc = hp.init()) != TA_OK) return rc;
    if (g_staging.bytes < 2 * set_bytes || g_staging.device != hp.device) {
        // growing the staging memory: nothing of an earlier call may still be using it
        if (g_staging.ptr) cudaDeviceSynchronize();
        hp.used[0] = hp.used[1] = false;
        if ((rc = g_staging.reserve(2 * set_bytes)) != TA_OK) return rc;
    }
    const int set = (int)(hp.turn++ & 1u);
    char *base = (char *)g_staging.ptr + (size_t)set * set_bytes;
    char *dq = base, *dk = dq + up(qb), *dv = dk + up(kb), *dout = dv + up(kb);
    cudaStream_t s = (cudaStream_t)stream;
    // groups of (batch, KV head) pairs: whole batch entries, each cut into `parts` equal runs of
    // KV heads (with their query heads), as long as a group still carries 32 MB of queries
    int parts = 1;
    for (int d = 1; d <= H_kv; ++d)
        if (H_kv % d == 0 && (long long)B * d <= kHostGroups && qb / ((size_t)B * d) >= (32u << 20)) parts = d;
    const int groups = (long long)B * parts <= kHostGroups ? B * parts : 1;
    const int gB = groups == 1 ? B : 1, gH = groups == 1 ? H : H / parts, gHkv = groups == 1 ? H_kv : H_kv / parts;
    const size_t gq = qb / groups, gk = kb / groups;          // bytes of a group's q (= out) and k (= v)
    // upload (own stream): only waits until this staging set's previous result has been read back
    if (hp.used[set] && cudaStreamWaitEvent(hp.s_in, hp.out_done[set], 0) != cudaSuccess) return TA_ERR_CUDA;
    for (int g = 0; g < groups; ++g) {
        if (cudaMemcpyAsync(dq + g * gq, (const char *)qh + g * gq, gq, cudaMemcpyHostToDevice, hp.s_in) != cudaSuccess ||
            cudaMemcpyAsync(dk + g * gk, (const char *)kh + g * gk, gk, cudaMemcpyHostToDevice, hp.s_in) != cudaSuccess ||
            cudaMemcpyAsync(dv + g * gk, (const char *)vh + g * gk, gk, cudaMemcpyHostToDevice, hp.s_in) != cudaSuccess ||
            cudaEventRecord(hp.in_done[set][g], hp.s_in) != cudaSuccess)
            return TA_ERR_CUDA;
    }
    for (int g = 0; g < groups; ++g) {
        // kernels on the caller's stream, as soon as the group's tensors are in
        if (cudaStreamWaitEvent(s, hp.in_done[set][g], 0) != cudaSuccess) return TA_ERR_CUDA;
        rc = forward_simple(dq + g * gq, dk + g * gk, dv + g * gk, dout + g * gq, gB, gH, gHkv, N, D, dims, ndims, causal,
                            dtype, stream);
        if (rc != TA_OK) return rc;
        if (cudaEventRecord(hp.k_done[set][g], s) != cudaSuccess) return TA_ERR_CUDA;
        // download (own stream)
        if (cudaStreamWaitEvent(hp.s_out, hp.k_done[set][g], 0) != cudaSuccess ||
            cudaMemcpyAsync((char *)outh + g * gq, dout + g * gq, gq, cudaMemcpyDeviceToHost, hp.s_out) != cudaSuccess)
            return TA_ERR_CUDA;
    }
    // the caller's stream completes only after the last download
    if (cudaEventRecord(hp.out_done[set], hp.s_out) != cudaSuccess ||
        cudaStreamWaitEvent(s, hp.out_done[set], 0) != cudaSuccess)
        return TA_ERR_CUDA;
    hp.used[set] = true;
    return TA_OK;
}

int ta_backward_ex(const ta_bwd_params *p) {
    if (!p || p->struct_bytes != sizeof(ta_bwd_params)) return TA_ERR_INVALID_ARG;
    tl_last_cuda_error = 0;
    return finish(backward_impl(*p));
}

int ta_backward(const void *dout, const void *q, const void *k, const void *v, const void *out, void *dq,
                void *dk, void *dv, int B, int H, int H_kv, int N, int D, const int *dims, int ndims,
                int causal, void *workspace, size_t workspace_bytes, ta_stream_t stream) {
    (void)out;
    ta_bwd_params p;
    memset(&p, 0, sizeof(p));
    p.struct_bytes = sizeof(p);
    p.dout = dout; p.q = q; p.k = k; p.v = v; p.dq = dq; p.dk = dk; p.dv = dv;
    p.B = B; p.H = H; p.H_kv = H_kv; p.N = N; p.D = D; p.dims = dims; p.ndims = ndims; p.causal = causal;
    p.dtype = TA_DTYPE_BF16; p.grad_dtype = TA_DTYPE_BF16;
    p.workspace = workspace; p.workspace_bytes = workspace_bytes; p.stream = stream;
    tl_last_cuda_error = 0;
    return finish(backward_impl(p));
}

static const char *buf_name(int id) {
    switch (id) {
        case BUF_V: return "v";
        case BUF_OUT: return "out";
        case BUF_SCRATCH: return "scratch";
        default: return "save";
    }
}

int ta_plan_describe(int B, int H, int H_kv, int N, int D, const int *dims, int ndims, int causal, int dtype,
                     unsigned flags, char *buf, size_t cap) {
    if (!buf || cap == 0) return TA_ERR_INVALID_ARG;
    buf[0] = 0;
    Plan plan;
    if (flags & kPlanAllowPairs) return TA_ERR_UNSUPPORTED;
    // (a head dim without a tensor-core kernel: the plan of the zero-padded problem that will run)
    int rc = validate_shape(B, H, H_kv, N, D, dims, ndims, dtype);
    if (rc != TA_OK) return rc;
    const int D_run = pad_eligible(D, dtype, flags) ? padded_dim(D) : D;
    rc = build_plan(B, H, H_kv, N, D_run, dims, ndims, dtype, flags, 0, 0, &plan);
    if (rc != TA_OK) return rc;
    size_t off = 0;
    auto emit = [&](const char *fmt, auto... a) {
        if (off >= cap) return;
        int w = snprintf(buf + off, cap - off, fmt, a...);
        if (w > 0) off += (size_t)w;
    };
    emit("hops=%d causal=%d dtype=%s scratch_bytes=%zu save_bytes=%zu", plan.nhops, causal ? 1 : 0,
         dtype == TA_DTYPE_F32 ? "f32" : "bf16", plan.scratch_bytes, plan.save_bytes);
    if (D_run != D) emit(" padded_head_dim=%d", D_run);
    emit("%s", "\n");
    for (int j = 0; j < plan.nhops; ++j) {
        const HopDesc &h = plan.hops[j];
        if (h.path == PATH_TC && h.nf > 1) {
            emit("hop=%d path=tc-fused hops=%d block=%d blocks_per_tile=%d rows=%d tiles_per_head=%lld src=%s dst=%s sub=",
                 h.hop, h.nf, h.n, h.co, h.rows, h.tiles_inner * h.tiles_outer, buf_name(h.src), buf_name(h.dst));
            for (int f = 0; f < h.nf; ++f) emit("%s%dx%d", f ? "," : "", h.sub_n[f], h.sub_stride[f]);
            emit("%s", "\n");
        } else if (h.path == PATH_TC)
            emit("hop=%d path=tc n=%d stride=%lld outer=%lld ci=%d co=%d rows=%d tiles_per_head=%lld src=%s dst=%s%s%s\n",
                 h.hop, h.n, h.stride, h.outer, h.ci, h.co, h.rows, h.tiles_inner * h.tiles_outer,
                 buf_name(h.src), buf_name(h.dst), h.out_f16 ? " dst_type=f16" : "",
                 h.pair ? " pair=first" : (j > 0 && plan.hops[j - 1].pair ? " pair=second" : ""));
        else if (h.path == PATH_TC_LONG)
            emit("hop=%d path=tc-long n=%d stride=%lld outer=%lld key_blocks=%d tiles_per_item=%d src=%s dst=%s\n", h.hop,
                 h.n, h.stride, h.outer, (h.n + 127) / 128, long_tiles_per_item(h.n), buf_name(h.src), buf_name(h.dst));
        else
            emit("hop=%d path=simt n=%d stride=%lld outer=%lld src=%s dst=%s\n", h.hop, h.n, h.stride, h.outer,
                 buf_name(h.src), buf_name(h.dst));
    }
    return TA_OK;
}

int ta_device_status(void) {
    if (cudaDeviceSynchronize() != cudaSuccess) return TA_ERR_CUDA;
    unsigned int w1 = 0, w2 = 0, w3 = 0, w4 = 0, w5 = 0, w6 = 0, w7 = 0;
    if (read_status_tc_forward(&w1) != TA_OK || read_status_tc_backward(&w2) != TA_OK ||
        read_status_tc_fused(&w3) != TA_OK || read_status_tc_long(&w4) != TA_OK ||
        read_status_tc_backward_long(&w5) != TA_OK || read_status_tc_pair(&w6) != TA_OK ||
        read_status_selftest(&w7) != TA_OK)
        return TA_ERR_CUDA;
    return (w1 | w2 | w3 | w4 | w5 | w6 | w7) ? TA_ERR_TIMEOUT : TA_OK;
}

unsigned long long ta_launch_count(void) { return g_launches.load(); }

int ta_release(void) {
    std::lock_guard<std::mutex> host_lock(g_host_mutex);
    std::lock_guard<std::mutex> lock(g_arena_mutex);
    cudaDeviceSynchronize();
    g_staging.release();
    g_host_pipe.destroy();
    {
        std::lock_guard<std::mutex> pool_lock(g_pool_mutex);
        for (int d = 0; d < 64; ++d)
            if (g_pools[d]) cudaMemPoolTrimTo(g_pools[d], 0);   // cached blocks back to the driver
    }
    return TA_OK;
}

const char *ta_status_string(int status) {
    switch (status) {
        case TA_OK: return "ok";
        case TA_ERR_INVALID_ARG: return "invalid argument";
        case TA_ERR_SHAPE: return "shape mismatch: prod(dims) != N or H % H_kv != 0";
        case TA_ERR_UNSUPPORTED: return "unsupported configuration";
        case TA_ERR_ALIGNMENT: return "pointer or row size not 16-byte aligned";
        case TA_ERR_WORKSPACE: return "workspace missing or too small";
        case TA_ERR_ARCH: return "device is not compute capability 10.x";
        case TA_ERR_CUDA: return "CUDA call failed";
        case TA_ERR_TIMEOUT: return "device-side wait timed out";
        case TA_ERR_TOO_LARGE: return "size beyond a fixed limit";
        default: return "unknown status";
    }
}

int ta_version(void) { return 100; }

}  // extern "C"
