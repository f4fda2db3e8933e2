// ta_forward_static: the forward pass for callers that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc at the point where they need attention:
// a latency-critical serving thread (cudaMalloc synchronises the device), processes whose
// memory was handed out up front to a pool that the library knows nothing about, and
// sandboxed plug-ins that are only allowed to launch kernels.
// The ordinary entry points satisfy the generic kernel's need for a second value buffer from
// a caller workspace or from a library arena (cudaMalloc on first use).  This one takes it
// from a fixed array that is part of the loaded module instead, so the call allocates
// nothing: no cudaMalloc / cudaFree, no allocating library routine.
//
// The price is a fixed ceiling (TA_STATIC_SCRATCH_BYTES) and shared state: every call on a
// device uses the same array, so two calls whose kernels may overlap on the GPU (different
// streams, or different host threads) race; issue them on one stream.  The array keeps
// whatever the previous call left in it; nothing needs clearing because the hop that writes
// to the scratch buffer writes every row of the value tensor before a later hop reads it.
#include <mutex>

#include "ta_internal.h"

namespace ta {
namespace {

constexpr size_t kStaticScratchBytes = TA_STATIC_SCRATCH_BYTES;

// Lives in every GPU that loads the library until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void *g_scratch_addr[kMaxDevices] = {};   // device address of g_static_scratch, per device

// In host code `g_static_scratch` is only a handle of the symbol, not a device address; the
// address a kernel can use has to be looked up, once per device, with that device current.
int static_scratch_for_current_device(void **ptr) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return TA_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return TA_ERR_TOO_LARGE;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        cudaError_t e = cudaGetSymbolAddress((void **)&p, g_static_scratch);
        if (e != cudaSuccess || !p) return cuda_fail(e);
        g_scratch_addr[dev] = p;
    }
    *ptr = g_scratch_addr[dev];
    return TA_OK;
}

}  // namespace
}  // namespace ta

using namespace ta;

extern "C" int ta_forward_static(const void *q, const void *k, const void *v, void *out, int B, int H, int H_kv,
                                 int N, int D, const int *dims, int ndims, int causal, int dtype,
                                 ta_stream_t stream) {
    if (!q || !k || !v || !out) return TA_ERR_INVALID_ARG;
    tl_last_cuda_error = 0;
    Plan plan;
    int rc = build_plan(B, H, H_kv, N, D, dims, ndims, dtype, 0u, 0, 0, &plan);
    if (rc != TA_OK) return rc;
    auto misaligned = [](const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
    if (misaligned(q) || misaligned(k) || misaligned(v) || misaligned(out)) return TA_ERR_ALIGNMENT;
    if (plan.scratch_bytes > kStaticScratchBytes) return TA_ERR_TOO_LARGE;

    int dev = 0, major = 0;
    cudaError_t ce = cudaGetDevice(&dev);
    if (ce == cudaSuccess) ce = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (ce != cudaSuccess) return cuda_fail(ce);
    if (major != 10) return TA_ERR_ARCH;

    void *scratch = nullptr;
    if (plan.need_scratch && (rc = static_scratch_for_current_device(&scratch)) != TA_OK) return rc;

    Problem pb;
    pb.q = q; pb.k = k; pb.v = v; pb.out = out;
    pb.B = B; pb.H = H; pb.H_kv = H_kv; pb.N = N; pb.D = D;
    for (int i = 0; i < ndims; ++i) pb.dims[i] = dims[i];
    pb.ndims = ndims; pb.causal = causal ? 1 : 0; pb.dtype = dtype;
    pb.scale = 1.0f / sqrtf((float)D);
    pb.rope_base = 0.f;
    pb.seq_lens = nullptr;
    pb.masks_per_head = 0;
    pb.pdl = 0;
    for (int i = 0; i < TA_MAX_DIMS; ++i) { pb.window[i] = 0; pb.masks[i] = nullptr; pb.dmask[i] = nullptr; pb.dmask_words[i] = 0; }
    pb.flags = 0; pb.hop_begin = 0; pb.hop_end = ndims;
    pb.stream = (cudaStream_t)stream;

    if (plan.nhops == 0) return launch_broadcast_kv(pb);
    for (int j = 0; j < plan.nhops; ++j) {
        const HopDesc &h = plan.hops[j];
        const void *xin = h.src == BUF_V ? v : (h.src == BUF_OUT ? (const void *)out : (const void *)scratch);
        void *xout = h.dst == BUF_OUT ? out : scratch;
        const int xin_heads = h.src == BUF_V ? H_kv : H;
        pb.pdl = j > 0 ? 1 : 0;
        rc = h.path == PATH_TC        ? launch_hop_tc(pb, h, xin, xin_heads, xout)
             : h.path == PATH_TC_LONG ? launch_hop_tc_long(pb, h, xin, xin_heads, xout)
                                      : launch_hop_simt(pb, h, xin, xin_heads, xout);
        if (rc != TA_OK) return rc;
    }
    return TA_OK;
}
