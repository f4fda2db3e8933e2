// Internal declarations shared by the translation units of libta_b200.so.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <atomic>

#include "ta.h"

namespace ta {

// Buffers a hop may read its value tensor from / write it to.
enum BufferId { BUF_V = 0, BUF_OUT = 1, BUF_SCRATCH = 2 };

enum HopPath {
    PATH_SIMT = 0,  // generic CUDA-core kernel, any n_i / D, fp32 or bf16 storage
    PATH_TC = 1,     // tcgen05 tensor-core kernel: bf16, D in {64,128}, n_i <= 128 (in place)
    PATH_TC_LONG = 2 // tcgen05 kernel with a loop over key blocks and online softmax: n_i > 128
};

// build_plan flag used inside the library only (never part of the public flag set): plan pair
// launches as a call with TA_FLAG_PAIR_HOPS would (ta_workspace_bytes sizes the counters with it).
constexpr unsigned kPlanAllowPairs = 1u << 16;

// One hop of Algorithm 1 as a strided view X[outer][t][inner][D] of a head:
//   token(outer, t, inner) = outer * n * stride + t * stride + inner.
struct HopDesc {
    int hop;          // index i in dims
    int n;            // n_i, segment length
    long long stride; // s_i = prod_{l>i} n_l  (= number of `inner` positions)
    long long outer;  // N / (n * stride), per head
    int path;         // HopPath
    int src, dst;     // BufferId of the value tensor read / written
    // Tensor-core tiling: a tile packs ci (along inner) x co (along outer) whole segments,
    // rows = ci * co * n <= 128, row r of the tile = (co_l * ci + ci_l) * n + t.
    int ci, co, rows;
    long long tiles_inner, tiles_outer;  // per head
    // Hop fusion: when the trailing dimensions i0..m-1 together span at most 128 tokens, their
    // hops run as ONE tensor-core pass over contiguous blocks of n = prod(dims[i0..]) rows (stride
    // 1): nf > 1 sub-hops, sub-hop f attends along a dimension of extent sub_n[f] whose
    // coordinate has stride sub_stride[f] tokens inside the block.  nf <= 1: an ordinary hop.
    int nf;
    int sub_n[TA_MAX_DIMS], sub_stride[TA_MAX_DIMS], sub_hop[TA_MAX_DIMS];   // sub_hop: index in dims
    // Storage of the value tensor this hop reads / writes: 0 = the call's dtype, 1 = fp16.  Between
    // two tensor-core hops of one call the tensor is an intermediate nobody else reads; fp16 has the
    // size of bf16 and three more mantissa bits, so a hop chain rounds to bf16 once, at its end.
    int in_f16, out_f16;
    // 1: this hop and the next one of the plan run as ONE launch of the pair kernel (the next hop's
    // entry is then skipped by the launch loop); both update `out` in place.
    int pair;
};

struct Plan {
    int nhops;  // hops with n_i > 1
    HopDesc hops[TA_MAX_DIMS];
    bool need_scratch;      // some hop writes to / reads from BUF_SCRATCH
    size_t scratch_bytes;   // B*H*N*D*elem when need_scratch
    size_t save_bytes;      // (nhops-1)*B*H*N*D*elem, hop inputs X_1.. for backward
    size_t flag_bytes;      // completion counters of the pair launches (after scratch and saved hops), 0 if none
};

struct Problem {
    const void *q, *k, *v;
    void *out;
    int B, H, H_kv, N, D;
    int dims[TA_MAX_DIMS];
    int ndims;
    int causal;
    int dtype;
    float scale;  // already resolved (1/sqrt(D) default)
    float rope_base;  // 0 = no positional encoding
    int window[TA_MAX_DIMS];  // per dimension: 0 = none, w > 0 = keys within w positions of the query
    const unsigned char *masks[TA_MAX_DIMS];  // per dimension: NULL or host n x n bytes, non-zero = visible
    const int *seq_lens;                      // device, B valid lengths, or NULL
    // Explicit masks of dimensions longer than 128 (too large for a kernel parameter): device
    // bit matrix, row t = query position, bit u of the row = key position u visible (causal flag and
    // window already folded in), dmask_words 32-bit words per row (a multiple of 4); behind the
    // rows, per 128-position query block, the first and one-past-the-last key block (of 128) that
    // any of its rows sees: 2 ints per block.  NULL for the other dimensions.
    const uint32_t *dmask[TA_MAX_DIMS];
    int dmask_words[TA_MAX_DIMS];
    // 1: every given mask holds one matrix per query head ([H][n][n] bytes on the host; the device
    // copy then holds H bit matrices, followed by H tables of key-block ranges), whatever n is
    int masks_per_head;
    int pdl;   // 1: this launch follows a hop kernel of the same call in the stream and may overlap its tail
    unsigned flags;
    int hop_begin, hop_end;
    cudaStream_t stream;
};

static inline size_t elem_bytes(int dtype) { return dtype == TA_DTYPE_F32 ? 4 : 2; }

// Host-only: validates sizes (not pointers) and builds the plan.  Returns TA_OK / TA_ERR_*.
int validate_shape(int B, int H, int H_kv, int N, int D, const int *dims, int ndims, int dtype);
int build_plan(int B, int H, int H_kv, int N, int D, const int *dims, int ndims, int dtype,
               unsigned flags, int hop_begin, int hop_end, Plan *plan);

// Visibility of key position u from query position t along a hop's dimension (bit u of row t;
// n <= 128): the explicit mask of the dimension combined with the causal flag and the window.
// Passed to the kernels by value (kernel parameter space).
struct HopMask {
    uint32_t bits[128][4];
};
// Host: fills hm for hop `hd`; TA_ERR_UNSUPPORTED if n > 128, TA_ERR_INVALID_ARG if a row is empty.
int build_hop_mask(const Problem &pb, const HopDesc &hd, HopMask *hm);
// Host: sets pb.window / pb.masks from the caller's arrays and checks them against the plan.
int take_masks(Problem *pb, const Plan &plan, const int *window, const unsigned char *const *hop_masks, int ndims);
// Masked hops with n > 128, and every masked hop when the masks differ per head: builds their bit
// matrices on the host, copies them into one pooled device buffer (*pooled; pool_free it after
// the last launch) in stream order and sets pb.dmask.  TA_ERR_INVALID_ARG if a query position
// is left without any visible key.
int upload_long_masks(Problem *pb, const Plan &plan, void **pooled);

// Kernel launchers (each returns TA_OK or TA_ERR_CUDA).  xin has `xin_heads` heads per batch
// (H_kv when reading v, H otherwise); xout always has H heads.
int launch_hop_simt(const Problem &pb, const HopDesc &hd, const void *xin, int xin_heads,
                    void *xout);
int launch_hop_tc(const Problem &pb, const HopDesc &hd, const void *xin, int xin_heads,
                  void *xout);
// Long segments (n_i > 128): key-block loop with online softmax, ta_tc_long.cu.  xin != xout.
int launch_hop_tc_long(const Problem &pb, const HopDesc &hd, const void *xin, int xin_heads, void *xout);
int read_status_tc_long(unsigned int *word);
// Query tiles per work item of that kernel for segments of n positions: 1 (two CTAs per SM) or 2.
int long_tiles_per_item(int n);
// Positional encoding on long-segment hops: rotated bf16 copies of q and k in a buffer taken from
// the library's pool on the call's stream (plus extra_bytes of scratch behind them; the caller
// hands *pooled back with pool_free after its last launch that reads it), and
// dst (=|+=) R^T src for fp32 gradients.
int rope_rotated_copies(const Problem &pb, const HopDesc &hd, const void **rq, const void **rk, size_t extra_bytes,
                        void **extra, void **pooled);
int rope_unrotate_add(const Problem &pb, const HopDesc &hd, const float *src, float *dst, int heads, bool accumulate);
// Statistics pass of the long-segment backward: stats[q_head * N + token] = (log2-sum-exp of the
// row's scaled scores, <g_t, out_t>), B*H*N float2; g laid out like q.
int launch_hop_tc_long_stats(const Problem &pb, const HopDesc &hd, const void *xin, int xin_heads, const void *g,
                             void *stats);
// Two adjacent hops in one L2-ordered launch (ta_tc_pair.cu).  `flags`: device, geo.flag_bytes,
// cleared by the launcher on the stream.  Both hops write `out`; hop A reads xin (v or out).
struct PairGeometry {
    int hsplit;                 // items per GQA group and tile position (query heads per item = g / hsplit)
    uint32_t items_a, items_b;  // work items of one unit in each phase
    uint32_t units, lag, total;
    size_t flag_bytes;
    double window_bytes;        // bytes touched between the two hops of a unit (must sit in L2 to pay)
};
bool pair_geometry(int B, int H, int H_kv, const HopDesc &ha, const HopDesc &hb, int num_sms, PairGeometry *geo);
int launch_hop_tc_pair(const Problem &pb, const HopDesc &ha, const HopDesc &hb, const void *xin, int xin_heads,
                       void *out, void *flags);
int read_status_tc_pair(unsigned int *word);
int read_status_selftest(unsigned int *word);
// Stream-ordered device memory from the library's own pool of the current device (created on
// first use; trimmed by ta_release): no device-wide synchronisation, nothing shared between
// streams or host threads, capturable.  pool_free returns the memory in stream order.
int pool_alloc(size_t bytes, cudaStream_t stream, void **ptr);
void pool_free(void *ptr, cudaStream_t stream);
// hands a pooled buffer back (in stream order) on every way out of a scope
struct PooledGuard {
    void *ptr;
    cudaStream_t stream;
    ~PooledGuard() { pool_free(ptr, stream); }
};
// Fused trailing hops (hd.nf > 1), ta_tc_fused.cu; called through launch_hop_tc.
int launch_hop_tc_fused(const Problem &pb, const HopDesc &hd, const void *xin, int xin_heads, void *xout);
// out[b,h] = v[b, h / (H/H_kv)] (all dims equal to 1).
int launch_broadcast_kv(const Problem &pb);

// Backward of one tensor-core hop (ta_tc_bwd.cu).  x = the hop's input value tensor (x_heads
// heads per batch), g_in = gradient w.r.t. the hop's output, g_out = gradient w.r.t. its input
// (bf16, may alias g_in; NULL when first_hop, where it is summed over the group into dv_acc
// instead).  accumulate = false: dq_acc / dk_acc are overwritten (the first hop processed),
// true: added to.  dv_acc is always overwritten (only the first hop writes it).
int launch_hop_tc_bwd(const Problem &pb, const HopDesc &hd, const void *x, int x_heads, const void *g_in,
                      void *g_out, float *dq_acc, float *dk_acc, float *dv_acc, bool first_hop, bool accumulate);
// Backward of one hop on the generic CUDA-core kernels (ta_simt_bwd.cu): any n_i, D <= 256, bf16
// storage.  Same arguments; g_out must differ from g_in (the key side reads every row of g_in),
// stats: B*H*N float2 of scratch (per-row log-sum-exp and rowsum(A o dP)).
int launch_hop_simt_bwd(const Problem &pb, const HopDesc &hd, const void *x, int x_heads, const void *g_in,
                        void *g_out, float *dq_acc, float *dk_acc, float *dv_acc, void *stats, bool first_hop,
                        bool accumulate);
// Backward of a long-segment hop on tensor cores (ta_tc_bwd_long.cu) where tc_bwd_long_eligible:
// bf16, D in {64,128}, no explicit mask.  Same arguments as
// launch_hop_simt_bwd (g_out != g_in; stats: B*H*N float2 of scratch).
bool tc_bwd_long_eligible(const Problem &pb, const HopDesc &hd);
int launch_hop_tc_bwd_long(const Problem &pb, const HopDesc &hd, const void *x, int x_heads, const void *g_in,
                           void *g_out, float *dq_acc, float *dk_acc, float *dv_acc, void *stats, bool first_hop,
                           bool accumulate);
int launch_f32_to_bf16(const float *src, void *dst, long long n, cudaStream_t stream);
// Head dims without a tensor-core kernel (ta_pad.cu): bf16 problems with D < 128, D != 64 run on
// zero-padded copies of D' = padded_dim(D) columns (first half of the features at column 0, second
// half at D' / 2), unless TA_FLAG_NO_TENSOR_CORE asks for the generic kernels.  elem: bytes per element.
bool pad_eligible(int D, int dtype, unsigned flags);
int padded_dim(int D);
int launch_pad_rows(const void *src, void *dst, long long rows, int D, int DP, int elem, cudaStream_t stream);
int launch_unpad_rows(const void *src, void *dst, long long rows, int D, int DP, int elem, cudaStream_t stream);
// base' with base'^(-2c / D') = base^(-2c / D); 0 when it leaves the float range
float padded_rope_base(float base, int D, int DP);
int launch_group_sum(const void *dout, int dout_is_f32, void *dv, int dv_is_f32, int B, int H, int H_kv,
                     long long per_head, cudaStream_t stream);

int backward_impl(const ta_bwd_params &p);
size_t backward_workspace_bytes(int B, int H, int H_kv, int N, int D, const int *dims, int ndims, int dtype,
                                int grad_dtype, bool have_saved_hops);

void count_launch(unsigned n = 1);

// TMA map of one tensor through a hop's strided view (ta_tc.cu); elem = 2 (bf16) or 4 (fp32).
int make_hop_map(CUtensorMap *map, const void *base, int heads_total, int N, int D, const HopDesc &hd, int elem);
// Same view with an explicit box: box_t positions along the hop's dimension, box_inner x box_outer segments.
int make_view_map(CUtensorMap *map, const void *base, int heads_total, int N, int D, const HopDesc &hd, int elem,
                  int box_t, int box_inner, int box_outer);

// Device error words (bounded waits that expired), one per tensor-core translation unit:
// copies the word to *word and clears it.
int read_status_tc_forward(unsigned int *word);
int read_status_tc_backward(unsigned int *word);
int read_status_tc_fused(unsigned int *word);
int read_status_tc_backward_long(unsigned int *word);

// CUDA error code seen by the last call of this host thread that returned TA_ERR_CUDA.
extern thread_local int tl_last_cuda_error;
inline int cuda_fail(cudaError_t e) {
    tl_last_cuda_error = (int)e;
    return TA_ERR_CUDA;
}

// Every kernel of the library is launched through here: the launch's own return value decides
// (an error some earlier CUDA call left behind in this thread is neither consumed nor mistaken
// for ours).  overlap_prev: programmatic stream serialization -- the kernel may be scheduled
// while the previous kernel in the stream drains and must execute griddepcontrol.wait before it
// touches anything that kernel writes.
template <typename... KArgs, typename... Args>
inline int launch_kernel(void (*kern)(KArgs...), unsigned grid, unsigned block, size_t smem, cudaStream_t stream,
                         bool overlap_prev, Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap_prev ? 1 : 0;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, static_cast<Args &&>(args)...);
    if (e != cudaSuccess) return cuda_fail(e);
    count_launch();
    return TA_OK;
}

// SM count of the calling thread's current device (looked up once per device); *dev gets its ordinal.
int current_device_sms(int *dev);

// "Configured once per device" marker for a launcher's kernel attributes (the maximum dynamic
// shared memory of a function is a per-device setting).  Ordinals beyond 63 configure on every call.
struct PerDeviceOnce {
    std::atomic<unsigned long long> done{0};
    bool is_done(int dev) const { return dev >= 0 && dev < 64 && ((done.load(std::memory_order_acquire) >> dev) & 1ull); }
    void mark(int dev) { if (dev >= 0 && dev < 64) done.fetch_or(1ull << dev, std::memory_order_release); }
};

}  // namespace ta
