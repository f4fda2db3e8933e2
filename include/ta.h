/*
 * ta.h -- C ABI of the B200 tensorized-attention library (libta_b200.so).
 *
 * The library computes the forward (and backward) pass of Tensorized Attention
 * (arxiv 2410.20926, Section 3.2, Algorithm 1) over already-projected q, k, v:
 *
 *     the N tokens of a head are viewed, by row-major reshape, as a tensor
 *     n_1 x ... x n_m  (dims[0] = n_1 varies slowest; prod(dims) == N);
 *     O = V;  for i = 0 .. m-1:  O <- A_i x_i O,  A_i = softmax(Q (x)_i K * scale o M_i)
 *
 * i.e. one "hop" per tensor dimension; hop i is a batch of N / n_i independent
 * n_i x n_i softmax attentions over the tokens {base + t * s_i}, s_i = prod_{l>i} n_l
 * (Eq. 3 / Eq. 4: mode-i flattening; done here by strided addressing, nothing is ever
 * transposed in memory).  Q and K are the same in every hop; only O is carried.
 * The causal mask M_i keeps key coordinate u <= query coordinate t along dimension i and
 * removes the other entries from the softmax.  Query head h reads KV head h / (H / H_kv).
 *
 * Conventions common to every call
 *   - Pointers named q/k/v/out/dout/dq/dk/dv/workspace are DEVICE pointers unless the
 *     function name ends in _host.  `dims` is always a HOST pointer, read during the call.
 *   - Layout: q, out, dout, dq: [B][H][N][D];  k, v, dk, dv: [B][H_kv][N][D];
 *     contiguous, D innermost, token order = row-major order of the n_1 x ... x n_m tensor.
 *     Base pointers must be 16-byte aligned.
 *   - All buffers are owned by the caller.  `out` must not overlap q, k or v (checked:
 *     TA_ERR_INVALID_ARG).
 *   - Calls only enqueue work on `stream` (they do not synchronise) unless stated.
 *   - Return value: TA_OK (0) or a negative TA_ERR_* code; nothing is thrown, printed or
 *     aborted.  On an error return no kernel has been launched by that call.
 *   - Hops with n_i == 1 are identities and are skipped.  ndims == 1 is ordinary attention.
 *   - Kernels are built for sm_100a only; on another device the calls return TA_ERR_ARCH.
 *   - Host threads: the calls may be made from several threads at once, on the same or on
 *     different streams and devices (the calling thread's current device is used).  Two calls
 *     whose kernels can overlap on the GPU must not share memory they write (outputs, caller
 *     workspaces).  Scratch the library takes by itself when `workspace` is NULL is a
 *     stream-ordered allocation (cudaMallocFromPoolAsync on the call's stream, from a memory pool
 *     the library creates per device, returned with cudaFreeAsync behind the call's last kernel):
 *     it is private to the call, involves no device-wide synchronisation and may be captured in
 *     a CUDA graph.  ta_forward_static is the exception (one fixed array, see there).
 */
#ifndef TA_B200_H
#define TA_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Same type as the CUDA runtime's cudaStream_t. */
typedef struct CUstream_st *ta_stream_t;

enum {
    TA_OK = 0,
    TA_ERR_INVALID_ARG = -1, /* NULL pointer, non-positive size, ndims outside [1, TA_MAX_DIMS], dims[i] < 1 */
    TA_ERR_SHAPE = -2,       /* prod(dims) != N, or H % H_kv != 0 */
    TA_ERR_UNSUPPORTED = -3, /* D > TA_MAX_HEAD_DIM, unknown dtype or flag */
    TA_ERR_ALIGNMENT = -4,   /* a base pointer is not 16-byte aligned */
    TA_ERR_WORKSPACE = -5,   /* workspace missing or too small (see ta_workspace_bytes) */
    TA_ERR_ARCH = -6,        /* current device is not compute capability 10.x */
    TA_ERR_CUDA = -7,        /* a CUDA runtime / driver call failed (cudaGetLastError is preserved) */
    TA_ERR_TIMEOUT = -8,     /* a bounded device-side wait gave up (seen by ta_device_status) */
    TA_ERR_TOO_LARGE = -9    /* size beyond a documented fixed limit */
};

enum { TA_DTYPE_BF16 = 0, TA_DTYPE_F32 = 1 };

enum {
    TA_MAX_DIMS = 8,
    TA_MAX_HEAD_DIM = 256
};

/* flags of ta_params.flags */
enum {
    TA_FLAG_NO_TENSOR_CORE = 1u << 0, /* run every hop on the generic CUDA-core kernel (and a  */
                                      /* head dim other than 64 / 128 on the tensors as they are) */
    TA_FLAG_NO_HOP_FUSION = 1u << 1,  /* one launch per hop: trailing hops that together fit one  */
                                      /* 128-row tile are not fused into one pass (and            */
                                      /* TA_FLAG_PAIR_HOPS is ignored)                            */
    TA_FLAG_SAVE_HOPS = 1u << 2,      /* store hop inputs X_1..X_{m-1} in the workspace (for ta_backward) */
    TA_FLAG_NO_HOP_OVERLAP = 1u << 3, /* launch every hop fully serialised.  By default a hop's kernel  */
                                      /* may start on SMs the previous hop has left and prefetch its   */
                                      /* first Q / K tiles (programmatic dependent launch); it waits    */
                                      /* for that hop before touching the value tensor.  Same results.  */
    TA_FLAG_BF16_INTERMEDIATES = 1u << 5, /* store the value tensor between hops as bf16.  By default,  */
                                      /* between two tensor-core hops (n_i <= 128) of one call it is    */
                                      /* stored in `out` as fp16 -- same bytes, three more mantissa     */
                                      /* bits -- and only the last hop rounds to bf16.  Every value of  */
                                      /* that tensor is a convex combination of entries of v, so fp16   */
                                      /* is safe while |v| <= 65504 (and entries below 6e-8 flush to 0); */
                                      /* set this flag for inputs outside that range.  Implied by       */
                                      /* TA_FLAG_SAVE_HOPS (the backward reads the hop inputs as bf16). */
    TA_FLAG_PAIR_HOPS = 1u << 4       /* run two adjacent tensor-core hops whose common block is too    */
                                      /* large for one SM as ONE launch in which the second hop's tiles */
                                      /* follow the first hop's tiles of the same block closely enough  */
                                      /* to find them in the L2 cache (see ta_forward).  Same results,  */
                                      /* bit for bit; half the HBM traffic of the two hops.  Off by     */
                                      /* default: on B200 the distance that keeps the CTAs from waiting */
                                      /* on one another is longer than what the L2 retains; measured    */
                                      /* 5-10 % slower than hop by hop.  (TA_PAIR_LAG_UNITS=<n> in the   */
                                      /* environment sets that distance, in blocks, for measurements.)  */
};

/* modes of ta_workspace_bytes */
enum { TA_WS_FORWARD = 0, TA_WS_FORWARD_SAVE = 1, TA_WS_BACKWARD = 2, TA_WS_BACKWARD_F32_GRADS = 3 };

/*
 * Forward pass, bf16 storage (Algorithm 1; fp32 accumulation and fp32 softmax; the
 * attention weights are rounded to 16 bits before the value product, and the value tensor
 * carried between hops is stored in `out` in 16 bits: as fp16 between two tensor-core hops,
 * whose weights are then fp16 too, else as bf16; the result is bf16).
 *   q [B,H,N,D], k, v [B,H_kv,N,D]: device, bf16, read only.
 *   out [B,H,N,D]: device, bf16, written (used as the in-place value tensor between hops).
 *   dims: host array of ndims positive ints, prod == N.  causal: 0 or 1.
 * Scale is 1/sqrt(D) in every hop (Eq. 4).
 * Hops with D in {64,128} and n_i <= 128 run on the tensor-core kernel in place in `out` and
 * need no other memory.  Hops with n_i > 128 (key-block loop with online softmax on the tensor
 * cores, D in {64,128}) cannot update in place: for them the library takes a scratch buffer of
 * B*H*N*D elements from its memory pool for the duration of the call (stream-ordered, see
 * above).  ta_forward_ex takes a caller workspace instead.
 * Other head dims below 128 (100, 96, 80, 40, odd ones ...): the same tensor-core kernels run on
 * zero-padded copies of q, k, v with 64 or 128 columns, and the result is copied back without the
 * padding (zero columns add nothing to Q K^T and give zero output columns; the scale stays
 * 1/sqrt(D); the positional encoding keeps its pairs c, c + D/2 and its frequencies).  The copies
 * -- about 2.3 x (2 H + 2 H_kv) / H times the value tensor -- and the padded problem's scratch
 * come from the memory pool whether or not the caller passed a workspace; hop inputs saved with
 * TA_FLAG_SAVE_HOPS arrive in the caller's workspace in the caller's layout; the backward does the
 * same with dout and the gradients and recomputes the hop inputs.  With TA_FLAG_NO_TENSOR_CORE,
 * for D > 128 and for fp32 tensors the generic CUDA-core kernels run on the tensors as they are.
 * With TA_FLAG_PAIR_HOPS (ta_forward_ex), two adjacent hops with D in {64,128} and n_i <= 128
 * whose common block (n_i * n_{i+1} * s_{i+1} tokens) is too large for one SM but small against
 * the L2 cache run as ONE cooperative launch in which the second hop's tiles follow the first
 * hop's tiles of the same block closely enough to find them in L2 (same arithmetic, same result
 * bit for bit as hop-by-hop launches).  That launch needs a few KB of completion counters, taken
 * from the pool or from the workspace (ta_workspace_bytes accounts for them).
 */
int ta_forward(const void *q, const void *k, const void *v, void *out,
               int B, int H, int H_kv, int N, int D,
               const int *dims, int ndims, int causal, ta_stream_t stream);

/* Same, fp32 storage and fp32 arithmetic throughout (CUDA-core kernels; no tensor cores,
 * because TF32 would not meet a 1e-4 tolerance). */
int ta_forward_f32(const void *q, const void *k, const void *v, void *out,
                   int B, int H, int H_kv, int N, int D,
                   const int *dims, int ndims, int causal, ta_stream_t stream);

/* Extended forward.  Zero-initialise the struct, set struct_bytes = sizeof(ta_params). */
typedef struct ta_params {
    size_t struct_bytes;   /* sizeof(ta_params) of the caller's header                       */
    const void *q, *k, *v; /* device                                                         */
    void *out;             /* device                                                         */
    int B, H, H_kv, N, D;
    const int *dims;       /* host                                                           */
    int ndims;
    int causal;
    int dtype;             /* TA_DTYPE_*                                                     */
    float softmax_scale;   /* 0 -> 1/sqrt(D)                                                 */
    void *workspace;       /* device, 256-byte aligned, or NULL                              */
    size_t workspace_bytes;
    unsigned flags;        /* TA_FLAG_*                                                      */
    int hop_begin;         /* run hops [hop_begin, hop_end) only; 0,0 -> all hops.  With      */
    int hop_end;           /* hop_begin > 0 the value tensor is read from `out` (layout of q) */
                           /* instead of v.                                                  */
    float rope_base;       /* 0: none.  > 0 (Llama: 10000): tensorized positional encoding    */
                           /* (Section 3.2), applied inside the kernels -- see ta_forward_ex  */
    const int *window;     /* host, ndims ints, or NULL: per-hop sliding window, see below     */
    const unsigned char *const *hop_masks; /* host, ndims pointers, or NULL: explicit M_i, see below */
    const int *seq_lens;   /* DEVICE, B ints, or NULL: valid length per batch entry, see below  */
    int masks_per_head;    /* 0: hop_masks[i] is one n_i x n_i matrix for every head;            */
                           /* 1: H matrices, one per query head ([H][n_i][n_i] bytes)            */
    ta_stream_t stream;
} ta_params;

/*
 * ta_forward_ex: as ta_forward with every option explicit.  If `workspace` is non-NULL it
 * is used for the generic kernel's second value buffer (and, with TA_FLAG_SAVE_HOPS, for
 * the hop inputs X_1..X_{m-1}, [m-1][B][H][N][D] in the storage dtype, which ta_backward
 * reads); it must hold ta_workspace_bytes(...) bytes or TA_ERR_WORKSPACE is returned.
 *
 * Tensorized positional encoding (Section 3.2, "Tensorized Positional Encoding": a token's
 * position is the vector of its coordinates j_1..j_m, encoded with RoPE as in Llama).  With
 * rope_base > 0 the un-rotated q and k are passed as usual and, in hop i, every query and
 * key is rotated by its coordinate j_i along the dimension the hop attends over: feature c is
 * paired with c + D/2 and turned by the angle j_i * rope_base^(-2c/D), so the hop's scores
 * depend on relative positions along that dimension.  The rotation happens on the operand
 * tiles in shared memory, between the TMA load and the MMA -- no rotated copy of q or k ever
 * exists in global memory.  D must be even (else TA_ERR_UNSUPPORTED); a negative or NaN base
 * is TA_ERR_INVALID_ARG.  The value tensor is never rotated.
 * (Hops with n_i > 128 instead run on rotated copies of q and k, written once per hop into a
 * buffer the library takes from its memory pool for the duration of the hop.)
 * ta_backward_ex takes the same rope_base (ta_backward, the short form, does not).
 *
 * Per-hop sparsity mask (Eq. 3 allows any mask M_i): window[i] = w > 0 keeps, in hop i, only
 * the keys within w positions of the query along dimension i (|t - u| < w; with `causal` also
 * u <= t, i.e. the last w positions up to the query's own); window[i] = 0 or window == NULL:
 * no window.  A query always sees its own position, so no row is empty.  Negative entries
 * are TA_ERR_INVALID_ARG.  ta_backward_ex takes the same array.
 *
 * Explicit masks: hop_masks[i] = NULL, or a host matrix of n_i x n_i bytes (row = query position
 * along dimension i, column = key position, non-zero = visible), the same for every mode-i
 * vector of the hop, applied on top of `causal` and window[i].  Read during the call.  Any
 * pattern can be given this way (block-sparse layouts, a few always-visible leading keys plus a
 * local band, ...).  A query position left without any visible key is TA_ERR_INVALID_ARG.  Up to
 * n_i = 128 the mask travels as a kernel parameter; for longer dimensions the library packs it to
 * a bit matrix (n_i * n_i / 8 bytes) in pooled device memory, copied in stream order from pageable
 * memory (such a call cannot be captured in a CUDA graph), the tensor-core kernel skips the key
 * blocks before the first and after the last one a block of 128 queries sees and tests one bit
 * per score in between, and the backward of such a hop runs on the generic kernels.  With
 * masks_per_head = 1 every non-NULL hop_masks[i] holds H matrices, one per query head (heads of a
 * GQA group may then see different keys; their dK, dV contributions are summed as always); such
 * masks travel as bit matrices in device memory whatever n_i is.  Hops are not fused when a mask
 * is given.  ta_backward_ex takes the same.
 *
 * Valid lengths (padding to prod(dims), batches of different lengths; a mask M_i that depends
 * on the segment): with seq_lens != NULL only the tokens of batch entry b with flat index
 * < seq_lens[b] exist.  A padding token is never visible as a key, and the row of `out` of a
 * padding query is written as 0.  seq_lens is read on the device, in stream order (no host
 * synchronisation); values are clamped to [0, N].  The padding rows of q, k and v must hold
 * finite values (they are multiplied by weights that are exactly 0).  With `causal` the rows
 * below the length equal those of the call without seq_lens (a causal hop only reads tokens of
 * smaller flat index).  Hops are not fused.  ta_backward_ex takes the same array: the padding rows of dq, dk, dv are 0 and those
 * of dout are not used (but must be finite).
 */
int ta_forward_ex(const ta_params *p);

/*
 * Backward pass of Algorithm 1.  The paper states no formula; this is the chain rule through
 * the recurrence X_{i+1} = A_i X_i (X_0 = V, out = X_m), hops in reverse order:
 *     G_m = dout;   per hop:  dP = G_{i+1} X_i^T,  dS = A_i o (dP - rowsum(A_i o dP)) * scale,
 *     G_i = A_i^T G_{i+1},  dQ += dS K,  dK += dS^T Q;   dV = G_0
 * with dQ, dK summed over hops and dK, dV summed over the H/H_kv query heads of a KV head.
 *   dout [B,H,N,D], q, k, v: device, bf16, read only.  `out` is not read (may be NULL).
 *   dq [B,H,N,D], dk, dv [B,H_kv,N,D]: device, bf16, written.
 *   workspace: device, 256-byte aligned, ta_workspace_bytes(..., TA_WS_BACKWARD) bytes.  It
 *   holds the hop inputs X_1..X_{m-1} (recomputed here by running the forward hops), the bf16
 *   gradient G carried between hops, and fp32 accumulators for dq, dk, dv, which are rounded
 *   to bf16 once at the end.
 * Arithmetic: bf16 operands, fp32 accumulation; the attention weights are recomputed.
 * The sums over the query heads of a group are taken inside one CTA and the sums over hops in
 * launch order (no atomics), so the result is bit-reproducible from run to run.
 * Hops with D in {64,128} run on tensor-core backward kernels: one for n_i <= 128, and for longer
 * segments a block-by-block one (its dQ -- and, on small problems where a group's heads are split
 * over CTAs, dK and dV -- are summed by reduce-adds whose order is not fixed, so they are
 * reproducible only up to fp32 summation order).  Other head dims up to 256 run on generic
 * CUDA-core kernels with fp32 arithmetic.  Hops with n_i > 128 or on the generic kernels need a second G
 * buffer and two floats per query row in the workspace (ta_workspace_bytes accounts for them).
 * D > 256: TA_ERR_UNSUPPORTED.
 */
int ta_backward(const void *dout, const void *q, const void *k, const void *v, const void *out,
                void *dq, void *dk, void *dv,
                int B, int H, int H_kv, int N, int D,
                const int *dims, int ndims, int causal,
                void *workspace, size_t workspace_bytes, ta_stream_t stream);

/* Extended backward.  Zero-initialise, set struct_bytes = sizeof(ta_bwd_params). */
typedef struct ta_bwd_params {
    size_t struct_bytes;
    const void *dout, *q, *k, *v; /* device, bf16                                              */
    void *dq, *dk, *dv;           /* device, grad_dtype                                        */
    int B, H, H_kv, N, D;
    const int *dims;              /* host                                                      */
    int ndims;
    int causal;
    int dtype;                    /* storage of q, k, v, dout: TA_DTYPE_BF16, or TA_DTYPE_F32    */
                                  /* (generic kernels, fp32 throughout; needs grad_dtype F32)   */
    int grad_dtype;               /* TA_DTYPE_BF16, or TA_DTYPE_F32: dq/dk/dv are the fp32      */
                                  /* accumulators themselves (no final rounding, less workspace)*/
    float softmax_scale;          /* 0 -> 1/sqrt(D)                                            */
    float rope_base;              /* 0: none; > 0: tensorized positional encoding as in        */
                                  /* ta_forward_ex (q, k un-rotated; dq, dk are the gradients   */
                                  /* with respect to the un-rotated q, k).  D must be even.     */
    const int *window;            /* host, ndims ints, or NULL: sliding windows as in ta_forward_ex */
    const unsigned char *const *hop_masks; /* host, ndims pointers, or NULL: explicit masks, as in ta_forward_ex */
    const int *seq_lens;          /* DEVICE, B ints, or NULL: valid lengths, as in ta_forward_ex */
    int masks_per_head;           /* as in ta_forward_ex                                        */
    const void *saved_hops;       /* X_1..X_{m-1} as written by ta_forward_ex(TA_FLAG_SAVE_HOPS) */
                                  /* (the part of its workspace after the scratch tensor), or    */
                                  /* NULL: recomputed                                          */
    void *workspace;              /* device, 256-byte aligned                                  */
    size_t workspace_bytes;       /* >= ta_workspace_bytes(.., TA_WS_BACKWARD[_F32_GRADS])      */
    ta_stream_t stream;
} ta_bwd_params;

int ta_backward_ex(const ta_bwd_params *p);

/* Bytes of device workspace a call needs (0 if none); mode = TA_WS_*.  dtype = TA_DTYPE_*.
 * Returns 0 for invalid shapes as well (the call itself reports the error). */
size_t ta_workspace_bytes(int B, int H, int H_kv, int N, int D,
                          const int *dims, int ndims, int dtype, int mode);

/*
 * Whole forward pass from HOST buffers (bf16 or fp32 by `dtype`): copies q, k, v to device
 * staging memory owned by the library (two sets, allocated on first use, grown on demand,
 * released by ta_release), runs ta_forward_ex there on `stream` and copies `out` back.  The
 * uploads and the download run on two copy streams of the library, tied to `stream` by events:
 * `stream` completes only when out_host has been written, while the upload of the NEXT call can
 * already run during this call's kernels and download (PCIe is full duplex), so back-to-back
 * calls cost about the longer of the two transfer directions.  The upload starts when the call
 * is made (it is not ordered after earlier work on `stream`): q_host, k_host, v_host must hold
 * their data by then and stay untouched, like out_host, until `stream` has completed this
 * call.  The host buffers should be pinned for the copies to be asynchronous.  Returns after
 * enqueueing; the caller synchronises `stream` before reading out_host.
 */
int ta_forward_host(const void *q_host, const void *k_host, const void *v_host, void *out_host,
                    int B, int H, int H_kv, int N, int D,
                    const int *dims, int ndims, int causal, int dtype, ta_stream_t stream);

/*
 * ta_forward_static: forward pass that allocates nothing.  (The paper has no counterpart;
 * this entry point exists for deployment reasons only.)
 *
 * For callers that cannot call cudaMalloc where they need the result: code inside a
 * latency-critical serving loop (cudaMalloc synchronises the device), processes whose device
 * memory is entirely managed by a pool the library cannot reach, and plug-ins that are only
 * permitted to launch kernels.  Same arguments and result as ta_forward_ex with default
 * options (dtype = TA_DTYPE_*; for bf16 head dims other than 64 and 128, which ta_forward_ex
 * pads in buffers from its pool, the result of TA_FLAG_NO_TENSOR_CORE: the generic kernels on the
 * tensors as they are), but the second value buffer that hops which cannot update in
 * place need (fp32 storage, n_i > 128, head dims other than 64 / 128) comes from a fixed array of
 * TA_STATIC_SCRATCH_BYTES that is part of the loaded module -- every GPU that loads the
 * library holds those bytes until the process exits.  The call makes no cudaMalloc / cudaFree
 * and calls no allocating routine.
 *   - Problems whose value tensor (B*H*N*D elements) exceeds the array are rejected with
 *     TA_ERR_TOO_LARGE before anything is launched.  Problems that need no second buffer
 *     (bf16, D in {64,128}, every n_i <= 128) have no size limit here.
 *   - The first call on each device looks up the array's device address (with that device
 *     current), which also makes the driver load the module and back the array with memory:
 *     "allocates nothing" holds from the second call on a device.  Make that first call during
 *     start-up, outside latency-critical sections and before any stream capture begins.
 *   - All calls on a device share the one array and it keeps the previous call's contents.
 *     Nothing has to be cleared (each call overwrites every row it later reads), but calls
 *     whose kernels can overlap on the GPU -- different streams or host threads -- race:
 *     issue them on a single stream.
 */
#define TA_STATIC_SCRATCH_BYTES (16u << 20)
int ta_forward_static(const void *q, const void *k, const void *v, void *out,
                      int B, int H, int H_kv, int N, int D,
                      const int *dims, int ndims, int causal, int dtype, ta_stream_t stream);

/*
 * Text description of the launch plan the library would use for a problem (one line per hop:
 * kernel path -- tc, tc-fused, tc-long or simt --, segment length, stride, tile packing,
 * source / destination buffer).  Pure
 * host code: needs no GPU.  Writes at most `cap` bytes including the terminating NUL into
 * `buf` (host) and returns TA_OK or the TA_ERR_* the forward call would return.
 */
int ta_plan_describe(int B, int H, int H_kv, int N, int D, const int *dims, int ndims,
                     int causal, int dtype, unsigned flags, char *buf, size_t cap);

/* Error word written by device code when a bounded wait expired (0 = none).  Synchronises
 * the device; clears the word.  Returns TA_OK, TA_ERR_TIMEOUT or TA_ERR_CUDA. */
int ta_device_status(void);

/*
 * Self-test of the time-out path.  (The paper has no counterpart.)  Every wait inside the
 * tensor-core kernels is bounded; when one expires the kernel records an error word, ends all
 * its roles, lets its copies in flight land and returns, and ta_device_status reports
 * TA_ERR_TIMEOUT.  This call runs that sequence deliberately in a one-CTA kernel: one role
 * starts a bulk copy and then waits, with a limit of `limit_us` microseconds (1 .. 1 000 000),
 * on a barrier nobody arrives at; a second role waits with the ordinary limit and must leave
 * through the abort flag.  Nothing faults and the context stays usable.  Synchronises `stream`.
 * report (host, 4 words, or NULL): [0] 1 = the short wait expired, [1] 1 = the second role left
 * through the abort flag, [2] 1 = the copy in flight was seen to land, [3] nanoseconds spent in
 * the expired wait.  After the call ta_device_status() returns TA_ERR_TIMEOUT once.
 */
int ta_selftest_wait_timeout(unsigned limit_us, unsigned *report, ta_stream_t stream);

/* Number of kernels this library has launched in the calling process (all streams). */
unsigned long long ta_launch_count(void);

/* Frees device memory the library holds (the staging memory of ta_forward_host; cached blocks
 * of its memory pools go back to the driver).  Synchronises the device. */
int ta_release(void);

/* The CUDA runtime error code (cudaError_t as int) behind the last TA_ERR_CUDA that
 * ta_forward*, ta_backward* returned to the calling host thread; 0 if none.  A value
 * <= -1000 is -(1000 + CUresult) of the driver's tensor-map encoder (-1000: encoder not found). */
int ta_last_cuda_error(void);

const char *ta_status_string(int status);
int ta_version(void);

#ifdef __cplusplus
}
#endif
#endif /* TA_B200_H */
