// Host side of the backward pass: workspace layout, recomputation of the hop inputs, the
// reverse hop loop and the final conversion of the fp32 gradient accumulators.
#include <cmath>
#include <cstring>

#include "ta_internal.h"

namespace ta {
namespace {

size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }

struct BwdLayout {
    size_t save_off, gbuf_off, gbuf2_off, stats_off, dq_off, dk_off, dv_off, total;
};

bool any_generic_hop(const Plan &plan) {
    for (int j = 0; j < plan.nhops; ++j)
        if (plan.hops[j].path != PATH_TC) return true;
    return false;
}

// [saved hop inputs X_1..X_{k-1}] [G buffer] [dq fp32] [dk fp32] [dv fp32]; the last three only
// when the caller wants bf16 gradients, the first only when the hop inputs are recomputed.
BwdLayout layout(const Plan &plan, int B, int H, int H_kv, int N, int D, bool need_save, bool need_acc, size_t elem) {
    const size_t tq = (size_t)B * H * N * D, tkv = (size_t)B * H_kv * N * D;
    BwdLayout L;
    size_t off = 0;
    L.save_off = off;
    if (need_save && plan.nhops > 1) off += up256((size_t)(plan.nhops - 1) * tq * elem);
    L.gbuf_off = off;
    if (plan.nhops > 1) off += up256(tq * elem);
    // hops on the generic kernels cannot update G in place and keep two floats per query row
    const bool generic = any_generic_hop(plan);
    L.gbuf2_off = off;
    if (generic && plan.nhops > 2) off += up256(tq * elem);
    L.stats_off = off;
    if (generic) off += up256((size_t)B * H * N * 8);
    L.dq_off = off;
    if (need_acc) off += up256(tq * 4);
    L.dk_off = off;
    if (need_acc) off += up256(tkv * 4);
    L.dv_off = off;
    if (need_acc) off += up256(tkv * 4);
    L.total = off;
    return L;
}

}  // namespace

size_t backward_workspace_bytes(int B, int H, int H_kv, int N, int D, const int *dims, int ndims, int dtype,
                                int grad_dtype, bool have_saved_hops) {
    Plan plan;
    if (dtype == TA_DTYPE_F32 && grad_dtype != TA_DTYPE_F32) return 0;   // fp32 tensors take fp32 gradients
    if (build_plan(B, H, H_kv, N, D, dims, ndims, dtype, TA_FLAG_NO_HOP_FUSION | TA_FLAG_BF16_INTERMEDIATES, 0, 0, &plan) != TA_OK)
        return 0;
    return layout(plan, B, H, H_kv, N, D, !have_saved_hops, grad_dtype != TA_DTYPE_F32,
                  dtype == TA_DTYPE_F32 ? 4 : 2).total;
}

int backward_impl(const ta_bwd_params &p);

namespace {
// A bf16 problem whose head dim has no tensor-core kernel: the backward of the zero-padded problem
// (ta_pad.cu), whose gradients in the padding columns are dropped.  One stream-ordered allocation holds
// [dout'][q'][k'][v'][dq'][dk'][dv'][workspace]; the hop inputs are recomputed there (saved ones are in
// the caller's layout and are not used).
int backward_padded(const ta_bwd_params &p) {
    const int DP = padded_dim(p.D);
    if (p.grad_dtype != TA_DTYPE_BF16 && p.grad_dtype != TA_DTYPE_F32) return TA_ERR_UNSUPPORTED;
    int rc = validate_shape(p.B, p.H, p.H_kv, p.N, p.D, p.dims, p.ndims, p.dtype);
    if (rc != TA_OK) return rc;
    auto misaligned = [](const void *x) { return (reinterpret_cast<uintptr_t>(x) & 15u) != 0; };
    if (misaligned(p.dout) || misaligned(p.q) || misaligned(p.k) || misaligned(p.v) || misaligned(p.dq) ||
        misaligned(p.dk) || misaligned(p.dv))
        return TA_ERR_ALIGNMENT;
    const size_t gelem = p.grad_dtype == TA_DTYPE_F32 ? 4 : 2;
    const size_t tq = (size_t)p.B * p.H * p.N, tkv = (size_t)p.B * p.H_kv * p.N;     // rows
    const size_t q_bytes = up256(tq * DP * 2), kv_bytes = up256(tkv * DP * 2);
    const size_t gq_bytes = up256(tq * DP * gelem), gkv_bytes = up256(tkv * DP * gelem);
    const size_t ws_bytes = backward_workspace_bytes(p.B, p.H, p.H_kv, p.N, DP, p.dims, p.ndims, p.dtype, p.grad_dtype, false);
    cudaStream_t stream = (cudaStream_t)p.stream;
    PooledGuard guard{nullptr, stream};
    if ((rc = pool_alloc(2 * q_bytes + 2 * kv_bytes + gq_bytes + 2 * gkv_bytes + up256(ws_bytes), stream, &guard.ptr)) != TA_OK)
        return rc;
    char *gp = (char *)guard.ptr, *qp = gp + q_bytes, *kp = qp + q_bytes, *vp = kp + kv_bytes, *dqp = vp + kv_bytes,
         *dkp = dqp + gq_bytes, *dvp = dkp + gkv_bytes, *wsp = dvp + gkv_bytes;
    if ((rc = launch_pad_rows(p.dout, gp, (long long)tq, p.D, DP, 2, stream)) != TA_OK) return rc;
    if ((rc = launch_pad_rows(p.q, qp, (long long)tq, p.D, DP, 2, stream)) != TA_OK) return rc;
    if ((rc = launch_pad_rows(p.k, kp, (long long)tkv, p.D, DP, 2, stream)) != TA_OK) return rc;
    if ((rc = launch_pad_rows(p.v, vp, (long long)tkv, p.D, DP, 2, stream)) != TA_OK) return rc;
    ta_bwd_params p2 = p;
    p2.dout = gp; p2.q = qp; p2.k = kp; p2.v = vp;
    p2.dq = dqp; p2.dk = dkp; p2.dv = dvp;
    p2.D = DP;
    p2.softmax_scale = p.softmax_scale != 0.f ? p.softmax_scale : 1.0f / sqrtf((float)p.D);
    if (p.rope_base > 0.f) p2.rope_base = padded_rope_base(p.rope_base, p.D, DP);
    p2.saved_hops = nullptr;
    p2.workspace = ws_bytes ? wsp : nullptr;
    p2.workspace_bytes = ws_bytes;
    if ((rc = backward_impl(p2)) != TA_OK) return rc;
    if ((rc = launch_unpad_rows(dqp, p.dq, (long long)tq, p.D, DP, (int)gelem, stream)) != TA_OK) return rc;
    if ((rc = launch_unpad_rows(dkp, p.dk, (long long)tkv, p.D, DP, (int)gelem, stream)) != TA_OK) return rc;
    return launch_unpad_rows(dvp, p.dv, (long long)tkv, p.D, DP, (int)gelem, stream);
}
}  // namespace

int backward_impl(const ta_bwd_params &p) {
    if (!p.dout || !p.q || !p.k || !p.v || !p.dq || !p.dk || !p.dv) return TA_ERR_INVALID_ARG;
    if (pad_eligible(p.D, p.dtype, 0) && p.ndims >= 1 && p.ndims <= TA_MAX_DIMS && !(p.rope_base < 0.f) &&
        p.rope_base == p.rope_base &&
        !(p.rope_base > 0.f && ((p.D & 1) || padded_rope_base(p.rope_base, p.D, padded_dim(p.D)) == 0.f))) {
        bool hops = false;
        for (int i = 0; i < p.ndims; ++i) hops = hops || p.dims[i] > 1;
        if (hops) return backward_padded(p);
    }
    if (p.dtype != TA_DTYPE_BF16 && p.dtype != TA_DTYPE_F32) return TA_ERR_UNSUPPORTED;
    if (p.grad_dtype != TA_DTYPE_BF16 && p.grad_dtype != TA_DTYPE_F32) return TA_ERR_UNSUPPORTED;
    if (p.dtype == TA_DTYPE_F32 && p.grad_dtype != TA_DTYPE_F32) return TA_ERR_UNSUPPORTED;   // fp32 in, fp32 gradients
    const size_t elem = p.dtype == TA_DTYPE_F32 ? 4 : 2;
    if (p.rope_base < 0.f || !(p.rope_base == p.rope_base)) return TA_ERR_INVALID_ARG;
    if (p.rope_base > 0.f && (p.D & 1)) return TA_ERR_UNSUPPORTED;
    if (p.window && p.ndims >= 1 && p.ndims <= TA_MAX_DIMS)
        for (int i = 0; i < p.ndims; ++i)
            if (p.window[i] < 0) return TA_ERR_INVALID_ARG;
    Plan plan;
    // hop by hop: the backward needs every hop's input
    // the recomputed hop inputs are operands of the backward kernels: bf16 like the gradients
    const unsigned plan_flags = (unsigned)(TA_FLAG_NO_HOP_FUSION | TA_FLAG_BF16_INTERMEDIATES);
    int rc = build_plan(p.B, p.H, p.H_kv, p.N, p.D, p.dims, p.ndims, p.dtype, plan_flags, 0, 0, &plan);
    if (rc != TA_OK) return rc;
    if (p.D > 256) return TA_ERR_UNSUPPORTED;   // limit of the generic backward kernels
    auto misaligned = [](const void *x) { return (reinterpret_cast<uintptr_t>(x) & 15u) != 0; };
    if (misaligned(p.dout) || misaligned(p.q) || misaligned(p.k) || misaligned(p.v) || misaligned(p.dq) ||
        misaligned(p.dk) || misaligned(p.dv) || (p.saved_hops && misaligned(p.saved_hops)))
        return TA_ERR_ALIGNMENT;
    const bool need_acc = p.grad_dtype != TA_DTYPE_F32;
    const BwdLayout L = layout(plan, p.B, p.H, p.H_kv, p.N, p.D, p.saved_hops == nullptr, need_acc, elem);
    if (L.total > 0) {
        if (!p.workspace || p.workspace_bytes < L.total) return TA_ERR_WORKSPACE;
        if (reinterpret_cast<uintptr_t>(p.workspace) & 255u) return TA_ERR_ALIGNMENT;
    }
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
        return TA_ERR_CUDA;
    if (major != 10) return TA_ERR_ARCH;

    Problem pb;
    pb.q = p.q; pb.k = p.k; pb.v = p.v; pb.out = nullptr;
    pb.B = p.B; pb.H = p.H; pb.H_kv = p.H_kv; pb.N = p.N; pb.D = p.D;
    for (int i = 0; i < p.ndims; ++i) pb.dims[i] = p.dims[i];
    pb.ndims = p.ndims; pb.causal = p.causal ? 1 : 0; pb.dtype = p.dtype;
    pb.scale = p.softmax_scale != 0.f ? p.softmax_scale : 1.0f / sqrtf((float)p.D);
    pb.rope_base = p.rope_base;
    pb.seq_lens = p.seq_lens;
    pb.masks_per_head = (p.hop_masks && p.masks_per_head) ? 1 : 0;
    pb.pdl = 0;
    pb.causal = p.causal ? 1 : 0;
    if ((rc = take_masks(&pb, plan, p.window, p.hop_masks, p.ndims)) != TA_OK) return rc;
    pb.flags = 0; pb.hop_begin = 0; pb.hop_end = p.ndims;
    pb.stream = (cudaStream_t)p.stream;
    PooledGuard long_masks{nullptr, pb.stream};      // bit matrices of masked dimensions longer than 128
    if ((rc = upload_long_masks(&pb, plan, &long_masks.ptr)) != TA_OK) return rc;

    const size_t tq = (size_t)p.B * p.H * p.N * p.D, tkv = (size_t)p.B * p.H_kv * p.N * p.D;
    char *ws = (char *)p.workspace;
    float *dq_acc = need_acc ? (float *)(ws + L.dq_off) : (float *)p.dq;
    float *dk_acc = need_acc ? (float *)(ws + L.dk_off) : (float *)p.dk;
    float *dv_acc = need_acc ? (float *)(ws + L.dv_off) : (float *)p.dv;
    const int k = plan.nhops;

    if (k == 0) {
        if (p.seq_lens) return TA_ERR_UNSUPPORTED;   // no hop to apply the valid lengths in
        if (cudaMemsetAsync(dq_acc, 0, tq * 4, pb.stream) != cudaSuccess ||
            cudaMemsetAsync(dk_acc, 0, tkv * 4, pb.stream) != cudaSuccess)
            return TA_ERR_CUDA;
        // every dimension is 1: out = v broadcast over the group, so dv = sum of dout, dq = dk = 0
        rc = launch_group_sum(p.dout, p.dtype == TA_DTYPE_F32 ? 1 : 0, need_acc ? (void *)p.dv : (void *)dv_acc,
                              need_acc ? 0 : 1, p.B, p.H, p.H_kv, (long long)p.N * p.D, pb.stream);
        if (rc != TA_OK) return rc;
    } else {
        // No clearing: the first hop processed (the last hop) stores dq / dk, later ones add to
        // them, and hop 0 stores dv; every row of every head is covered by exactly one tile.
        // X_j = input of hop j: X_0 = v, X_1.. = saved (or recomputed here by running hops 0..k-2)
        const char *saved = p.saved_hops ? (const char *)p.saved_hops : ws + L.save_off;
        auto hop_input = [&](int j) -> const void * { return j == 0 ? p.v : (const void *)(saved + (size_t)(j - 1) * tq * elem); };
        if (!p.saved_hops) {
            for (int j = 0; j + 1 < k; ++j) {
                const HopDesc &h = plan.hops[j];
                const void *xin = hop_input(j);
                const int xin_heads = j == 0 ? p.H_kv : p.H;
                void *xout = ws + L.save_off + (size_t)j * tq * elem;
                rc = h.path == PATH_TC        ? launch_hop_tc(pb, h, xin, xin_heads, xout)
                     : h.path == PATH_TC_LONG ? launch_hop_tc_long(pb, h, xin, xin_heads, xout)
                                              : launch_hop_simt(pb, h, xin, xin_heads, xout);
                if (rc != TA_OK) return rc;
            }
        }
        // G travels from hop to hop in bf16: in place through the tensor-core kernel, from one
        // buffer to the other through the generic kernels
        void *gbuf[2] = {k > 1 ? (void *)(ws + L.gbuf_off) : nullptr, (void *)(ws + L.gbuf2_off)};
        void *stats = ws + L.stats_off;
        const void *g_in = p.dout;
        for (int j = k - 1; j >= 0; --j) {
            const HopDesc &h = plan.hops[j];
            void *g_out = nullptr;
            if (j > 0) g_out = (h.path == PATH_TC && g_in != p.dout) ? const_cast<void *>(g_in)
                                                                      : (g_in == gbuf[0] ? gbuf[1] : gbuf[0]);
            const int x_heads = j == 0 ? p.H_kv : p.H;
            if (h.path == PATH_TC)
                rc = launch_hop_tc_bwd(pb, h, hop_input(j), x_heads, g_in, g_out, dq_acc, dk_acc, dv_acc, j == 0, j != k - 1);
            else if (tc_bwd_long_eligible(pb, h))
                rc = launch_hop_tc_bwd_long(pb, h, hop_input(j), x_heads, g_in, g_out, dq_acc, dk_acc, dv_acc, stats, j == 0,
                                            j != k - 1);
            else
                rc = launch_hop_simt_bwd(pb, h, hop_input(j), x_heads, g_in, g_out, dq_acc, dk_acc, dv_acc, stats, j == 0,
                                         j != k - 1);
            if (rc != TA_OK) return rc;
            g_in = g_out;
        }
    }
    if (need_acc) {
        if ((rc = launch_f32_to_bf16(dq_acc, p.dq, (long long)tq, pb.stream)) != TA_OK) return rc;
        if ((rc = launch_f32_to_bf16(dk_acc, p.dk, (long long)tkv, pb.stream)) != TA_OK) return rc;
        if (k > 0 && (rc = launch_f32_to_bf16(dv_acc, p.dv, (long long)tkv, pb.stream)) != TA_OK) return rc;
    }
    return TA_OK;
}

}  // namespace ta
