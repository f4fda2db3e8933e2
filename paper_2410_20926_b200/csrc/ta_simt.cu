// Generic CUDA-core kernel for one hop of tensorized attention (Algorithm 1, loop body;
// Eq. 4): any segment length n_i, any head dim <= 256, fp32 or bf16 storage, fp32 arithmetic.
//
// One CTA handles BQ consecutive query positions of one segment and walks the segment's keys
// in blocks of 32 with a running (online) softmax, so n_i is unbounded (ndims == 1 is ordinary
// attention).  Because several CTAs read the same value rows, the hop cannot update the value
// tensor in place: xin and xout are different buffers.
//
// This is the path of the fp32 configuration (TF32 tensor cores cannot meet its 1e-4
// tolerance) and of hops the tcgen05 kernel does not cover.
#include <cuda_bf16.h>

#include <string.h>

#include "ta_internal.h"
#include "ta_simt.cuh"

namespace ta {
namespace {

constexpr int kThreads = 128;
constexpr int kWarps = kThreads / 32;
constexpr int kRowsPerWarp = 4;
constexpr int BQ = kWarps * kRowsPerWarp;  // 16 query rows per CTA
constexpr int BK = 32;                     // keys per block: one per lane

struct SimtArgs {
    int N, D, n, H, H_kv, xin_heads, causal;
    long long stride, outer;      // s_i, outer count per head
    long long segs_per_head;      // outer * stride
    int qblocks;                  // ceil(n / BQ)
    long long items;              // B*H*segs_per_head*qblocks
    float scale;
    float rope_log2_base;         // 0: no positional encoding; else log2 of the RoPE base
    int window;                   // 0, or sliding window along the hop's dimension
    int masked;                   // 1: visibility comes from the HopMask parameter (n <= 128), 2: from dmask
    const uint32_t *dmask;        // device bit matrix (longer dimensions, per-head masks)
    int dmask_words;
    int dmask_heads;              // bit matrices behind dmask: 1 (every head alike) or H
    const int *lens;              // device, valid length per batch entry, or nullptr
};

template <typename T, int DPL>  // DPL = columns per lane, D <= 32 * DPL
__global__ void __launch_bounds__(kThreads)
hop_simt_kernel(const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ xin,
                T *__restrict__ xout, SimtArgs a, const __grid_constant__ HopMask hop_mask) {
    extern __shared__ float smem[];
    const int D = a.D, ldk = D + 1;
    float *sQ = smem;                 // [BQ][D]
    float *sK = sQ + BQ * D;          // [BK][D+1]
    float *sV = sK + BK * ldk;        // [BK][D+1]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = a.H / a.H_kv;

    for (long long item = blockIdx.x; item < a.items; item += gridDim.x) {
        const int qb = (int)(item % a.qblocks);
        long long rest = item / a.qblocks;
        const long long seg = rest % a.segs_per_head;
        const long long bh = rest / a.segs_per_head;
        const int b = (int)(bh / a.H), h = (int)(bh % a.H);
        const long long kvh = (long long)b * a.H_kv + h / g;
        const long long xh = (a.xin_heads == a.H) ? bh : kvh;
        const long long outer = seg / a.stride, inner = seg % a.stride;
        const long long base = outer * a.n * a.stride + inner;   // first token of the segment
        const T *qh = q + bh * (long long)a.N * D;
        const T *kh = k + kvh * (long long)a.N * D;
        const T *xh_p = xin + xh * (long long)a.N * D;
        T *oh = xout + bh * (long long)a.N * D;
        const int t0 = qb * BQ;
        // valid length: the first `exist` positions of this segment are tokens of the batch entry
        int exist = a.n;
        if (a.lens != nullptr) {
            const long long len = min(max(__ldg(a.lens + b), 0), a.N);
            const long long left = (len - base + a.stride - 1) / a.stride;
            exist = len <= base ? 0 : (int)(left < a.n ? left : a.n);
        }

        __syncthreads();   // previous item's smem no longer in use
        for (int idx = threadIdx.x; idx < BQ * D; idx += kThreads) {
            int r = idx / D, c = idx % D, t = t0 + r;
            sQ[idx] = (t < a.n) ? to_f32<T>(qh[(base + (long long)t * a.stride) * D + c]) : 0.f;
        }
        if (a.rope_log2_base != 0.f) {
            __syncthreads();
            rope_rows(sQ, BQ, D, D, t0, a.rope_log2_base);
        }

        float m[kRowsPerWarp], l[kRowsPerWarp], o[kRowsPerWarp][DPL];
#pragma unroll
        for (int r = 0; r < kRowsPerWarp; ++r) {
            m[r] = -INFINITY;
            l[r] = 0.f;
#pragma unroll
            for (int j = 0; j < DPL; ++j) o[r][j] = 0.f;
        }

        const int t_last = min(a.n, t0 + BQ) - 1;
        const int key_end = min(a.causal ? t_last + 1 : a.n, exist);
        for (int k0 = 0; k0 < key_end; k0 += BK) {
            __syncthreads();
            for (int idx = threadIdx.x; idx < BK * D; idx += kThreads) {
                int u = idx / D, c = idx % D, key = k0 + u;
                float kvv = 0.f, xv = 0.f;
                if (key < exist) {
                    long long off = (base + (long long)key * a.stride) * D + c;
                    kvv = to_f32<T>(kh[off]);
                    xv = to_f32<T>(xh_p[off]);
                }
                sK[u * ldk + c] = kvv;
                sV[u * ldk + c] = xv;
            }
            __syncthreads();
            if (a.rope_log2_base != 0.f) {
                rope_rows(sK, BK, ldk, D, k0, a.rope_log2_base);
                __syncthreads();
            }
            const int key = k0 + lane;
#pragma unroll
            for (int r = 0; r < kRowsPerWarp; ++r) {
                const int row = warp * kRowsPerWarp + r, t = t0 + row;
                if (t >= a.n) continue;                        // warp-uniform
                const float *qr = sQ + row * D, *kr = sK + lane * ldk;
                float s = 0.f;
                for (int c = 0; c < D; ++c) s = fmaf(qr[c], kr[c], s);
                s *= a.scale;
                bool valid = key < exist && t < exist && (!a.causal || key <= t) &&
                             (a.window == 0 || (key > t - a.window && key < t + a.window));
                if (a.masked == 1) valid = valid && ((hop_mask.bits[t][key >> 5] >> (key & 31)) & 1u);
                if (a.masked == 2 && valid)
                    valid = ((__ldg(a.dmask + ((size_t)(a.dmask_heads > 1 ? h : 0) * a.n + t) * a.dmask_words + (key >> 5)) >>
                              (key & 31)) & 1u) != 0;
                s = valid ? s : -INFINITY;
                // a block may hold no visible key of this row (window): keep the arithmetic finite
                const float m_new = fmaxf(m[r], warp_max(s));
                const float m_ref = m_new == -INFINITY ? 0.f : m_new;
                const float p = valid ? expf(s - m_ref) : 0.f;
                const float alpha = m[r] == -INFINITY ? 1.f : expf(m[r] - m_ref);
                l[r] = l[r] * alpha + warp_sum(p);
                m[r] = m_new;
#pragma unroll
                for (int j = 0; j < DPL; ++j) o[r][j] *= alpha;
                for (int u = 0; u < BK; ++u) {
                    const float pu = __shfl_sync(0xffffffffu, p, u);
#pragma unroll
                    for (int j = 0; j < DPL; ++j) {
                        const int c = lane + 32 * j;
                        if (c < D) o[r][j] = fmaf(pu, sV[u * ldk + c], o[r][j]);
                    }
                }
            }
        }
#pragma unroll
        for (int r = 0; r < kRowsPerWarp; ++r) {
            const int t = t0 + warp * kRowsPerWarp + r;
            if (t >= a.n) continue;
            const float inv = l[r] > 0.f ? 1.f / l[r] : 0.f;   // a padding row has seen nothing: 0
#pragma unroll
            for (int j = 0; j < DPL; ++j) {
                const int c = lane + 32 * j;
                if (c < D) oh[(base + (long long)t * a.stride) * D + c] = from_f32<T>(o[r][j] * inv);
            }
        }
    }
}

template <typename T>
__global__ void broadcast_kv_kernel(const T *__restrict__ v, T *__restrict__ out, long long per_head,
                                    int H, int H_kv, long long total, const int *lens, int D) {
    const int g = H / H_kv;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        long long bh = i / per_head, r = i % per_head;
        long long b = bh / H, h = bh % H;
        const bool exists = lens == nullptr || r / D < __ldg(lens + b);
        out[i] = exists ? v[(b * H_kv + h / g) * per_head + r] : from_f32<T>(0.f);
    }
}

template <typename T, int DPL>
int launch_t(const Problem &pb, const HopDesc &hd, const void *xin, int xin_heads, void *xout) {
    SimtArgs a;
    a.N = pb.N; a.D = pb.D; a.n = hd.n; a.H = pb.H; a.H_kv = pb.H_kv; a.xin_heads = xin_heads;
    a.causal = pb.causal; a.stride = hd.stride; a.outer = hd.outer;
    a.segs_per_head = hd.outer * hd.stride;
    a.qblocks = (hd.n + BQ - 1) / BQ;
    a.items = (long long)pb.B * pb.H * a.segs_per_head * a.qblocks;
    a.scale = pb.scale;
    a.rope_log2_base = pb.rope_base > 0.f ? log2f(pb.rope_base) : 0.f;
    a.window = pb.window[hd.hop];
    a.masked = 0;
    a.dmask = nullptr;
    a.dmask_words = 0;
    a.lens = pb.seq_lens;
    HopMask hm;
    memset(&hm, 0, sizeof(hm));
    a.dmask_heads = 1;
    if (pb.masks[hd.hop] && (hd.n > 128 || pb.masks_per_head)) {
        if (!pb.dmask[hd.hop]) return TA_ERR_INVALID_ARG;
        a.masked = 2;                                  // bit matrix in device memory
        a.dmask = pb.dmask[hd.hop];
        a.dmask_words = pb.dmask_words[hd.hop];
        a.dmask_heads = pb.masks_per_head ? pb.H : 1;
    } else if (pb.masks[hd.hop]) {
        const int rc = build_hop_mask(pb, hd, &hm);   // explicit mask ^ causal flag ^ window
        if (rc != TA_OK) return rc;
        a.masked = 1;
    }
    size_t smem = sizeof(float) * ((size_t)BQ * pb.D + 2 * (size_t)BK * (pb.D + 1));
    auto kern = hop_simt_kernel<T, DPL>;
    if (smem > 48 * 1024) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return TA_ERR_CUDA;
    }
    long long grid = a.items < (1ll << 20) ? a.items : (1ll << 20);
    return launch_kernel(kern, (unsigned)grid, kThreads, smem, pb.stream, false, (const T *)pb.q, (const T *)pb.k,
                         (const T *)xin, (T *)xout, a, hm);
}

template <typename T>
int launch_d(const Problem &pb, const HopDesc &hd, const void *xin, int xin_heads, void *xout) {
    const int dpl = (pb.D + 31) / 32;
    switch (dpl) {
        case 1: return launch_t<T, 1>(pb, hd, xin, xin_heads, xout);
        case 2: return launch_t<T, 2>(pb, hd, xin, xin_heads, xout);
        case 3: case 4: return launch_t<T, 4>(pb, hd, xin, xin_heads, xout);
        default: return launch_t<T, 8>(pb, hd, xin, xin_heads, xout);
    }
}

}  // namespace

int launch_hop_simt(const Problem &pb, const HopDesc &hd, const void *xin, int xin_heads, void *xout) {
    if (xin == xout) return TA_ERR_INVALID_ARG;   // CTAs read rows other CTAs write: never in place
    if (pb.dtype == TA_DTYPE_F32) return launch_d<float>(pb, hd, xin, xin_heads, xout);
    return launch_d<__nv_bfloat16>(pb, hd, xin, xin_heads, xout);
}

int launch_broadcast_kv(const Problem &pb) {
    const long long per_head = (long long)pb.N * pb.D;
    const long long total = per_head * pb.B * pb.H;
    const unsigned grid = (unsigned)((total + 255) / 256 < 148 * 16 ? (total + 255) / 256 : 148 * 16);
    if (pb.dtype == TA_DTYPE_F32)
        return launch_kernel(broadcast_kv_kernel<float>, grid, 256, 0, pb.stream, false, (const float *)pb.v,
                             (float *)pb.out, per_head, pb.H, pb.H_kv, total, pb.seq_lens, pb.D);
    return launch_kernel(broadcast_kv_kernel<__nv_bfloat16>, grid, 256, 0, pb.stream, false, (const __nv_bfloat16 *)pb.v,
                         (__nv_bfloat16 *)pb.out, per_head, pb.H, pb.H_kv, total, pb.seq_lens, pb.D);
}

}  // namespace ta
