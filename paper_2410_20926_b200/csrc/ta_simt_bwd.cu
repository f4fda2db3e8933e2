// Generic CUDA-core backward of one hop of tensorized attention: any segment length n_i, any
// head dim <= 256, bf16 or fp32 storage, fp32 arithmetic.  Used by ta_backward for the hops the tcgen05
// backward kernel does not cover (segments longer than 128, head dims other than 64 / 128).
//
// The paper gives no backward; this is the chain rule through X_{i+1} = A_i X_i for one hop:
//     dP = G X^T,  dS = A o (dP - rowsum(A o dP)) * scale,
//     G_in = A^T G,  dQ += dS K,  dK += dS^T Q        (G = gradient w.r.t. the hop's output)
// in two kernels that both recompute the scores (nothing of size n x n is stored):
//   hop_simt_bwd_q_kernel  one CTA per 16 query positions of a segment: first the forward row
//       (online softmax, output row O) for lse = m + log l and delta = <G_t, O_t> (which equals
//       rowsum(A o dP)), then a second walk over the keys for dS and dQ.  Writes dQ (fp32,
//       stored or added) and (lse, delta) per row.
//   hop_simt_bwd_k_kernel  one CTA per 16 key positions of a segment and KV head: walks the
//       query heads of the GQA group and their query blocks, A = exp(s - lse), and accumulates
//       G_in (per query head; summed over the group into dV for the first hop) and dK (summed
//       over the group) without atomics, so the result is reproducible.
// Masks as in the forward: causal flag, window, explicit mask (a kernel parameter up to n = 128, a bit
// matrix in device memory beyond), valid lengths.
#include <cuda_bf16.h>

#include <string.h>

#include "ta_internal.h"
#include "ta_simt.cuh"

namespace ta {
namespace {

constexpr int kThreads = 128;
constexpr int kWarps = kThreads / 32;
constexpr int kPerWarp = 4;
constexpr int BR = kWarps * kPerWarp;   // rows a CTA owns: 16 queries (q kernel) or 16 keys (k kernel)
constexpr int BL = 32;                  // rows it walks per step: one per lane

struct SimtBwdArgs {
    int N, D, n, H, H_kv, x_heads, causal;
    long long stride, segs_per_head;
    int rblocks;                  // ceil(n / BR)
    long long items;
    float scale;
    float rope_log2_base;         // 0: no positional encoding
    int window, masked;           // masked: 1 = HopMask parameter (n <= 128), 2 = device bit matrix dmask
    const uint32_t *dmask;
    int dmask_words, dmask_heads; // bit matrices behind dmask: 1 (every head alike) or H
    const int *lens;
    int first_hop, accumulate;
};

__device__ __forceinline__ int segment_exist(const SimtBwdArgs &a, int b, long long base) {
    if (a.lens == nullptr) return a.n;
    const long long len = min(max(__ldg(a.lens + b), 0), a.N);
    const long long left = (len - base + a.stride - 1) / a.stride;
    return len <= base ? 0 : (int)(left < a.n ? left : a.n);
}

__device__ __forceinline__ bool pair_visible(const SimtBwdArgs &a, const HopMask &hm, int t, int key, int exist, int h) {
    bool v = key < exist && t < exist && (!a.causal || key <= t) &&
             (a.window == 0 || (key > t - a.window && key < t + a.window));
    if (a.masked == 1) v = v && ((hm.bits[t][key >> 5] >> (key & 31)) & 1u);
    if (a.masked == 2 && v)
        v = ((__ldg(a.dmask + ((size_t)(a.dmask_heads > 1 ? h : 0) * a.n + t) * a.dmask_words + (key >> 5)) >> (key & 31)) & 1u) != 0;
    return v;
}

// ------------------------------------------------------------------------------------ query side
template <typename T, int DPL>
__global__ void __launch_bounds__(kThreads)
hop_simt_bwd_q_kernel(const T *__restrict__ q, const T *__restrict__ k,
                      const T *__restrict__ x, const T *__restrict__ g,
                      float *__restrict__ dq_acc, float2 *__restrict__ stats, SimtBwdArgs a,
                      const __grid_constant__ HopMask hop_mask) {
    extern __shared__ float smem[];
    const int D = a.D, ld = D + 1;
    float *sQ = smem;                  // [BR][D]   query rows (rotated); later the dQ rows
    float *sG = sQ + BR * D;           // [BR][D]   rows of G
    float *sK = sG + BR * D;           // [BL][D+1] key rows (rotated)
    float *sX = sK + BL * ld;          // [BL][D+1] value rows
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int grp = a.H / a.H_kv;

    for (long long item = blockIdx.x; item < a.items; item += gridDim.x) {
        const int qb = (int)(item % a.rblocks);
        long long rest = item / a.rblocks;
        const long long seg = rest % a.segs_per_head;
        const long long bh = rest / a.segs_per_head;
        const int b = (int)(bh / a.H), h = (int)(bh % a.H);
        const long long kvh = (long long)b * a.H_kv + h / grp;
        const long long xh = (a.x_heads == a.H) ? bh : kvh;
        const long long outer = seg / a.stride, inner = seg % a.stride;
        const long long base = outer * a.n * a.stride + inner;
        const long long per_head = (long long)a.N * D;
        const T *qh = q + bh * per_head, *kh = k + kvh * per_head, *xp = x + xh * per_head, *gh = g + bh * per_head;
        const int t0 = qb * BR;
        const int exist = segment_exist(a, b, base);

        __syncthreads();
        for (int idx = threadIdx.x; idx < BR * D; idx += kThreads) {
            const int r = idx / D, c = idx % D, t = t0 + r;
            const bool in = t < a.n && t < exist;
            const long long off = (base + (long long)t * a.stride) * D + c;
            sQ[idx] = in ? to_f32<T>(qh[off]) : 0.f;
            sG[idx] = in ? to_f32<T>(gh[off]) : 0.f;
        }
        if (a.rope_log2_base != 0.f) {
            __syncthreads();
            rope_rows(sQ, BR, D, D, t0, a.rope_log2_base);
        }

        const int t_last = min(a.n, t0 + BR) - 1;
        const int key_end = min(a.causal ? t_last + 1 : a.n, exist);
        float m[kPerWarp], l[kPerWarp], acc[kPerWarp][DPL];
#pragma unroll
        for (int r = 0; r < kPerWarp; ++r) {
            m[r] = -INFINITY;
            l[r] = 0.f;
#pragma unroll
            for (int j = 0; j < DPL; ++j) acc[r][j] = 0.f;
        }

        auto load_keys = [&](int k0) {
            __syncthreads();
            for (int idx = threadIdx.x; idx < BL * D; idx += kThreads) {
                const int u = idx / D, c = idx % D, key = k0 + u;
                float kv = 0.f, xv = 0.f;
                if (key < exist) {
                    const long long off = (base + (long long)key * a.stride) * D + c;
                    kv = to_f32<T>(kh[off]);
                    xv = to_f32<T>(xp[off]);
                }
                sK[u * ld + c] = kv;
                sX[u * ld + c] = xv;
            }
            __syncthreads();
            if (a.rope_log2_base != 0.f) {
                rope_rows(sK, BL, ld, D, k0, a.rope_log2_base);
                __syncthreads();
            }
        };

        // ---- walk 1: the forward row (m, l, O)
        for (int k0 = 0; k0 < key_end; k0 += BL) {
            load_keys(k0);
            const int key = k0 + lane;
#pragma unroll
            for (int r = 0; r < kPerWarp; ++r) {
                const int row = warp * kPerWarp + r, t = t0 + row;
                if (t >= a.n) continue;
                const float *qr = sQ + row * D, *kr = sK + lane * ld;
                float s = 0.f;
                for (int c = 0; c < D; ++c) s = fmaf(qr[c], kr[c], s);
                s *= a.scale;
                const bool valid = pair_visible(a, hop_mask, t, key, exist, h);
                s = valid ? s : -INFINITY;
                const float m_new = fmaxf(m[r], warp_max(s));
                const float m_ref = m_new == -INFINITY ? 0.f : m_new;
                const float p = valid ? expf(s - m_ref) : 0.f;
                const float alpha = m[r] == -INFINITY ? 1.f : expf(m[r] - m_ref);
                l[r] = l[r] * alpha + warp_sum(p);
                m[r] = m_new;
#pragma unroll
                for (int j = 0; j < DPL; ++j) acc[r][j] *= alpha;
                for (int u = 0; u < BL; ++u) {
                    const float pu = __shfl_sync(0xffffffffu, p, u);
#pragma unroll
                    for (int j = 0; j < DPL; ++j) {
                        const int c = lane + 32 * j;
                        if (c < D) acc[r][j] = fmaf(pu, sX[u * ld + c], acc[r][j]);
                    }
                }
            }
        }
        // lse and delta = <G_t, O_t>; a row that saw nothing (padding) gets weights 0 everywhere
        float lse[kPerWarp], delta[kPerWarp];
#pragma unroll
        for (int r = 0; r < kPerWarp; ++r) {
            const int row = warp * kPerWarp + r;
            float d = 0.f;
#pragma unroll
            for (int j = 0; j < DPL; ++j) {
                const int c = lane + 32 * j;
                if (c < D) d = fmaf(sG[row * D + c], acc[r][j], d);
            }
            d = warp_sum(d);
            const bool live = l[r] > 0.f;
            lse[r] = live ? m[r] + logf(l[r]) : INFINITY;
            delta[r] = live ? d / l[r] : 0.f;
#pragma unroll
            for (int j = 0; j < DPL; ++j) acc[r][j] = 0.f;      // reused for dQ
        }

        // ---- walk 2: dS and dQ
        for (int k0 = 0; k0 < key_end; k0 += BL) {
            load_keys(k0);
            const int key = k0 + lane;
#pragma unroll
            for (int r = 0; r < kPerWarp; ++r) {
                const int row = warp * kPerWarp + r, t = t0 + row;
                if (t >= a.n) continue;
                const float *qr = sQ + row * D, *gr = sG + row * D, *kr = sK + lane * ld, *xr = sX + lane * ld;
                float s = 0.f, dp = 0.f;
                for (int c = 0; c < D; ++c) {
                    s = fmaf(qr[c], kr[c], s);
                    dp = fmaf(gr[c], xr[c], dp);
                }
                const bool valid = pair_visible(a, hop_mask, t, key, exist, h);
                const float p = valid ? expf(s * a.scale - lse[r]) : 0.f;
                const float ds = valid ? p * (dp - delta[r]) * a.scale : 0.f;
                for (int u = 0; u < BL; ++u) {
                    const float du = __shfl_sync(0xffffffffu, ds, u);
#pragma unroll
                    for (int j = 0; j < DPL; ++j) {
                        const int c = lane + 32 * j;
                        if (c < D) acc[r][j] = fmaf(du, sK[u * ld + c], acc[r][j]);
                    }
                }
            }
        }

        // ---- dQ rows (rotated back if the hop rotates), statistics
        __syncthreads();                                   // every warp is done with sQ
#pragma unroll
        for (int r = 0; r < kPerWarp; ++r) {
            const int row = warp * kPerWarp + r;
#pragma unroll
            for (int j = 0; j < DPL; ++j) {
                const int c = lane + 32 * j;
                if (c < D) sQ[row * D + c] = acc[r][j];
            }
        }
        __syncthreads();
        if (a.rope_log2_base != 0.f) {
            rope_rows(sQ, BR, D, D, t0, a.rope_log2_base, -1.f);
            __syncthreads();
        }
        for (int idx = threadIdx.x; idx < BR * D; idx += kThreads) {
            const int r = idx / D, c = idx % D, t = t0 + r;
            if (t >= a.n) continue;
            float *dst = dq_acc + bh * per_head + (base + (long long)t * a.stride) * D + c;
            *dst = a.accumulate ? *dst + sQ[idx] : sQ[idx];
        }
        if (lane == 0) {
#pragma unroll
            for (int r = 0; r < kPerWarp; ++r) {
                const int t = t0 + warp * kPerWarp + r;
                if (t < a.n) stats[bh * a.N + base + (long long)t * a.stride] = make_float2(lse[r], delta[r]);
            }
        }
    }
}

// -------------------------------------------------------------------------------------- key side
template <typename T, int DPL>
__global__ void __launch_bounds__(kThreads)
hop_simt_bwd_k_kernel(const T *__restrict__ q, const T *__restrict__ k,
                      const T *__restrict__ x, const T *__restrict__ g,
                      const float2 *__restrict__ stats, T *__restrict__ g_out,
                      float *__restrict__ dk_acc, float *__restrict__ dv_acc, SimtBwdArgs a,
                      const __grid_constant__ HopMask hop_mask) {
    extern __shared__ float smem[];
    const int D = a.D, ld = D + 1;
    float *sK = smem;                  // [BR][D]   key rows (rotated); later the dK rows
    float *sX = sK + BR * D;           // [BR][D]   value rows
    float *sQ = sX + BR * D;           // [BL][D+1] query rows (rotated)
    float *sG = sQ + BL * ld;          // [BL][D+1] rows of G
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int grp = a.H / a.H_kv;

    for (long long item = blockIdx.x; item < a.items; item += gridDim.x) {
        const int kb = (int)(item % a.rblocks);
        long long rest = item / a.rblocks;
        const long long seg = rest % a.segs_per_head;
        const long long kvh = rest / a.segs_per_head;     // b * H_kv + kv head
        const int b = (int)(kvh / a.H_kv), kv = (int)(kvh % a.H_kv);
        const long long outer = seg / a.stride, inner = seg % a.stride;
        const long long base = outer * a.n * a.stride + inner;
        const long long per_head = (long long)a.N * D;
        const T *kh = k + kvh * per_head;
        const int u0 = kb * BR;
        const int exist = segment_exist(a, b, base);
        const int q_end = min(a.n, exist);

        float acc_k[kPerWarp][DPL], acc_v[kPerWarp][DPL];     // dK and (first hop) dV, summed over the group
#pragma unroll
        for (int r = 0; r < kPerWarp; ++r)
#pragma unroll
            for (int j = 0; j < DPL; ++j) { acc_k[r][j] = 0.f; acc_v[r][j] = 0.f; }

        __syncthreads();
        for (int idx = threadIdx.x; idx < BR * D; idx += kThreads) {
            const int r = idx / D, c = idx % D, key = u0 + r;
            sK[idx] = key < exist ? to_f32<T>(kh[(base + (long long)key * a.stride) * D + c]) : 0.f;
        }
        if (a.rope_log2_base != 0.f) {
            __syncthreads();
            rope_rows(sK, BR, D, D, u0, a.rope_log2_base);
        }

        for (int hh = 0; hh < grp; ++hh) {
            const long long bh = (long long)b * a.H + (long long)kv * grp + hh;
            const long long xh = (a.x_heads == a.H) ? bh : kvh;
            const T *qh = q + bh * per_head, *gh = g + bh * per_head, *xp = x + xh * per_head;
            if (hh == 0 || a.x_heads == a.H) {
                __syncthreads();
                for (int idx = threadIdx.x; idx < BR * D; idx += kThreads) {
                    const int r = idx / D, c = idx % D, key = u0 + r;
                    sX[idx] = key < exist ? to_f32<T>(xp[(base + (long long)key * a.stride) * D + c]) : 0.f;
                }
            }
            float acc_g[kPerWarp][DPL];
#pragma unroll
            for (int r = 0; r < kPerWarp; ++r)
#pragma unroll
                for (int j = 0; j < DPL; ++j) acc_g[r][j] = 0.f;

            const int t_begin = a.causal ? (u0 / BL) * BL : 0;   // causal: queries at or after the keys
            for (int tb = t_begin; tb < q_end; tb += BL) {
                __syncthreads();
                for (int idx = threadIdx.x; idx < BL * D; idx += kThreads) {
                    const int r = idx / D, c = idx % D, t = tb + r;
                    float qv = 0.f, gv = 0.f;
                    if (t < q_end) {
                        const long long off = (base + (long long)t * a.stride) * D + c;
                        qv = to_f32<T>(qh[off]);
                        gv = to_f32<T>(gh[off]);
                    }
                    sQ[r * ld + c] = qv;
                    sG[r * ld + c] = gv;
                }
                __syncthreads();
                if (a.rope_log2_base != 0.f) {
                    rope_rows(sQ, BL, ld, D, tb, a.rope_log2_base);
                    __syncthreads();
                }
                const int t = tb + lane;
                float2 st = make_float2(INFINITY, 0.f);
                if (t < q_end) st = stats[bh * a.N + base + (long long)t * a.stride];
#pragma unroll
                for (int r = 0; r < kPerWarp; ++r) {
                    const int row = warp * kPerWarp + r, key = u0 + row;
                    if (key >= a.n) continue;
                    const float *kr = sK + row * D, *xr = sX + row * D, *qr = sQ + lane * ld, *gr = sG + lane * ld;
                    float s = 0.f, dp = 0.f;
                    for (int c = 0; c < D; ++c) {
                        s = fmaf(qr[c], kr[c], s);
                        dp = fmaf(gr[c], xr[c], dp);
                    }
                    const bool valid = t < q_end && pair_visible(a, hop_mask, t, key, exist, kv * grp + hh);
                    const float p = valid ? expf(s * a.scale - st.x) : 0.f;
                    const float ds = valid ? p * (dp - st.y) * a.scale : 0.f;
                    for (int tt = 0; tt < BL; ++tt) {
                        const float pt = __shfl_sync(0xffffffffu, p, tt);
                        const float dt = __shfl_sync(0xffffffffu, ds, tt);
#pragma unroll
                        for (int j = 0; j < DPL; ++j) {
                            const int c = lane + 32 * j;
                            if (c < D) {
                                acc_g[r][j] = fmaf(pt, sG[tt * ld + c], acc_g[r][j]);
                                acc_k[r][j] = fmaf(dt, sQ[tt * ld + c], acc_k[r][j]);
                            }
                        }
                    }
                }
            }
            // G_in of this query head: its own rows (or, first hop, summed over the group into dV)
#pragma unroll
            for (int r = 0; r < kPerWarp; ++r) {
                const int key = u0 + warp * kPerWarp + r;
                if (key >= a.n) continue;
#pragma unroll
                for (int j = 0; j < DPL; ++j) {
                    const int c = lane + 32 * j;
                    if (c >= D) continue;
                    if (a.first_hop) acc_v[r][j] += acc_g[r][j];
                    else g_out[bh * per_head + (base + (long long)key * a.stride) * D + c] = from_f32<T>(acc_g[r][j]);
                }
            }
        }

        // ---- dK rows (rotated back if the hop rotates), dV rows
        __syncthreads();
#pragma unroll
        for (int r = 0; r < kPerWarp; ++r) {
            const int row = warp * kPerWarp + r;
#pragma unroll
            for (int j = 0; j < DPL; ++j) {
                const int c = lane + 32 * j;
                if (c < D) sK[row * D + c] = acc_k[r][j];
            }
        }
        __syncthreads();
        if (a.rope_log2_base != 0.f) {
            rope_rows(sK, BR, D, D, u0, a.rope_log2_base, -1.f);
            __syncthreads();
        }
        for (int idx = threadIdx.x; idx < BR * D; idx += kThreads) {
            const int r = idx / D, c = idx % D, key = u0 + r;
            if (key >= a.n) continue;
            float *dst = dk_acc + kvh * per_head + (base + (long long)key * a.stride) * D + c;
            *dst = a.accumulate ? *dst + sK[idx] : sK[idx];
        }
        if (a.first_hop) {
#pragma unroll
            for (int r = 0; r < kPerWarp; ++r) {
                const int key = u0 + warp * kPerWarp + r;
                if (key >= a.n) continue;
#pragma unroll
                for (int j = 0; j < DPL; ++j) {
                    const int c = lane + 32 * j;
                    if (c < D) dv_acc[kvh * per_head + (base + (long long)key * a.stride) * D + c] = acc_v[r][j];
                }
            }
        }
    }
}

template <typename T, int DPL>
int launch_dpl(const Problem &pb, const HopDesc &hd, const void *x, int x_heads, const void *g_in, void *g_out,
               float *dq_acc, float *dk_acc, float *dv_acc, float2 *stats, bool first_hop, bool accumulate) {
    SimtBwdArgs a;
    a.N = pb.N; a.D = pb.D; a.n = hd.n; a.H = pb.H; a.H_kv = pb.H_kv; a.x_heads = x_heads; a.causal = pb.causal;
    a.stride = hd.stride;
    a.segs_per_head = hd.outer * hd.stride;
    a.rblocks = (hd.n + BR - 1) / BR;
    a.scale = pb.scale;
    a.rope_log2_base = pb.rope_base > 0.f ? log2f(pb.rope_base) : 0.f;
    a.window = pb.window[hd.hop];
    a.masked = 0;
    a.lens = pb.seq_lens;
    a.first_hop = first_hop ? 1 : 0;
    a.accumulate = accumulate ? 1 : 0;
    a.dmask = nullptr;
    a.dmask_words = 0;
    HopMask hm;
    memset(&hm, 0, sizeof(hm));
    a.dmask_heads = 1;
    if (pb.masks[hd.hop] && (hd.n > 128 || pb.masks_per_head)) {
        if (!pb.dmask[hd.hop]) return TA_ERR_INVALID_ARG;
        a.masked = 2;
        a.dmask = pb.dmask[hd.hop];
        a.dmask_words = pb.dmask_words[hd.hop];
        a.dmask_heads = pb.masks_per_head ? pb.H : 1;
    } else if (pb.masks[hd.hop]) {
        const int rc = build_hop_mask(pb, hd, &hm);
        if (rc != TA_OK) return rc;
        a.masked = 1;
    }
    const size_t smem = sizeof(float) * (2 * (size_t)BR * pb.D + 2 * (size_t)BL * (pb.D + 1));
    auto kq = hop_simt_bwd_q_kernel<T, DPL>;
    auto kk = hop_simt_bwd_k_kernel<T, DPL>;
    if (smem > 48 * 1024) {
        if (cudaFuncSetAttribute(kq, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
            cudaFuncSetAttribute(kk, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return cuda_fail(cudaPeekAtLastError());
    }
    const T *q = (const T *)pb.q, *k = (const T *)pb.k;
    a.items = (long long)pb.B * pb.H * a.segs_per_head * a.rblocks;
    long long grid = a.items < (1ll << 20) ? a.items : (1ll << 20);
    int rc = launch_kernel(kq, (unsigned)grid, kThreads, smem, pb.stream, false, q, k, (const T *)x,
                           (const T *)g_in, dq_acc, stats, a, hm);
    if (rc != TA_OK) return rc;
    a.items = (long long)pb.B * pb.H_kv * a.segs_per_head * a.rblocks;
    grid = a.items < (1ll << 20) ? a.items : (1ll << 20);
    return launch_kernel(kk, (unsigned)grid, kThreads, smem, pb.stream, false, q, k, (const T *)x,
                         (const T *)g_in, (const float2 *)stats, (T *)g_out, dk_acc, dv_acc, a, hm);
}

}  // namespace

int launch_hop_simt_bwd(const Problem &pb, const HopDesc &hd, const void *x, int x_heads, const void *g_in,
                        void *g_out, float *dq_acc, float *dk_acc, float *dv_acc, void *stats, bool first_hop,
                        bool accumulate) {
    if (!first_hop && (g_out == nullptr || g_out == g_in)) return TA_ERR_INVALID_ARG;   // the key side reads all of g_in
    float2 *st = (float2 *)stats;
#define TA_BWD_DISPATCH(T)                                                                                              \
    do {                                                                                                                \
        if (pb.D <= 32) return launch_dpl<T, 1>(pb, hd, x, x_heads, g_in, g_out, dq_acc, dk_acc, dv_acc, st, first_hop, accumulate);  \
        if (pb.D <= 64) return launch_dpl<T, 2>(pb, hd, x, x_heads, g_in, g_out, dq_acc, dk_acc, dv_acc, st, first_hop, accumulate);  \
        if (pb.D <= 128) return launch_dpl<T, 4>(pb, hd, x, x_heads, g_in, g_out, dq_acc, dk_acc, dv_acc, st, first_hop, accumulate); \
        if (pb.D <= 256) return launch_dpl<T, 8>(pb, hd, x, x_heads, g_in, g_out, dq_acc, dk_acc, dv_acc, st, first_hop, accumulate); \
    } while (0)
    if (pb.dtype == TA_DTYPE_F32) TA_BWD_DISPATCH(float);
    else if (pb.dtype == TA_DTYPE_BF16) TA_BWD_DISPATCH(__nv_bfloat16);
#undef TA_BWD_DISPATCH
    return TA_ERR_UNSUPPORTED;
}

}  // namespace ta
