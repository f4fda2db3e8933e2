/*
 * Tensorized-attention CPU oracle (fp64).  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, step-by-step implementation of the paper's Algorithm 1
 * ("Tensorized attention forward") for ONE attention head, plus the reverse-mode
 * derivative of exactly that recurrence.  Nothing here is blocked, fused or
 * reordered beyond what the algorithm states; the only parallelism is an OpenMP
 * loop over the independent mode-i vectors ("segments") of one hop.
 *
 * This file shares no code with the CUDA path and is never called by it.
 *
 * Notation (Section 3.1 / 3.2 of the paper): the N tokens of a head are viewed,
 * by row-major reshape, as a tensor n_1 x ... x n_m (dims[0] = n_1 is the
 * slowest-varying coordinate).  Mode-i flattening (Eq. 4) batches the
 * N / n_i vectors obtained by fixing every coordinate except the i-th; the
 * tokens of one such vector are base + t * s_i, t = 0..n_i-1, with
 * s_i = prod_{l>i} n_l.
 *
 * Forward (Algorithm 1):
 *     O = V
 *     for i = 0 .. m-1:                      (first dimension first)
 *         A_i = softmax(Q_i K_i^T * scale  o  M_i)       (Eq. 4, row-wise softmax)
 *         O_i = A_i O_i                                   (value update)
 *     return vec(O)
 * Q and K are the same un-updated projections in every hop; only O is carried.
 * The mask M_i removes entries from the softmax (their weight is exactly 0);
 * the causal M_i keeps key position u <= query position t along mode i.
 *
 * Tensorized positional encoding (Section 3.2, "Tensorized Positional Encoding"): the
 * position of a token is the vector of its coordinates (j_1..j_m) and, following Llama,
 * RoPE encodes it.  The paper gives no formula (its appendix on this is not in the text);
 * the reading implemented here, when rope_base > 0: in hop i the queries and keys are
 * rotated by the token's coordinate j_i along the dimension the hop attends over, with
 * the Llama pairing of feature c with c + D/2 and angle j_i * rope_base^(-2c/D),
 *     x'_c       = x_c cos a - x_{c+D/2} sin a
 *     x'_{c+D/2} = x_{c+D/2} cos a + x_c sin a ,       c = 0 .. D/2-1,
 * so that a hop's scores depend on the relative position t - u along that dimension.
 * The value tensor is never rotated.
 *
 * Per-hop sparsity masks (the paper notes that M_i may be any sparsity mask, Section 3.1 /
 * Eq. 3): besides the causal mask, hop i may carry a sliding window w_i > 0 along its
 * dimension -- key position u is visible from query position t iff |t - u| < w_i (and u <= t
 * when causal).  w_i = 0 means no window.  Every row keeps its own position, so no row is
 * fully masked.  Hop i may also carry an explicit n_i x n_i mask (row = query position, column
 * = key position, non-zero = visible), applied on top of the causal flag and the window; a row
 * left without any visible key is an error.
 *
 * Valid length (padding; M_i of Eq. 3 may depend on the segment): with len < N only the tokens
 * with flat index < len exist.  A padding token is never visible as a key; a padding query has
 * an all-zero row of weights, so its output row is 0 and nothing flows back through it (its rows
 * of dq, dk, dv are 0 and its row of dout is ignored).  len = N means no padding.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* Attention weights of one segment: P[t*n+u], rows sum to 1 (Eq. 1 / Eq. 4). */
/* Is key position u visible from query position t in this hop? */
static int visible(int t, int u, int causal, int window, const unsigned char *mask, int n)
{
    if (causal && u > t) return 0;
    if (window > 0 && (t - u >= window || u - t >= window)) return 0;
    if (mask && !mask[(long)t * n + u]) return 0;
    return 1;
}

/* Attention weights of one segment: P[t*n+u], rows sum to 1 (Eq. 1 / Eq. 4); entries the mask
 * removes have weight exactly 0.  Returns -1 if a row has no visible key. */
static int segment_weights(const double *Q, const double *K, long base, long stride,
                           int n, int D, double scale, int causal, int window,
                           const unsigned char *mask, long len, double *P)
{
    for (int t = 0; t < n; ++t) {
        const double *qt = Q + (base + (long)t * stride) * D;
        double mx = -INFINITY;
        int any = 0;
        if (base + (long)t * stride >= len) {               /* padding query: no weights at all */
            for (int u = 0; u < n; ++u) P[t * n + u] = 0.0;
            continue;
        }
        for (int u = 0; u < n; ++u) {
            if (base + (long)u * stride >= len ||           /* padding key */
                !visible(t, u, causal, window, mask, n)) { P[t * n + u] = 0.0; continue; }
            const double *ku = K + (base + (long)u * stride) * D;
            double s = 0.0;
            for (int c = 0; c < D; ++c) s += qt[c] * ku[c];
            s *= scale;
            P[t * n + u] = s;
            if (s > mx) mx = s;
            any = 1;
        }
        if (!any) return -1;
        double den = 0.0;
        for (int u = 0; u < n; ++u) {
            if (base + (long)u * stride >= len || !visible(t, u, causal, window, mask, n)) continue;
            double e = exp(P[t * n + u] - mx);
            P[t * n + u] = e;
            den += e;
        }
        for (int u = 0; u < n; ++u) P[t * n + u] /= den;   /* masked entries stay 0 */
    }
    return 0;
}

/* stride s_i and the enumeration of segments of hop i:
 * segment index g in [0, N/n_i) -> (outer, inner) -> base token outer*n_i*s_i + inner */
static long hop_stride(const int *dims, int ndims, int i)
{
    long s = 1;
    for (int l = i + 1; l < ndims; ++l) s *= dims[l];
    return s;
}

/* y[j] = R(p_j) x[j] with p_j = (j / stride) mod n, the coordinate of token j along the hop's
 * dimension; sign = +1 rotates, -1 applies the transpose (inverse) rotation. */
static void rope_rotate(const double *x, double *y, long N, int D, long stride, int n,
                        double base, int sign)
{
    const int half = D / 2;
    for (long j = 0; j < N; ++j) {
        const double p = (double)((j / stride) % n);
        for (int c = 0; c < half; ++c) {
            const double a = sign * p * pow(base, -2.0 * c / D);
            const double cs = cos(a), sn = sin(a);
            const double x1 = x[j * D + c], x2 = x[j * D + c + half];
            y[j * D + c] = x1 * cs - x2 * sn;
            y[j * D + c + half] = x2 * cs + x1 * sn;
        }
        if (D & 1) y[j * D + D - 1] = x[j * D + D - 1];
    }
}

/*
 * One head, forward.  q,k,v: [N][D] fp64 (k,v are the head's KV head).
 * out: [N][D].  xs (optional, may be NULL): [(ndims+1)][N][D], receives
 * X_0 = V, X_1, ..., X_m = out (the value tensor after each hop), which the
 * backward pass below needs.
 * Returns 0, or -1 on bad arguments / allocation failure.
 */
static int forward_head_impl(const double *q, const double *k, const double *v, double *out,
                             long N, int D, const int *dims, int ndims, int causal,
                             double scale, double rope_base, const int *window,
                             const unsigned char *const *masks, long len, double *xs)
{
    if (!q || !k || !v || !out || !dims || ndims < 1 || N < 1 || D < 1) return -1;
    if (len < 0 || len > N) return -1;
    long prod = 1;
    for (int i = 0; i < ndims; ++i) { if (dims[i] < 1) return -1; prod *= dims[i]; }
    if (prod != N) return -1;

    size_t bytes = (size_t)N * D * sizeof(double);
    double *cur = (double *)malloc(bytes), *nxt = (double *)malloc(bytes);
    double *qr = NULL, *kr = NULL;                          /* rotated q, k of the current hop */
    if (rope_base > 0.0) { qr = (double *)malloc(bytes); kr = (double *)malloc(bytes); }
    if (!cur || !nxt || (rope_base > 0.0 && (!qr || !kr))) {
        free(cur); free(nxt); free(qr); free(kr);
        return -1;
    }
    memcpy(cur, v, bytes);                                  /* Initialize O = V */
    if (xs) memcpy(xs, v, bytes);

    int fail = 0;
    const double *q_in = q, *k_in = k;
    for (int i = 0; i < ndims; ++i) {                       /* for i = 0 to m-1 */
        const int n = dims[i];
        const long s = hop_stride(dims, ndims, i);
        const long nseg = N / n;
        if (rope_base > 0.0) {                              /* positions along dimension i */
            rope_rotate(q_in, qr, N, D, s, n, rope_base, +1);
            rope_rotate(k_in, kr, N, D, s, n, rope_base, +1);
            q = qr; k = kr;
        }
        #pragma omp parallel
        {
            double *P = (double *)malloc((size_t)n * n * sizeof(double));
            if (!P) {
                #pragma omp atomic write
                fail = 1;
            }
            #pragma omp for schedule(static)
            for (long g = 0; g < nseg; ++g) {
                if (!P) continue;
                long outer = g / s, inner = g % s;
                long base = outer * n * s + inner;
                if (segment_weights(q, k, base, s, n, D, scale, causal, window ? window[i] : 0,
                                    masks ? masks[i] : NULL, len, P) != 0) {            /* A_i */
                    #pragma omp atomic write
                    fail = 1;
                    continue;
                }
                for (int t = 0; t < n; ++t) {               /* O_i = A_i O_i, folded back */
                    double *o = nxt + (base + (long)t * s) * D;
                    for (int c = 0; c < D; ++c) o[c] = 0.0;
                    for (int u = 0; u < n; ++u) {
                        double p = P[t * n + u];
                        if (p == 0.0) continue;
                        const double *x = cur + (base + (long)u * s) * D;
                        for (int c = 0; c < D; ++c) o[c] += p * x[c];
                    }
                }
            }
            free(P);
        }
        if (fail) break;
        double *tmp = cur; cur = nxt; nxt = tmp;
        if (xs) memcpy(xs + (size_t)(i + 1) * N * D, cur, bytes);
    }
    if (!fail) memcpy(out, cur, bytes);
    free(cur); free(nxt); free(qr); free(kr);
    return fail ? -1 : 0;
}

int ta_oracle_forward_head(const double *q, const double *k, const double *v, double *out,
                           long N, int D, const int *dims, int ndims, int causal,
                           double scale, double *xs)
{
    return forward_head_impl(q, k, v, out, N, D, dims, ndims, causal, scale, 0.0, NULL, NULL, N, xs);
}

/* As above with the tensorized positional encoding (rope_base > 0, e.g. 10000). */
int ta_oracle_forward_head_rope(const double *q, const double *k, const double *v, double *out,
                                long N, int D, const int *dims, int ndims, int causal,
                                double scale, double rope_base, double *xs)
{
    if (!(rope_base > 0.0)) return -1;
    return forward_head_impl(q, k, v, out, N, D, dims, ndims, causal, scale, rope_base, NULL, NULL, N, xs);
}

/* Every option: rope_base 0 = none; window NULL or [ndims] ints, 0 = no window in that hop;
 * masks NULL or [ndims] pointers, each NULL or an n_i x n_i byte matrix (non-zero = visible). */
int ta_oracle_forward_head_ex(const double *q, const double *k, const double *v, double *out,
                              long N, int D, const int *dims, int ndims, int causal,
                              double scale, double rope_base, const int *window,
                              const unsigned char *const *masks, double *xs)
{
    if (rope_base < 0.0) return -1;
    if (window) for (int i = 0; i < ndims; ++i) if (window[i] < 0) return -1;
    return forward_head_impl(q, k, v, out, N, D, dims, ndims, causal, scale, rope_base, window, masks, N, xs);
}

/* As ta_oracle_forward_head_ex with a valid length: tokens with flat index >= len are padding. */
int ta_oracle_forward_head_len(const double *q, const double *k, const double *v, double *out,
                               long N, int D, const int *dims, int ndims, int causal,
                               double scale, double rope_base, const int *window,
                               const unsigned char *const *masks, long len, double *xs)
{
    if (rope_base < 0.0) return -1;
    if (window) for (int i = 0; i < ndims; ++i) if (window[i] < 0) return -1;
    return forward_head_impl(q, k, v, out, N, D, dims, ndims, causal, scale, rope_base, window, masks, len, xs);
}

/*
 * One head, backward of the recurrence above (the paper gives no formula for it;
 * this is the chain rule applied hop by hop, in reverse hop order).
 * With X_0 = V, X_{i+1} = A_i X_i per segment, out = X_m and G_m = dout:
 *     G_i  = A_i^T G_{i+1}                       gradient w.r.t. the hop's input
 *     dP   = G_{i+1} X_i^T
 *     dS   = A_i o (dP - rowsum(A_i o dP))       softmax derivative, masked entries 0
 *     dQ  += scale * dS K        dK += scale * dS^T Q        (summed over hops)
 *     dV   = G_0
 * xs: [(ndims+1)][N][D] as written by ta_oracle_forward_head.
 * dq, dk, dv: [N][D], overwritten (the caller sums dk, dv over a GQA group).
 * With rope_base > 0 each hop works on its rotated queries and keys q' = R q, k' = R k and
 * the gradients it finds for them are rotated back (dq += R^T dq') before they are summed.
 */
static int backward_head_impl(const double *q, const double *k, const double *xs,
                              const double *dout, double *dq, double *dk, double *dv,
                              long N, int D, const int *dims, int ndims, int causal,
                              double scale, double rope_base, const int *window,
                              const unsigned char *const *masks, long len)
{
    if (!q || !k || !xs || !dout || !dq || !dk || !dv || !dims || ndims < 1) return -1;
    if (len < 0 || len > N) return -1;
    long prod = 1;
    for (int i = 0; i < ndims; ++i) { if (dims[i] < 1) return -1; prod *= dims[i]; }
    if (prod != N) return -1;

    size_t bytes = (size_t)N * D * sizeof(double);
    double *g = (double *)malloc(bytes), *gn = (double *)malloc(bytes);
    double *qr = NULL, *kr = NULL, *dqr = NULL, *dkr = NULL, *tmp_rot = NULL;
    const int rope = rope_base > 0.0;
    if (rope) {
        qr = (double *)malloc(bytes); kr = (double *)malloc(bytes);
        dqr = (double *)malloc(bytes); dkr = (double *)malloc(bytes);
        tmp_rot = (double *)malloc(bytes);
    }
    if (!g || !gn || (rope && (!qr || !kr || !dqr || !dkr || !tmp_rot))) {
        free(g); free(gn); free(qr); free(kr); free(dqr); free(dkr); free(tmp_rot);
        return -1;
    }
    memcpy(g, dout, bytes);
    memset(dq, 0, bytes);
    memset(dk, 0, bytes);

    int fail = 0;
    const double *q_in = q, *k_in = k;
    double *dq_out = dq, *dk_out = dk;
    for (int i = ndims - 1; i >= 0; --i) {
        const int n = dims[i];
        const long s = hop_stride(dims, ndims, i);
        const long nseg = N / n;
        const double *x = xs + (size_t)i * N * D;           /* X_i: the hop's input */
        if (rope) {
            rope_rotate(q_in, qr, N, D, s, n, rope_base, +1);
            rope_rotate(k_in, kr, N, D, s, n, rope_base, +1);
            q = qr; k = kr;
            memset(dqr, 0, bytes); memset(dkr, 0, bytes);
            dq = dqr; dk = dkr;                             /* this hop's dq', dk' */
        }
        #pragma omp parallel
        {
            double *P = (double *)malloc((size_t)n * n * sizeof(double));
            double *dS = (double *)malloc((size_t)n * n * sizeof(double));
            if (!P || !dS) {
                #pragma omp atomic write
                fail = 1;
            }
            #pragma omp for schedule(static)
            for (long sg = 0; sg < nseg; ++sg) {
                if (!P || !dS) continue;
                long outer = sg / s, inner = sg % s;
                long base = outer * n * s + inner;
                if (segment_weights(q, k, base, s, n, D, scale, causal, window ? window[i] : 0,
                                    masks ? masks[i] : NULL, len, P) != 0) {
                    #pragma omp atomic write
                    fail = 1;
                    continue;
                }
                /* dP[t][u] = <G_{i+1}[t], X_i[u]>, then dS */
                for (int t = 0; t < n; ++t) {
                    const double *gt = g + (base + (long)t * s) * D;
                    double dot = 0.0;
                    for (int u = 0; u < n; ++u) {
                        const double *xu = x + (base + (long)u * s) * D;
                        double a = 0.0;
                        for (int c = 0; c < D; ++c) a += gt[c] * xu[c];
                        dS[t * n + u] = a;
                        if (P[t * n + u] != 0.0) dot += P[t * n + u] * a;
                    }
                    for (int u = 0; u < n; ++u)        /* weight 0 (masked, padding): exactly 0 */
                        dS[t * n + u] = P[t * n + u] != 0.0 ? P[t * n + u] * (dS[t * n + u] - dot) : 0.0;
                }
                /* G_i = P^T G_{i+1};  dQ += scale dS K;  dK += scale dS^T Q
                 * (segments are disjoint token sets, so no two threads touch the same row) */
                for (int u = 0; u < n; ++u) {
                    double *go = gn + (base + (long)u * s) * D;
                    double *dku = dk + (base + (long)u * s) * D;
                    for (int c = 0; c < D; ++c) go[c] = 0.0;
                    for (int t = 0; t < n; ++t) {
                        const double *gt = g + (base + (long)t * s) * D;
                        const double *qt = q + (base + (long)t * s) * D;
                        double p = P[t * n + u], ds = scale * dS[t * n + u];
                        if (p == 0.0) continue;             /* then ds = 0 too: nothing flows */
                        for (int c = 0; c < D; ++c) { go[c] += p * gt[c]; dku[c] += ds * qt[c]; }
                    }
                }
                for (int t = 0; t < n; ++t) {
                    double *dqt = dq + (base + (long)t * s) * D;
                    for (int u = 0; u < n; ++u) {
                        const double *ku = k + (base + (long)u * s) * D;
                        double ds = scale * dS[t * n + u];
                        if (P[t * n + u] == 0.0) continue;
                        for (int c = 0; c < D; ++c) dqt[c] += ds * ku[c];
                    }
                }
            }
            free(P); free(dS);
        }
        if (fail) break;
        if (rope) {                                         /* dq += R^T dq', dk += R^T dk' */
            rope_rotate(dqr, tmp_rot, N, D, s, n, rope_base, -1);
            for (long e = 0; e < N * D; ++e) dq_out[e] += tmp_rot[e];
            rope_rotate(dkr, tmp_rot, N, D, s, n, rope_base, -1);
            for (long e = 0; e < N * D; ++e) dk_out[e] += tmp_rot[e];
        }
        double *tmp = g; g = gn; gn = tmp;
    }
    if (!fail) memcpy(dv, g, bytes);
    free(g); free(gn); free(qr); free(kr); free(dqr); free(dkr); free(tmp_rot);
    return fail ? -1 : 0;
}

int ta_oracle_backward_head(const double *q, const double *k, const double *xs,
                            const double *dout, double *dq, double *dk, double *dv,
                            long N, int D, const int *dims, int ndims, int causal,
                            double scale)
{
    return backward_head_impl(q, k, xs, dout, dq, dk, dv, N, D, dims, ndims, causal, scale, 0.0, NULL, NULL, N);
}

int ta_oracle_backward_head_rope(const double *q, const double *k, const double *xs,
                                 const double *dout, double *dq, double *dk, double *dv,
                                 long N, int D, const int *dims, int ndims, int causal,
                                 double scale, double rope_base)
{
    if (!(rope_base > 0.0)) return -1;
    return backward_head_impl(q, k, xs, dout, dq, dk, dv, N, D, dims, ndims, causal, scale,
                              rope_base, NULL, NULL, N);
}

int ta_oracle_backward_head_ex(const double *q, const double *k, const double *xs,
                               const double *dout, double *dq, double *dk, double *dv,
                               long N, int D, const int *dims, int ndims, int causal,
                               double scale, double rope_base, const int *window,
                               const unsigned char *const *masks)
{
    if (rope_base < 0.0) return -1;
    return backward_head_impl(q, k, xs, dout, dq, dk, dv, N, D, dims, ndims, causal, scale,
                              rope_base, window, masks, N);
}

/* As ta_oracle_backward_head_ex with a valid length (xs from ta_oracle_forward_head_len). */
int ta_oracle_backward_head_len(const double *q, const double *k, const double *xs,
                                const double *dout, double *dq, double *dk, double *dv,
                                long N, int D, const int *dims, int ndims, int causal,
                                double scale, double rope_base, const int *window,
                                const unsigned char *const *masks, long len)
{
    if (rope_base < 0.0) return -1;
    return backward_head_impl(q, k, xs, dout, dq, dk, dv, N, D, dims, ndims, causal, scale,
                              rope_base, window, masks, len);
}

int ta_oracle_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
    #pragma omp parallel
    {
        #pragma omp master
        n = omp_get_num_threads();
    }
#endif
    return n;
}
