/*
 * Bounded-cache attention oracle: TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, double-precision CPU statement of what one Bounded-Cache
 * Transformer attention layer computes per token and per (sequence, kv-head)
 * unit.  It shares no code with the CUDA library and is only ever called from
 * the tests, the smoke check and the CPU-baseline leg of the benchmark.
 *
 * Notation follows the paper's Method section:
 *   M   (here C, "capacity")  number of cache slots
 *   MK  [C][d]                key vector sequence; never assigned by Algorithm 1
 *   MV  [C][d]                key-value vector sequence; the state the rule rewrites
 *   wq_t (here k_t)           write query of token t
 *   wv_t (here v_t)           write key-value vector of token t
 *   score_t = wq_t . MK^T     (Algorithm 1, the score statement)
 *   ww_t    = softmax(score_t) (Algorithm 1, the softmax statement)
 *   MV_t    = MV_{t-1} + ww_t^T . wv_t   (Method step 4; Illustration step 3)
 *
 * The paper does not print the read path; the layer is an attention layer
 * (Method, "Model Structure"), so the read is ordinary softmax attention of the
 * token's G read queries over the resident (MK, MV).
 *
 * Readings taken where the paper is silent (each is also a switch here):
 *   - no scale factor is printed on score_t: write_scale is an explicit argument
 *     (1.0 = literal); read_scale likewise.
 *   - order inside a token: read MV_{t-1}, then write (default), or write then
 *     read (BCT_ORACLE_WRITE_THEN_READ).
 *   - Algorithm 1's "if t = 1" branch keeps MV_0 for the first token, while the
 *     exception-free formula of Method step 4 updates on every token.  Default:
 *     every token writes.  BCT_ORACLE_SKIP_FIRST_WRITE takes the branch literally.
 *   - step size (Features, "Learning Rate Adaptation": the step size is adjusted
 *     for each token; no formula is printed): eta_t multiplies the token's
 *     increment, MV_t = MV_{t-1} + eta_t * ww_t^T . wv_t.  eta_t = 1 is Method
 *     step 4 as printed.  How eta_t is produced is upstream of this layer: it is
 *     an input.  The fill phase has no soft write and ignores it.
 *   - write threshold (not in the paper; a reading of the library under test): with
 *     write_eps > 0 a slot whose write weight ww_j is below write_eps keeps its row,
 *     i.e. its increment eta_t * ww_j * wv_t is dropped.  write_eps = 0 is the printed
 *     rule, every slot updated.  The weights themselves stay normalised over all slots.
 *   - fill phase (not in the paper, whose MV_0 is full-size): while len < C the
 *     token's (k_t, v_t) is appended at slot len, the read then covers the
 *     len+1 resident slots (so the token sees itself), and no soft write happens.
 *
 * No blocking, fusion or reordering: every loop below is the definition.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define BCT_ORACLE_SKIP_FIRST_WRITE 1u
#define BCT_ORACLE_WRITE_THEN_READ 2u

/* p[j] = exp(s[j] - max s) / sum_j exp(s[j] - max s), j < n  (softmax, Algorithm 1). */
static void softmax(const double *s, int64_t n, double *p) {
    double m = s[0];
    for (int64_t j = 1; j < n; ++j)
        if (s[j] > m) m = s[j];
    double sum = 0.0;
    for (int64_t j = 0; j < n; ++j) {
        p[j] = exp(s[j] - m);
        sum += p[j];
    }
    for (int64_t j = 0; j < n; ++j) p[j] /= sum;
}

/* Read path for one query head: o = softmax(read_scale * q . MK[0:n]^T) . MV[0:n]. */
static void read_head(const double *q, const double *MK, const double *MV, int64_t n, int d,
                      double read_scale, double *s, double *p, double *o) {
    for (int64_t j = 0; j < n; ++j) {
        double dot = 0.0;
        for (int e = 0; e < d; ++e) dot += q[e] * MK[j * d + e];
        s[j] = read_scale * dot;
    }
    softmax(s, n, p);
    for (int e = 0; e < d; ++e) o[e] = 0.0;
    for (int64_t j = 0; j < n; ++j)
        for (int e = 0; e < d; ++e) o[e] += p[j] * MV[j * d + e];
}

/* Write path: score = write_scale * wq . MK^T; ww = softmax(score); MV += eta * ww^T . wv
 * on the slots with ww_j >= write_eps (all of them when write_eps = 0).
 * ww (length C) is left in `ww` for the caller. */
static void write_update(const double *wq, const double *wv, const double *MK, double *MV,
                         int64_t C, int d, double write_scale, double eta, double write_eps,
                         double *s, double *ww) {
    for (int64_t j = 0; j < C; ++j) {
        double dot = 0.0;
        for (int e = 0; e < d; ++e) dot += wq[e] * MK[j * d + e];
        s[j] = write_scale * dot;
    }
    softmax(s, C, ww);
    for (int64_t j = 0; j < C; ++j) {
        if (ww[j] < write_eps) continue;
        for (int e = 0; e < d; ++e) MV[j * d + e] += eta * (ww[j] * wv[e]);
    }
}

/*
 * One token for one unit.  `len` is the number of resident slots before the
 * token; the return value is the number after it.  `do_write` is 0 only for
 * the literal first-token branch of Algorithm 1.  `out` may be NULL
 * (state-only, as UpdateKV returns only MV_N).
 */
static int64_t unit_token(int G, int d, int64_t C, int64_t len, double *MK, double *MV,
                          const double *q, const double *k, const double *v, double *out,
                          double read_scale, double write_scale, double eta, double write_eps,
                          unsigned flags, int do_write, double *s, double *p) {
    if (len < C) { /* fill phase: append, then read over len+1 slots, no soft write */
        memcpy(MK + len * d, k, sizeof(double) * (size_t)d);
        memcpy(MV + len * d, v, sizeof(double) * (size_t)d);
        len += 1;
        if (out)
            for (int g = 0; g < G; ++g)
                read_head(q + (int64_t)g * d, MK, MV, len, d, read_scale, s, p, out + (int64_t)g * d);
        return len;
    }
    if ((flags & BCT_ORACLE_WRITE_THEN_READ) && do_write)
        write_update(k, v, MK, MV, C, d, write_scale, eta, write_eps, s, p);
    if (out)
        for (int g = 0; g < G; ++g)
            read_head(q + (int64_t)g * d, MK, MV, C, d, read_scale, s, p, out + (int64_t)g * d);
    if (!(flags & BCT_ORACLE_WRITE_THEN_READ) && do_write)
        write_update(k, v, MK, MV, C, d, write_scale, eta, write_eps, s, p);
    return len;
}

/*
 * T tokens through U independent units.
 *
 * Layouts (all row-major, double):
 *   MK, MV  [U][C][d]      in/out (MK rows >= len are ignored until filled)
 *   q       [U][T][G][d]
 *   k, v    [U][T][d]
 *   out     [U][T][G][d]   or NULL
 *   eta     [U][T]         step size of each token's write, or NULL (all ones)
 * len_io        resident slots, the same for every unit (in/out)
 * n_written_io  soft writes applied so far per unit history (in/out); only its
 *               being zero matters (BCT_ORACLE_SKIP_FIRST_WRITE)
 * write_eps     slots whose write weight is below it are not rewritten (0: the printed rule)
 * nthreads      OpenMP threads over units (<= 0: library default)
 * Returns the number of threads used, or -1 on bad arguments / allocation failure.
 */
int bct_oracle_stream_eps(int64_t U, int64_t T, int G, int d, int64_t C, int64_t *len_io,
                          int64_t *n_written_io, double *MK, double *MV, const double *q,
                          const double *k, const double *v, const double *eta, double *out,
                          double read_scale, double write_scale, double write_eps, unsigned flags,
                          int nthreads) {
    if (U < 0 || T < 0 || G < 1 || d < 1 || C < 1 || !len_io || !n_written_io) return -1;
    if (*len_io < 0 || *len_io > C) return -1;
    int used = 1;
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
    used = omp_get_max_threads();
    if (used > U && U > 0) used = (int)U;
#endif
    int failed = 0;
    const int64_t len0 = *len_io;
    const int64_t w0 = *n_written_io;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1)
#endif
    for (int64_t u = 0; u < U; ++u) {
        double *s = (double *)malloc(sizeof(double) * (size_t)C);
        double *p = (double *)malloc(sizeof(double) * (size_t)C);
        if (!s || !p) {
            failed = 1;
        } else {
            int64_t len = len0, nw = w0;
            double *mk = MK + u * C * d, *mv = MV + u * C * d;
            for (int64_t t = 0; t < T; ++t) {
                const double *qt = q + ((u * T + t) * G) * d;
                const double *kt = k + (u * T + t) * d;
                const double *vt = v + (u * T + t) * d;
                double *ot = out ? out + ((u * T + t) * G) * d : NULL;
                int full = (len == C);
                int do_write = !((flags & BCT_ORACLE_SKIP_FIRST_WRITE) && nw == 0);
                len = unit_token(G, d, C, len, mk, mv, qt, kt, vt, ot, read_scale, write_scale,
                                 eta ? eta[u * T + t] : 1.0, write_eps, flags, do_write, s, p);
                if (full) nw += 1; /* counts full-phase tokens seen, written or skipped */
            }
        }
        free(s);
        free(p);
    }
    if (failed) return -1;
    /* every unit advances identically */
    int64_t len = len0, nw = w0;
    for (int64_t t = 0; t < T; ++t) {
        if (len < C) len += 1; else nw += 1;
    }
    *len_io = len;
    *n_written_io = nw;
    return used;
}

/* The same without a write threshold: every slot is updated. */
int bct_oracle_stream_eta(int64_t U, int64_t T, int G, int d, int64_t C, int64_t *len_io,
                          int64_t *n_written_io, double *MK, double *MV, const double *q,
                          const double *k, const double *v, const double *eta, double *out,
                          double read_scale, double write_scale, unsigned flags, int nthreads) {
    return bct_oracle_stream_eps(U, T, G, d, C, len_io, n_written_io, MK, MV, q, k, v, eta, out,
                                 read_scale, write_scale, 0.0, flags, nthreads);
}

/* The same with every step size equal to one: Method step 4 as printed. */
int bct_oracle_stream(int64_t U, int64_t T, int G, int d, int64_t C, int64_t *len_io,
                      int64_t *n_written_io, double *MK, double *MV, const double *q,
                      const double *k, const double *v, double *out, double read_scale,
                      double write_scale, unsigned flags, int nthreads) {
    return bct_oracle_stream_eta(U, T, G, d, C, len_io, n_written_io, MK, MV, q, k, v, NULL, out,
                                 read_scale, write_scale, flags, nthreads);
}

/* The write weights ww = softmax(write_scale * wq . MK^T) of one unit, for tests
 * of the row-sum and hard-addressing properties.  MK [C][d], wq [d], ww [C]. */
int bct_oracle_write_weights(int64_t C, int d, const double *MK, const double *wq,
                             double write_scale, double *ww) {
    if (C < 1 || d < 1) return -1;
    double *s = (double *)malloc(sizeof(double) * (size_t)C);
    if (!s) return -1;
    for (int64_t j = 0; j < C; ++j) {
        double dot = 0.0;
        for (int e = 0; e < d; ++e) dot += wq[e] * MK[j * d + e];
        s[j] = write_scale * dot;
    }
    softmax(s, C, ww);
    free(s);
    return 0;
}

/* The read weights p = softmax(read_scale * q . MK[0:n]^T) of one head. */
int bct_oracle_read_weights(int64_t n, int d, const double *MK, const double *q,
                            double read_scale, double *p) {
    if (n < 1 || d < 1) return -1;
    double *s = (double *)malloc(sizeof(double) * (size_t)n);
    if (!s) return -1;
    for (int64_t j = 0; j < n; ++j) {
        double dot = 0.0;
        for (int e = 0; e < d; ++e) dot += q[e] * MK[j * d + e];
        s[j] = read_scale * dot;
    }
    softmax(s, n, p);
    free(s);
    return 0;
}

/*
 * The projections in front of the layer (Algorithm 1, first two statements of the loop body:
 * wq_t = W_wq x_t, wv_t = W_wv x_t; the read query of the attention layer is projected the
 * same way):
 *     y[m][n] = sum_k x[m][k] * W[n][k]
 * x [M][K] one row per token, W [N][K] one row per output feature, y [M][N].
 * Returns the number of threads used, or -1 on bad arguments.
 */
int bct_oracle_project(int64_t M, int64_t K, int64_t N, const double *x, const double *W, double *y,
                       int nthreads) {
    if (M < 0 || K < 1 || N < 1 || !x || !W || !y) return -1;
    int used = 1;
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
    used = omp_get_max_threads();
#pragma omp parallel for schedule(static)
#endif
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int64_t k = 0; k < K; ++k) acc += x[m * K + k] * W[n * K + k];
            y[m * N + n] = acc;
        }
    return used;
}

/*
 * Backward of Algorithm 1's procedure UpdateKV in its token-parallel form (Key
 * Implementation Aspects, "Optimized for Parallelism": MK is never assigned, so every
 * ww_t depends on MK and wq_t alone and the final state is a plain sum over the tokens):
 *
 *     MV_N = MV_0 + sum_t eta_t * ww_t^T . wv_t,   ww_t = softmax(write_scale * wq_t . MK^T)
 *
 * Given G = dL/dMV_N for a scalar L, the chain rule through that sum and through the
 * softmax, token by token (nothing is blocked or reordered):
 *     r_t      = sum_j ww_tj * G_j                        (what the token's write sees of G)
 *     dwv_t    = eta_t * r_t
 *     deta_t   = <wv_t, r_t>
 *     dww_tj   = eta_t * <wv_t, G_j>
 *     ds_tj    = ww_tj * (dww_tj - sum_k ww_tk dww_tk)    (softmax Jacobian; the sum is eta_t * deta_t)
 *     dwq_t    = write_scale * sum_j ds_tj * MK_j
 *     dMK_j   += write_scale * ds_tj * wq_t               (summed over the tokens)
 *     dL/dMV_0 = G                                        (the state enters the sum as it is)
 * With a write threshold (write_eps > 0) the forward drops the slots with ww_tj < write_eps;
 * the mask is piecewise constant, so it multiplies ww_tj in r_t and dww_tj and nothing else.
 *
 * Layouts (row-major, double): MK [U][C][d] (full cache), wq, wv [U][T][d], eta [U][T] or NULL
 * (ones), G [U][C][d]; outputs dwq, dwv [U][T][d], dMK [U][C][d], deta [U][T] (any may be NULL).
 * Returns the number of threads used, or -1 on bad arguments / allocation failure.
 */
int bct_oracle_update_kv_backward(int64_t U, int64_t T, int d, int64_t C, const double *MK,
                                  const double *wq, const double *wv, const double *eta,
                                  const double *G, double write_scale, double write_eps,
                                  double *dwq, double *dwv, double *dMK, double *deta,
                                  int nthreads) {
    if (U < 0 || T < 0 || d < 1 || C < 1 || !MK || !wq || !wv || !G) return -1;
    int used = 1;
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
    used = omp_get_max_threads();
    if (used > U && U > 0) used = (int)U;
#endif
    int failed = 0;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1)
#endif
    for (int64_t u = 0; u < U; ++u) {
        double *s = (double *)malloc(sizeof(double) * (size_t)C);
        double *ww = (double *)malloc(sizeof(double) * (size_t)C);
        double *r = (double *)malloc(sizeof(double) * (size_t)d);
        if (!s || !ww || !r) {
            failed = 1;
        } else {
            const double *mk = MK + u * C * d, *g = G + u * C * d;
            if (dMK)
                for (int64_t i = 0; i < C * d; ++i) dMK[u * C * d + i] = 0.0;
            for (int64_t t = 0; t < T; ++t) {
                const double *qt = wq + (u * T + t) * d, *vt = wv + (u * T + t) * d;
                const double et = eta ? eta[u * T + t] : 1.0;
                for (int64_t j = 0; j < C; ++j) {
                    double dot = 0.0;
                    for (int e = 0; e < d; ++e) dot += qt[e] * mk[j * d + e];
                    s[j] = write_scale * dot;
                }
                softmax(s, C, ww);
                for (int e = 0; e < d; ++e) r[e] = 0.0;
                for (int64_t j = 0; j < C; ++j) {
                    if (ww[j] < write_eps) continue;
                    for (int e = 0; e < d; ++e) r[e] += ww[j] * g[j * d + e];
                }
                double de = 0.0;
                for (int e = 0; e < d; ++e) de += vt[e] * r[e];
                if (dwv)
                    for (int e = 0; e < d; ++e) dwv[(u * T + t) * d + e] = et * r[e];
                if (deta) deta[u * T + t] = de;
                if (dwq)
                    for (int e = 0; e < d; ++e) dwq[(u * T + t) * d + e] = 0.0;
                for (int64_t j = 0; j < C; ++j) {
                    double dww = 0.0;
                    if (ww[j] >= write_eps) {
                        for (int e = 0; e < d; ++e) dww += vt[e] * g[j * d + e];
                        dww *= et;
                    }
                    const double ds = ww[j] * (dww - et * de);
                    if (dwq)
                        for (int e = 0; e < d; ++e) dwq[(u * T + t) * d + e] += write_scale * ds * mk[j * d + e];
                    if (dMK)
                        for (int e = 0; e < d; ++e) dMK[(u * C + j) * d + e] += write_scale * ds * qt[e];
                }
            }
        }
        free(s);
        free(ww);
        free(r);
    }
    return failed ? -1 : used;
}
