/*
 * lot_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, float64 CPU statement of what the LOTFormer attention forward
 * path computes (arXiv 2509.23436, Section "Method": the dot-product costs, the
 * two entropic transport problems Eq. (1)-(2) in their Sinkhorn scaling form,
 * the glued coupling Eq. (3) and the factorised head output Eq. (4)).
 *
 * Only the tests, the smoke check and the bench's cpu_baseline / reference arm
 * may call this file.  It shares no code with the CUDA library and never
 * includes one of its headers.  Nothing here is blocked, fused or reordered:
 * every function is the definition (or, for the Sinkhorn solve, the iteration
 * in the order documented below) written as dense loops.
 *
 * Conventions (all arrays row-major, last index fastest, host memory, double):
 *   tokens x  [n, d]      pivots z  [r, d]      pivot masses beta [r] (>0, sum 1)
 *   cost   C  [n, r]      C[i][t] = <x_i, z_t>          (no 1/sqrt(d) factor)
 *   token marginal m [n]  m_i >= 0, sum 1; m_i == 0 removes token i from the
 *                         transport problem (it carries no mass)
 *   plan   P  [n, r]      token-major storage of Gamma^(1)^T resp. Gamma^(2)^T
 *
 * Pins (tests/test_oracle_pins.py): 2x2 closed form, brute-force n x n coupling
 * marginals / rank / outer-product identity, r = 1 and equal-pivot special
 * cases, objective-maximality under feasible perturbations, a scaling-domain
 * restatement at equal T, library matmul for the cost, metamorphic
 * invariances.  The finite-T iteration order (initial potentials zero, token
 * update first, one closing token update) is a reading the paper leaves open:
 * for that aspect alone the status is "parity unpinned"; the fixed point it
 * converges to is pinned.
 */
#include <math.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* ---- Section "Method", the unnumbered display that defines C^(1), C^(2) before Eq. (1):
 *      C_it = z_t^T x_i. */
void lot_oracle_cost(const double *x, const double *z, int n, int d, int r, double *C)
{
    for (int i = 0; i < n; ++i)
        for (int t = 0; t < r; ++t) {
            double acc = 0.0;
            for (int c = 0; c < d; ++c)
                acc += x[(size_t)i * d + c] * z[(size_t)t * d + c];
            C[(size_t)i * r + t] = acc;
        }
}

/* log(sum_k exp(a_k)) over k with weight mask; -inf if no term. */
static double lse(const double *a, const unsigned char *skip, int len, int stride)
{
    double mx = -INFINITY;
    for (int k = 0; k < len; ++k)
        if (!skip || !skip[k])
            if (a[(size_t)k * stride] > mx) mx = a[(size_t)k * stride];
    if (mx == -INFINITY) return -INFINITY;
    double s = 0.0;
    for (int k = 0; k < len; ++k)
        if (!skip || !skip[k])
            s += exp(a[(size_t)k * stride] - mx);
    return mx + log(s);
}

/* ---- Eq. (1)/(2) in the scaling form Gamma = Diag(u) exp(C/eps) Diag(v),
 *      u = exp(f/eps), v = exp(g/eps), solved by alternating marginal
 *      projections in the log domain.
 *
 *      g <- 0;  repeat iters times:
 *          f_i = eps (log m_i - LSE_t((C_it + g_t)/eps))      token side
 *          g_t = eps (log beta_t - LSE_i((C_it + f_i)/eps))    pivot side
 *      then one closing token-side update of f, and
 *          P_it = exp((C_it + f_i + g_t)/eps).
 *      Tokens with m_i == 0 take no part (f_i = -inf, P_i: = 0).
 *
 *      g [r], f [n], P [n,r] are outputs; f and P may be NULL. */
void lot_oracle_sinkhorn_from(const double *C, const double *beta, const double *m,
                              int n, int r, double eps, int iters, const double *g0,
                              double *g, double *f, double *P);

void lot_oracle_sinkhorn(const double *C, const double *beta, const double *m,
                         int n, int r, double eps, int iters,
                         double *g, double *f, double *P)
{
    lot_oracle_sinkhorn_from(C, beta, m, n, r, eps, iters, NULL, g, f, P);
}

/* The same iteration started from a given pivot potential g0 (NULL = zeros): the state of the
 * iteration between two passes is g alone, so T1 iterations followed by T2 more from the
 * exported g are T1 + T2 iterations (warm start across layers or steps). */
void lot_oracle_sinkhorn_from(const double *C, const double *beta, const double *m,
                              int n, int r, double eps, int iters, const double *g0,
                              double *g, double *f, double *P)
{
    double *fl = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
    double *tmp = (double *)malloc(sizeof(double) * (size_t)((n > r ? n : r) + 1));
    unsigned char *dead = (unsigned char *)malloc((size_t)(n > 0 ? n : 1));
    for (int i = 0; i < n; ++i) dead[i] = !(m[i] > 0.0);
    for (int t = 0; t < r; ++t) g[t] = g0 ? g0[t] : 0.0;

    for (int it = 0; it <= iters; ++it) {
        /* token-side update with the current g */
        for (int i = 0; i < n; ++i) {
            if (dead[i]) { fl[i] = -INFINITY; continue; }
            for (int t = 0; t < r; ++t) tmp[t] = (C[(size_t)i * r + t] + g[t]) / eps;
            fl[i] = eps * (log(m[i]) - lse(tmp, NULL, r, 1));
        }
        if (it == iters) break; /* closing token update done */
        /* pivot-side update with the new f */
        for (int t = 0; t < r; ++t) {
            for (int i = 0; i < n; ++i)
                tmp[i] = dead[i] ? 0.0 : (C[(size_t)i * r + t] + fl[i]) / eps;
            g[t] = eps * (log(beta[t]) - lse(tmp, dead, n, 1));
        }
    }
    if (f) memcpy(f, fl, sizeof(double) * (size_t)n);
    if (P)
        for (int i = 0; i < n; ++i)
            for (int t = 0; t < r; ++t)
                P[(size_t)i * r + t] =
                    dead[i] ? 0.0 : exp((C[(size_t)i * r + t] + fl[i] + g[t]) / eps);
    free(fl); free(tmp); free(dead);
}

/* ---- Eq. (3): Gamma = Gamma1^T Diag(beta)^-1 Gamma2, formed explicitly
 *      (brute force, tiny sizes only).  P1 [nq,r], P2 [nk,r], G [nq,nk]. */
void lot_oracle_coupling(const double *P1, const double *P2, const double *beta,
                         int nq, int nk, int r, double *G)
{
    for (int i = 0; i < nq; ++i)
        for (int j = 0; j < nk; ++j) {
            double acc = 0.0;
            for (int t = 0; t < r; ++t)
                acc += P1[(size_t)i * r + t] * P2[(size_t)j * r + t] / beta[t];
            G[(size_t)i * nk + j] = acc;
        }
}

/* ---- Eq. (4) and the paragraph "Rank and complexity":
 *      Y = Gamma2 V (r x dv), Z' = Diag(beta)^-1 Y, O = Gamma1^T Z',
 *      then the row-stochastic scaling out_i = O_i / a_i (a_i the query
 *      marginal; = n O_i in the balanced case, so that A 1 = 1).
 *      Rows with a_i == 0 are written as zeros. */
void lot_oracle_apply(const double *P1, const double *P2, const double *beta,
                      const double *a, const double *V,
                      int nq, int nk, int r, int dv, double *out)
{
    double *Y = (double *)calloc((size_t)r * dv, sizeof(double));
    for (int t = 0; t < r; ++t)
        for (int c = 0; c < dv; ++c) {
            double acc = 0.0;
            for (int j = 0; j < nk; ++j)
                acc += P2[(size_t)j * r + t] * V[(size_t)j * dv + c];
            Y[(size_t)t * dv + c] = acc / beta[t];
        }
    for (int i = 0; i < nq; ++i)
        for (int c = 0; c < dv; ++c) {
            double acc = 0.0;
            for (int t = 0; t < r; ++t)
                acc += P1[(size_t)i * r + t] * Y[(size_t)t * dv + c];
            out[(size_t)i * dv + c] = a[i] > 0.0 ? acc / a[i] : 0.0;
        }
    free(Y);
}

/* ---- One head, start to end: costs, both solves, apply.
 *      a [n] query marginal, b [n] key marginal.  Optional outputs g1,g2 [r],
 *      P1,P2 [n,r] may be NULL. */
void lot_oracle_head(const double *q, const double *k, const double *v,
                     const double *z, const double *beta,
                     const double *a, const double *b,
                     int n, int d, int r, double eps, int iters,
                     double *out, double *g1, double *g2, double *P1o, double *P2o)
{
    size_t nr = (size_t)n * r;
    double *C1 = (double *)malloc(sizeof(double) * (nr ? nr : 1));
    double *C2 = (double *)malloc(sizeof(double) * (nr ? nr : 1));
    double *P1 = (double *)malloc(sizeof(double) * (nr ? nr : 1));
    double *P2 = (double *)malloc(sizeof(double) * (nr ? nr : 1));
    double *ga = (double *)malloc(sizeof(double) * (size_t)r);
    double *gb = (double *)malloc(sizeof(double) * (size_t)r);
    lot_oracle_cost(q, z, n, d, r, C1);
    lot_oracle_cost(k, z, n, d, r, C2);
    lot_oracle_sinkhorn(C1, beta, a, n, r, eps, iters, ga, NULL, P1);
    lot_oracle_sinkhorn(C2, beta, b, n, r, eps, iters, gb, NULL, P2);
    lot_oracle_apply(P1, P2, beta, a, v, n, n, r, d, out);
    if (g1) memcpy(g1, ga, sizeof(double) * (size_t)r);
    if (g2) memcpy(g2, gb, sizeof(double) * (size_t)r);
    if (P1o) memcpy(P1o, P1, sizeof(double) * nr);
    if (P2o) memcpy(P2o, P2, sizeof(double) * nr);
    free(C1); free(C2); free(P1); free(P2); free(ga); free(gb);
}

/* ---- One head with its own query and key counts (cross-attention: Appendix "Bidirectional scope",
 *      closing paragraph), arbitrary marginals a [nq], b [nk] (Section "Empirical measures and
 *      pivot": weights p^1, p^2 on the simplex; zero weight removes the token) and optional
 *      starting potentials g1_0, g2_0 [r] (NULL = zeros).  v, out have dv columns. */
void lot_oracle_head_x(const double *q, const double *k, const double *v,
                       const double *z, const double *beta,
                       const double *a, const double *b,
                       int nq, int nk, int d, int dv, int r, double eps, int iters,
                       const double *g1_0, const double *g2_0,
                       double *out, double *g1, double *g2, double *P1o, double *P2o)
{
    size_t n1 = (size_t)nq * r, n2 = (size_t)nk * r;
    double *C1 = (double *)malloc(sizeof(double) * (n1 ? n1 : 1));
    double *C2 = (double *)malloc(sizeof(double) * (n2 ? n2 : 1));
    double *P1 = (double *)malloc(sizeof(double) * (n1 ? n1 : 1));
    double *P2 = (double *)malloc(sizeof(double) * (n2 ? n2 : 1));
    double *ga = (double *)malloc(sizeof(double) * (size_t)r);
    double *gb = (double *)malloc(sizeof(double) * (size_t)r);
    lot_oracle_cost(q, z, nq, d, r, C1);
    lot_oracle_cost(k, z, nk, d, r, C2);
    lot_oracle_sinkhorn_from(C1, beta, a, nq, r, eps, iters, g1_0, ga, NULL, P1);
    lot_oracle_sinkhorn_from(C2, beta, b, nk, r, eps, iters, g2_0, gb, NULL, P2);
    lot_oracle_apply(P1, P2, beta, a, v, nq, nk, r, dv, out);
    if (g1) memcpy(g1, ga, sizeof(double) * (size_t)r);
    if (g2) memcpy(g2, gb, sizeof(double) * (size_t)r);
    if (P1o) memcpy(P1o, P1, sizeof(double) * n1);
    if (P2o) memcpy(P2o, P2, sizeof(double) * n2);
    free(C1); free(C2); free(P1); free(P2); free(ga); free(gb);
}

/* ---- Eq. (5): the [CLS] row keeps a plain softmax over the keys,
 *      alpha_j = exp(tau <q_cls, k_j>) / sum_l exp(tau <q_cls, k_l>),  out_cls = sum_j alpha_j v_j
 *      (tau is the paper's beta > 0 of Eq. (5), renamed because beta names the pivot masses here).
 *      Keys with alive[j] == 0 are left out (alive == NULL: all keys). */
void lot_oracle_cls_row(const double *q0, const double *k, const double *v, const unsigned char *alive,
                        int nk, int d, int dv, double tau, double *out0)
{
    double *s = (double *)malloc(sizeof(double) * (size_t)(nk > 0 ? nk : 1));
    double mx = -INFINITY;
    for (int j = 0; j < nk; ++j) {
        double acc = 0.0;
        for (int c = 0; c < d; ++c) acc += q0[c] * k[(size_t)j * d + c];
        s[j] = tau * acc;
        if ((!alive || alive[j]) && s[j] > mx) mx = s[j];
    }
    double den = 0.0;
    for (int j = 0; j < nk; ++j)
        if (!alive || alive[j]) den += exp(s[j] - mx);
    for (int c = 0; c < dv; ++c) {
        double acc = 0.0;
        for (int j = 0; j < nk; ++j)
            if (!alive || alive[j]) acc += exp(s[j] - mx) / den * v[(size_t)j * dv + c];
        out0[c] = acc;
    }
    free(s);
}

/* ---- All (batch, head) slices.  q,k,v,out [B,H,n,d]; z [H,r,d]; beta [H,r]
 *      (per head, shared over the batch: Section "Method", closing remark on multi-head attention).
 *      Query marginal uniform 1/n.  Key marginal uniform 1/n, or, when
 *      key_len != NULL, 1/key_len[b] on tokens j < key_len[b] and zero beyond.
 *      g1,g2 [B,H,r] optional.  Slices are independent; OpenMP runs them side
 *      by side and changes no arithmetic.  Returns the thread count used. */
int lot_oracle_attention_fwd(const double *q, const double *k, const double *v,
                             const double *z, const double *beta, const int *key_len,
                             int B, int H, int n, int d, int r, double eps, int iters,
                             double *out, double *g1, double *g2, int threads)
{
    int used = 1;
#ifdef _OPENMP
    if (threads > 0) omp_set_num_threads(threads);
    used = omp_get_max_threads();
#else
    (void)threads;
#endif
    int slices = B * H;
#pragma omp parallel for schedule(dynamic, 1)
    for (int s = 0; s < slices; ++s) {
        int bi = s / H, h = s % H;
        size_t off = (size_t)s * n * d;
        double *a = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
        double *b = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
        int L = key_len ? key_len[bi] : n;
        for (int i = 0; i < n; ++i) {
            a[i] = 1.0 / (double)n;
            b[i] = i < L ? 1.0 / (double)L : 0.0;
        }
        lot_oracle_head(q + off, k + off, v + off,
                        z + (size_t)h * r * d, beta + (size_t)h * r, a, b,
                        n, d, r, eps, iters, out + off,
                        g1 ? g1 + (size_t)s * r : NULL, g2 ? g2 + (size_t)s * r : NULL,
                        NULL, NULL);
        free(a); free(b);
    }
    return used;
}
