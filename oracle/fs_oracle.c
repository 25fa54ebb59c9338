/*
 * fs_oracle.c -- plain fp64 CPU reference for the Sinkhorn hot path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the checker, not the product: it is
 * slow on purpose, shares no code with the CUDA library, and may be called only
 * from the test-suite, the smoke check and the benchmark's CPU-baseline leg.
 *
 * Every function takes the same fp32-rounded inputs the GPU path receives
 * (matrix, marginals), widens them to double on read and does all arithmetic
 * in fp64 with plain ascending-index sums.  There is no blocking, fusion or
 * reordering beyond what the definitions state.  The optional OpenMP pragmas
 * parallelise over OUTPUT elements only, so the order in which each output's
 * sum is accumulated never changes and results are identical for any thread
 * count.
 *
 * What is computed, and the passage each part follows:
 *   - Gibbs kernel K = exp(-C/eps), plan P = diag(u) K diag(v), the scaling
 *     iteration u <- a ./ (K v), v <- b ./ (K^T u)        (Section 1, Eq. 1 and
 *     the display after it; fixed-point map T of the convergence appendix)
 *   - order "u first, then v with the NEW u", start u = v = 1  (Algorithm 1)
 *   - the c-client All-to-All protocol with row blocks I_j, local matvecs
 *     q_I = K_{I,:} v and r_I = (K_{:,I})^T u, Allgather of slices
 *                                           (Algorithm 1, Section 3.1, Assumption 1)
 *   - the relaxed update u <- (1-eta) u + eta a ./ (K v) and its v counterpart         (Section 3.3)
 *   - the strict row-partition form r = sum_j K_{I_j,:}^T u_{I_j}
 *                                           (2D block baseline of the appendix)
 *   - stabilised log-domain updates with f = eps log u, g = eps log v
 *     (the paper names them in Section 1 / Section 2.1 / the DP appendix's
 *     l_u = log u; the formula is the standard one:
 *        f_i = eps log a_i - eps LSE_l((g_l - C_il)/eps),
 *        g_l = eps log b_l - eps LSE_i((f_i - C_il)/eps))
 *   - the same iteration with K applied implicitly from two point clouds,
 *     K_il = exp(-scale |x_i - y_l|^2 / eps)        (Section 3.1, Section 4.1 remark, Section 5.4)
 *   - marginal error err = || P 1 - a ||                 (Section 5.3, DP appendix)
 *   - transport cost <P,C>, dual and primal objective values      (Eq. 1)
 *
 * Pins (tests/test_oracle_*.py, all CPU): rank-1 closed form, large-eps limit,
 * scaling/log equivalence, protocol == centralized bit for bit (Prop. 1),
 * fixed-point marginals and strong duality, half-step invariants, the 2x2
 * quadratic closed form, an independent Newton solve of the dual for n <= 8,
 * brute force over all block compositions; for the implicit kernel: hand-placed
 * points with integer squared distances, symmetry and zero diagonal for one cloud,
 * translation invariance, agreement with the stored-cost iteration.  The paper's printed 3x3 toy plan
 * is internally inconsistent (its row sums are not the stated a) and pins
 * nothing; it is used only for "column sums equal b".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define OR_KIND_KERNEL 0 /* matrix holds K */
#define OR_KIND_COST 1   /* matrix holds C; K = exp(-C/eps) evaluated in fp64 */

/* K_il as a double, from either a stored kernel or a stored cost (Section 1). */
static inline double kern(const float *M, int64_t ld, int kind, double eps, int64_t i, int64_t l) {
    double m = (double)M[i * ld + l];
    return kind == OR_KIND_KERNEL ? m : exp(-m / eps);
}

/* ---------------------------------------------------------------- scaling domain */

/* q_i = sum_l K_il v_l for rows [r0, r1): the local matvec q_I = K_{I,:} v (Section 3.1). */
void or_matvec_rows(int64_t n, const float *M, int64_t ld, int kind, double eps, const double *v,
                    int64_t r0, int64_t r1, double *q /* length n, entries r0..r1-1 written */) {
#pragma omp parallel for schedule(static)
    for (int64_t i = r0; i < r1; ++i) {
        double s = 0.0;
        for (int64_t l = 0; l < n; ++l) s += kern(M, ld, kind, eps, i, l) * v[l];
        q[i] = s;
    }
}

/* r_l = sum_{i=0}^{n-1} K_il u_i for columns [c0, c1): the restricted transpose action
 * r_I = (K_{:,I})^T u of Assumption 1.  i ascending for every l. */
void or_matvec_cols(int64_t n, const float *M, int64_t ld, int kind, double eps, const double *u,
                    int64_t c0, int64_t c1, double *r /* length n, entries c0..c1-1 written */) {
    const int64_t strip = 256;
    int64_t nstrips = (c1 - c0 + strip - 1) / strip;
#pragma omp parallel for schedule(static)
    for (int64_t s = 0; s < nstrips; ++s) {
        int64_t lo = c0 + s * strip, hi = lo + strip < c1 ? lo + strip : c1;
        for (int64_t l = lo; l < hi; ++l) r[l] = 0.0;
        for (int64_t i = 0; i < n; ++i) {
            double ui = u[i];
            for (int64_t l = lo; l < hi; ++l) r[l] += kern(M, ld, kind, eps, i, l) * ui;
        }
    }
}

/* Partial transpose product over a ROW block only: p_l = sum_{i in [r0,r1)} K_il u_i, all l.
 * Building block of the strict row-partition form (2D block baseline). */
static void matvec_cols_rowblock(int64_t n, const float *M, int64_t ld, int kind, double eps,
                                 const double *u, int64_t r0, int64_t r1, double *p) {
    const int64_t strip = 256;
    int64_t nstrips = (n + strip - 1) / strip;
#pragma omp parallel for schedule(static)
    for (int64_t s = 0; s < nstrips; ++s) {
        int64_t lo = s * strip, hi = lo + strip < n ? lo + strip : n;
        for (int64_t l = lo; l < hi; ++l) p[l] = 0.0;
        for (int64_t i = r0; i < r1; ++i) {
            double ui = u[i];
            for (int64_t l = lo; l < hi; ++l) p[l] += kern(M, ld, kind, eps, i, l) * ui;
        }
    }
}

/* One row half-step: q = K v, u = a ./ q (Algorithm 1, first two statements of the loop). */
void or_row_pass(int64_t n, const float *M, int64_t ld, int kind, double eps, const float *a,
                 const double *v, double *u_out, double *q_out /* may be NULL */) {
    double *q = q_out ? q_out : (double *)malloc(sizeof(double) * (size_t)n);
    or_matvec_rows(n, M, ld, kind, eps, v, 0, n, q);
    for (int64_t i = 0; i < n; ++i) u_out[i] = (double)a[i] / q[i];
    if (!q_out) free(q);
}

/* One column half-step: r = K^T u, v = b ./ r (Algorithm 1, statements four and five). */
void or_col_pass(int64_t n, const float *M, int64_t ld, int kind, double eps, const float *b,
                 const double *u, double *v_out, double *r_out /* may be NULL */) {
    double *r = r_out ? r_out : (double *)malloc(sizeof(double) * (size_t)n);
    or_matvec_cols(n, M, ld, kind, eps, u, 0, n, r);
    for (int64_t l = 0; l < n; ++l) v_out[l] = (double)b[l] / r[l];
    if (!r_out) free(r);
}

/* Centralized Sinkhorn-Knopp: iters applications of the map T to (u, v), in place.
 * The caller supplies the start (Algorithm 1 uses u = v = 1). */
void or_sinkhorn_scaling(int64_t n, const float *M, int64_t ld, int kind, double eps,
                         const float *a, const float *b, int64_t iters, double *u, double *v) {
    for (int64_t t = 0; t < iters; ++t) {
        or_row_pass(n, M, ld, kind, eps, a, v, u, NULL);
        or_col_pass(n, M, ld, kind, eps, b, u, v, NULL);
    }
}

/* Relaxed (damped) scaling iteration, the centralized view given with the asynchronous variant
 * (Section 3.3):  u <- (1 - eta) u + eta a ./ (K v),  v <- (1 - eta) v + eta b ./ (K^T u), the v update
 * using the new u.  eta = 1 is or_sinkhorn_scaling. */
void or_sinkhorn_damped(int64_t n, const float *M, int64_t ld, int kind, double eps, const float *a,
                        const float *b, double eta, int64_t iters, double *u, double *v) {
    double *t = (double *)malloc(sizeof(double) * (size_t)n);
    for (int64_t it = 0; it < iters; ++it) {
        or_row_pass(n, M, ld, kind, eps, a, v, t, NULL);
        for (int64_t i = 0; i < n; ++i) u[i] = (1.0 - eta) * u[i] + eta * t[i];
        or_col_pass(n, M, ld, kind, eps, b, u, t, NULL);
        for (int64_t l = 0; l < n; ++l) v[l] = (1.0 - eta) * v[l] + eta * t[l];
    }
    free(t);
}

/* Algorithm 1 taken literally with c logical clients.  Client j keeps its OWN copy of the
 * global u and v (U[j], V[j]); it computes q_{I_j} from its row block and the v it holds,
 * updates its slice of u, the Allgather copies every client's slice into every client's
 * global u; then r_{I_j} from its column block K_{:,I_j} and the u it holds, its slice of
 * v, Allgather.  On return u, v are client 0's copies; *agree is 1 when all clients hold
 * identical copies at the end. */
void or_sinkhorn_protocol(int64_t n, int32_t c, const int64_t *off, const float *M, int64_t ld,
                          int kind, double eps, const float *a, const float *b, int64_t iters,
                          double *u, double *v, int32_t *agree) {
    size_t bytes = sizeof(double) * (size_t)n;
    double **U = (double **)malloc(sizeof(double *) * (size_t)c);
    double **V = (double **)malloc(sizeof(double *) * (size_t)c);
    double *buf = (double *)malloc(bytes);
    for (int32_t j = 0; j < c; ++j) {
        U[j] = (double *)malloc(bytes);
        V[j] = (double *)malloc(bytes);
        memcpy(U[j], u, bytes);
        memcpy(V[j], v, bytes);
    }
    for (int64_t t = 0; t < iters; ++t) {
        /* local row work, each client with its own view of v */
        for (int32_t j = 0; j < c; ++j) {
            or_matvec_rows(n, M, ld, kind, eps, V[j], off[j], off[j + 1], buf);
            for (int64_t i = off[j]; i < off[j + 1]; ++i) U[j][i] = (double)a[i] / buf[i];
        }
        /* Allgather u: slice j of client j goes to every client */
        for (int32_t j = 0; j < c; ++j)
            for (int32_t k = 0; k < c; ++k)
                if (k != j)
                    memcpy(U[k] + off[j], U[j] + off[j], sizeof(double) * (size_t)(off[j + 1] - off[j]));
        /* local column work from the column block K_{:,I_j} */
        for (int32_t j = 0; j < c; ++j) {
            or_matvec_cols(n, M, ld, kind, eps, U[j], off[j], off[j + 1], buf);
            for (int64_t l = off[j]; l < off[j + 1]; ++l) V[j][l] = (double)b[l] / buf[l];
        }
        /* Allgather v */
        for (int32_t j = 0; j < c; ++j)
            for (int32_t k = 0; k < c; ++k)
                if (k != j)
                    memcpy(V[k] + off[j], V[j] + off[j], sizeof(double) * (size_t)(off[j + 1] - off[j]));
    }
    int32_t same = 1;
    for (int32_t j = 1; j < c; ++j)
        if (memcmp(U[j], U[0], bytes) != 0 || memcmp(V[j], V[0], bytes) != 0) same = 0;
    memcpy(u, U[0], bytes);
    memcpy(v, V[0], bytes);
    if (agree) *agree = same;
    for (int32_t j = 0; j < c; ++j) {
        free(U[j]);
        free(V[j]);
    }
    free(U);
    free(V);
    free(buf);
}

/* Strict row partition: client j owns only ROWS I_j, so the transpose product is assembled
 * as r = sum_j K_{I_j,:}^T u_{I_j}, the per-client partial vectors added in client order
 * (what a sum-Allreduce of the partials delivers).  Same mathematics as the centralized
 * iteration, different association of the sum. */
void or_sinkhorn_rowpartition(int64_t n, int32_t c, const int64_t *off, const float *M, int64_t ld,
                              int kind, double eps, const float *a, const float *b, int64_t iters,
                              double *u, double *v) {
    size_t bytes = sizeof(double) * (size_t)n;
    double *q = (double *)malloc(bytes), *r = (double *)malloc(bytes), *p = (double *)malloc(bytes);
    for (int64_t t = 0; t < iters; ++t) {
        for (int32_t j = 0; j < c; ++j) or_matvec_rows(n, M, ld, kind, eps, v, off[j], off[j + 1], q);
        for (int64_t i = 0; i < n; ++i) u[i] = (double)a[i] / q[i];
        for (int64_t l = 0; l < n; ++l) r[l] = 0.0;
        for (int32_t j = 0; j < c; ++j) {
            matvec_cols_rowblock(n, M, ld, kind, eps, u, off[j], off[j + 1], p);
            for (int64_t l = 0; l < n; ++l) r[l] += p[l];
        }
        for (int64_t l = 0; l < n; ++l) v[l] = (double)b[l] / r[l];
    }
    free(q);
    free(r);
    free(p);
}

/* ---------------------------------------------------------------- log domain */

/* L_i = log sum_l exp((g_l - C_il)/eps) for every row i, by the two-pass definition:
 * first the maximum of the exponents, then the sum of exp(shifted), then the log. */
void or_lse_rows(int64_t n, const float *C, int64_t ld, double eps, const double *g, double *L) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        double mx = -INFINITY;
        for (int64_t l = 0; l < n; ++l) {
            double t = (g[l] - (double)C[i * ld + l]) / eps;
            if (t > mx) mx = t;
        }
        double s = 0.0;
        for (int64_t l = 0; l < n; ++l) s += exp((g[l] - (double)C[i * ld + l]) / eps - mx);
        L[i] = mx + log(s);
    }
}

/* M_l = log sum_i exp((f_i - C_il)/eps) for every column l, same two-pass definition. */
void or_lse_cols(int64_t n, const float *C, int64_t ld, double eps, const double *f, double *L) {
#pragma omp parallel for schedule(static)
    for (int64_t l = 0; l < n; ++l) {
        double mx = -INFINITY;
        for (int64_t i = 0; i < n; ++i) {
            double t = (f[i] - (double)C[i * ld + l]) / eps;
            if (t > mx) mx = t;
        }
        double s = 0.0;
        for (int64_t i = 0; i < n; ++i) s += exp((f[i] - (double)C[i * ld + l]) / eps - mx);
        L[l] = mx + log(s);
    }
}

/* f_i = eps log a_i - eps L_i  with L from or_lse_rows (log-domain row half-step). */
void or_log_row_pass(int64_t n, const float *C, int64_t ld, double eps, const float *a,
                     const double *g, double *f_out) {
    double *L = (double *)malloc(sizeof(double) * (size_t)n);
    or_lse_rows(n, C, ld, eps, g, L);
    for (int64_t i = 0; i < n; ++i) f_out[i] = eps * log((double)a[i]) - eps * L[i];
    free(L);
}

/* g_l = eps log b_l - eps M_l  with M from or_lse_cols (log-domain column half-step). */
void or_log_col_pass(int64_t n, const float *C, int64_t ld, double eps, const float *b,
                     const double *f, double *g_out) {
    double *L = (double *)malloc(sizeof(double) * (size_t)n);
    or_lse_cols(n, C, ld, eps, f, L);
    for (int64_t l = 0; l < n; ++l) g_out[l] = eps * log((double)b[l]) - eps * L[l];
    free(L);
}

/* Log-domain Sinkhorn, iters full iterations in place (start is the caller's; f = g = 0
 * corresponds to u = v = 1). */
void or_sinkhorn_log(int64_t n, const float *C, int64_t ld, double eps, const float *a,
                     const float *b, int64_t iters, double *f, double *g) {
    for (int64_t t = 0; t < iters; ++t) {
        or_log_row_pass(n, C, ld, eps, a, g, f);
        or_log_col_pass(n, C, ld, eps, b, f, g);
    }
}

/* ---------------------------------------------------------------- implicit (on-the-fly) kernel from points */

/* Embedding cost between point i of cloud X and point l of cloud Y (both n x d, fp32, row-major):
 * C_il = scale * sum_k (x_ik - y_lk)^2 -- the squared Euclidean cost of the embedding experiment (Section 5.4),
 * optionally rescaled (the workloads divide by the largest entry).  Plain differences, k ascending. */
static inline double sqdist_cost(const float *X, const float *Y, int64_t d, double scale, int64_t i, int64_t l) {
    double s = 0.0;
    for (int64_t k = 0; k < d; ++k) {
        double t = (double)X[i * d + k] - (double)Y[l * d + k];
        s += t * t;
    }
    return scale * s;
}

/* C (n x n doubles, row-major) from the two clouds. */
void or_cost_from_points(int64_t n, int64_t d, const float *X, const float *Y, double scale, double *C) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i)
        for (int64_t l = 0; l < n; ++l) C[i * n + l] = sqdist_cost(X, Y, d, scale, i, l);
}

/* Sinkhorn-Knopp with the kernel applied implicitly: K_il = exp(-C_il/eps) is evaluated from the points every
 * time it is needed and never stored (Section 3.1 "do not assume it is explicitly materialized"; Section 4.1,
 * remark on on-the-fly kernels).  Same iteration, order and start convention as or_sinkhorn_scaling. */
void or_sinkhorn_points(int64_t n, int64_t d, const float *X, const float *Y, double scale, double eps,
                        const float *a, const float *b, int64_t iters, double *u, double *v) {
    for (int64_t t = 0; t < iters; ++t) {
#pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < n; ++i) {
            double q = 0.0;
            for (int64_t l = 0; l < n; ++l) q += exp(-sqdist_cost(X, Y, d, scale, i, l) / eps) * v[l];
            u[i] = (double)a[i] / q;
        }
#pragma omp parallel for schedule(static)
        for (int64_t l = 0; l < n; ++l) {
            double r = 0.0;
            for (int64_t i = 0; i < n; ++i) r += exp(-sqdist_cost(X, Y, d, scale, i, l) / eps) * u[i];
            v[l] = (double)b[l] / r;
        }
    }
}

/* Marginals of P = diag(u) K diag(v) with the implicit kernel: row_i = u_i (K v)_i, col_l = v_l (K^T u)_l. */
void or_marginals_points(int64_t n, int64_t d, const float *X, const float *Y, double scale, double eps,
                         const double *u, const double *v, double *row, double *col) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        double q = 0.0;
        for (int64_t l = 0; l < n; ++l) q += exp(-sqdist_cost(X, Y, d, scale, i, l) / eps) * v[l];
        row[i] = u[i] * q;
    }
#pragma omp parallel for schedule(static)
    for (int64_t l = 0; l < n; ++l) {
        double r = 0.0;
        for (int64_t i = 0; i < n; ++i) r += exp(-sqdist_cost(X, Y, d, scale, i, l) / eps) * u[i];
        col[l] = v[l] * r;
    }
}

/* ---------------------------------------------------------------- errors and objectives */

/* Marginals of P = diag(u) K diag(v) in the scaling domain: row_i = u_i (K v)_i,
 * col_l = v_l (K^T u)_l. */
void or_marginals_scaling(int64_t n, const float *M, int64_t ld, int kind, double eps,
                          const double *u, const double *v, double *row, double *col) {
    or_matvec_rows(n, M, ld, kind, eps, v, 0, n, row);
    or_matvec_cols(n, M, ld, kind, eps, u, 0, n, col);
    for (int64_t i = 0; i < n; ++i) row[i] *= u[i];
    for (int64_t l = 0; l < n; ++l) col[l] *= v[l];
}

/* Marginals of P_il = exp((f_i + g_l - C_il)/eps) in the log domain:
 * row_i = exp(f_i/eps + LSE_l((g_l - C_il)/eps)), col_l likewise. */
void or_marginals_log(int64_t n, const float *C, int64_t ld, double eps, const double *f,
                      const double *g, double *row, double *col) {
    or_lse_rows(n, C, ld, eps, g, row);
    or_lse_cols(n, C, ld, eps, f, col);
    for (int64_t i = 0; i < n; ++i) row[i] = exp(f[i] / eps + row[i]);
    for (int64_t l = 0; l < n; ++l) col[l] = exp(g[l] / eps + col[l]);
}

/* err[0] = sum_i |row_i - a_i|, err[1] = sqrt(sum_i (row_i - a_i)^2) (the paper's err_a),
 * err[2], err[3] the same for the columns against b. */
void or_marginal_errors(int64_t n, const double *row, const double *col, const float *a,
                        const float *b, double *err) {
    double r1 = 0, r2 = 0, c1 = 0, c2 = 0;
    for (int64_t i = 0; i < n; ++i) {
        double d = row[i] - (double)a[i];
        r1 += fabs(d);
        r2 += d * d;
    }
    for (int64_t l = 0; l < n; ++l) {
        double d = col[l] - (double)b[l];
        c1 += fabs(d);
        c2 += d * d;
    }
    err[0] = r1;
    err[1] = sqrt(r2);
    err[2] = c1;
    err[3] = sqrt(c2);
}

/* Writes P_il into P (n*n doubles, row-major).  domain 0: u_i K_il v_l; domain 1:
 * exp((x_i + y_l - C_il)/eps) with x = f, y = g and the matrix being C. */
void or_plan(int64_t n, const float *M, int64_t ld, int kind, double eps, int domain,
             const double *x, const double *y, double *P) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i)
        for (int64_t l = 0; l < n; ++l)
            P[i * n + l] = domain == 0 ? x[i] * kern(M, ld, kind, eps, i, l) * y[l]
                                       : exp((x[i] + y[l] - (double)M[i * ld + l]) / eps);
}

/* out[0] = <P,C> = sum_il P_il C_il
 * out[1] = primal objective of Eq. 1: <P,C> + eps sum_il P_il (log P_il - 1)
 * out[2] = sum_il P_il (total mass)
 * C is given separately (fp32, leading dimension ldc) so that a stored kernel can be used
 * for P in the scaling domain. */
void or_objectives(int64_t n, const float *M, int64_t ld, int kind, double eps, int domain,
                   const double *x, const double *y, const float *C, int64_t ldc, double *out) {
    double cost = 0, ent = 0, mass = 0;
    for (int64_t i = 0; i < n; ++i) {
        double rc = 0, re = 0, rm = 0;
        for (int64_t l = 0; l < n; ++l) {
            double p = domain == 0 ? x[i] * kern(M, ld, kind, eps, i, l) * y[l]
                                   : exp((x[i] + y[l] - (double)M[i * ld + l]) / eps);
            rc += p * (double)C[i * ldc + l];
            if (p > 0) re += p * (log(p) - 1.0);
            rm += p;
        }
        cost += rc;
        ent += re;
        mass += rm;
    }
    out[0] = cost;
    out[1] = cost + eps * ent;
    out[2] = mass;
}
