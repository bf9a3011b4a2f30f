/*
 * CPU oracle for the Gated KalmaNet (GKA) forward recurrence and decode step.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, token-by-token fp64
 * statement of what the method computes.  It shares no code with the CUDA
 * library and must never be reached from the product path; only the tests, the
 * smoke check and the benchmark's CPU-baseline leg may build, load or call it.
 *
 * What it follows (paper section / equation / algorithm):
 *   - forward recurrence, eq. (CH), Section 4.1:
 *         H_t = gamma_t H_{t-1} + k_t k_t^T,   U_t = gamma_t U_{t-1} + v_t k_t^T,
 *         x_t = CH(H_t + lambda_t I, q_t, r),  y_t = U_t x_t
 *   - beta_t-augmented write, Remark "canonical beta_t-augmented variant" (Section 4.1) and the
 *     appendix's modified eq. (CH): H_t = gamma_t H_{t-1} + beta_t k_t k_t^T,
 *     U_t = gamma_t U_{t-1} + beta_t v_t k_t^T (beta == NULL means beta_t = 1, the paper's experiments)
 *   - alpha-connection, Section 4.3 "Architectural Consideration": the read uses the convex combination
 *     alpha_t x_t + (1 - alpha_t) q_t in place of x_t (alpha == NULL means alpha_t = 1: y_t = U_t x_t)
 *   - Chebyshev Iteration, Algorithm 1 (weight schedule, grad descent, momentum)
 *   - eigenvalue bounds, Section 4.1 "Adaptive Regularization":
 *         L = ||H_t||_F + lambda_t,   mu = lambda_t
 *   - exact target, Section 4.1 "Motivation" (closed form of eq. (3)):
 *         y_t = U_t (H_t + lambda_t I)^{-1} q_t          (solved by Cholesky)
 *
 * Readings where the paper is silent:
 *   - lambda_t is a per-token input (absolute value); the optional adaptive mode
 *     lambda_t = a ||H_t||_F of Section 4.1 is selected with lam_mode = 1, in
 *     which case lam[] holds the per-token constant a.
 *   - the state is decayed, then written, then used: token t sees H_t and U_t.
 *   - n_iter = r counts matrix-vector products; r = 0 returns xi_0 = 2 q / (L + mu).
 *   - the matrix applied inside the loop is H_t + lambda_t I.
 *   - no blocking, fusion or reordering: one token at a time, direct Frobenius norm.
 *
 * Layouts (row-major, contiguous): q, k: [B, T, heads, d_k]; v, out: [B, T, heads, d_v];
 * gate, lam, fro: [B, T, heads]; state: [B, heads, d_k*d_k + d_v*d_k] = H then U,
 * H[i][j] row-major, U[i][j] = sum v_i k_j row-major (d_v rows, d_k columns).
 *
 * Parity pins live in tests/test_oracle_pins.py (brute-force ridge argmin, the
 * closed polynomial form of the Chebyshev iterate, the sharp Chebyshev error
 * bound, the printed contraction numbers of the Remark after Lemma 4, the
 * first-token closed form, recursive least squares for gamma == 1, the large
 * lambda limit).
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* Algorithm 1, weight schedule only: omega[0] = 2, omega[i] = 4 / (4 - rho^2 omega[i-1]). */
void gka_oracle_omega(double L, double mu, int r, double *omega /* r + 1 */)
{
    double rho = (L - mu) / (L + mu);
    omega[0] = 2.0;
    for (int i = 1; i <= r; ++i) omega[i] = 4.0 / (4.0 - rho * rho * omega[i - 1]);
}

/*
 * Algorithm 1 for a dense symmetric matrix A (D x D, row-major), right-hand side q,
 * bounds L >= mu > 0, r iterations.  xi receives xi_r.  The matrix handed in is the
 * one whose system is solved (the caller adds the ridge).
 */
void gka_oracle_chebyshev(int D, const double *A, const double *q, double L, double mu, int r,
                          double *xi)
{
    double *prev = (double *)calloc((size_t)D, sizeof(double)); /* xi_{i-2}, starts as xi_{-1} = 0 */
    double *cur = (double *)malloc((size_t)D * sizeof(double));  /* xi_{i-1}, starts as xi_0 */
    double *nxt = (double *)malloc((size_t)D * sizeof(double));
    double rho = (L - mu) / (L + mu);
    double omega = 2.0;
    for (int d = 0; d < D; ++d) cur[d] = 2.0 * q[d] / (L + mu);
    for (int i = 1; i <= r; ++i) {
        omega = 4.0 / (4.0 - rho * rho * omega);                 /* weight schedule */
        for (int d = 0; d < D; ++d) {
            double Ax = 0.0;
            for (int e = 0; e < D; ++e) Ax += A[(size_t)d * D + e] * cur[e];
            double g = cur[d] - (2.0 * omega / (L + mu)) * (Ax - q[d]); /* grad descent */
            nxt[d] = g + (omega - 1.0) * (cur[d] - prev[d]);            /* momentum */
        }
        double *t = prev; prev = cur; cur = nxt; nxt = t;
    }
    memcpy(xi, cur, (size_t)D * sizeof(double));
    free(prev); free(cur); free(nxt);
}

/* Solve A x = b for symmetric positive definite A by Cholesky (A = G G^T). Returns 0 on success. */
int gka_oracle_cholesky_solve(int D, const double *A, const double *b, double *x)
{
    double *G = (double *)malloc((size_t)D * D * sizeof(double));
    int rc = 0;
    for (int i = 0; i < D && !rc; ++i) {
        for (int j = 0; j <= i; ++j) {
            double s = A[(size_t)i * D + j];
            for (int p = 0; p < j; ++p) s -= G[(size_t)i * D + p] * G[(size_t)j * D + p];
            if (i == j) {
                if (!(s > 0.0)) { rc = 1; break; }
                G[(size_t)i * D + i] = sqrt(s);
            } else {
                G[(size_t)i * D + j] = s / G[(size_t)j * D + j];
            }
        }
    }
    if (!rc) {
        for (int i = 0; i < D; ++i) {           /* G y = b */
            double s = b[i];
            for (int p = 0; p < i; ++p) s -= G[(size_t)i * D + p] * x[p];
            x[i] = s / G[(size_t)i * D + i];
        }
        for (int i = D - 1; i >= 0; --i) {      /* G^T x = y */
            double s = x[i];
            for (int p = i + 1; p < D; ++p) s -= G[(size_t)p * D + i] * x[p];
            x[i] = s / G[(size_t)i * D + i];
        }
    }
    free(G);
    return rc;
}

/* One token of eq. (CH) on one head's state.  H: dk x dk, U: dv x dk, A: scratch dk x dk. */
static int gka_token(int dk, int dv, double *H, double *U, double *A,
                     const double *q, const double *k, const double *v,
                     double gamma, double beta, double alpha, double lam_in, int lam_mode, int r,
                     double *xi, double *y_ch, double *y_exact, double *fro_out, double *xi_exact)
{
    /* state write: decay, then rank-one update */
    for (int i = 0; i < dk; ++i)
        for (int j = 0; j < dk; ++j)
            H[(size_t)i * dk + j] = gamma * H[(size_t)i * dk + j] + beta * k[i] * k[j];
    for (int i = 0; i < dv; ++i)
        for (int j = 0; j < dk; ++j)
            U[(size_t)i * dk + j] = gamma * U[(size_t)i * dk + j] + beta * v[i] * k[j];
    /* direct Frobenius norm */
    double ss = 0.0;
    for (size_t e = 0; e < (size_t)dk * dk; ++e) ss += H[e] * H[e];
    double f = sqrt(ss);
    if (fro_out) *fro_out = f;
    double lam = lam_mode ? lam_in * f : lam_in;   /* adaptive mode: lambda_t = a ||H_t||_F */
    double L = f + lam, mu = lam;
    /* A = H_t + lambda_t I */
    memcpy(A, H, (size_t)dk * dk * sizeof(double));
    for (int i = 0; i < dk; ++i) A[(size_t)i * dk + i] += lam;
    gka_oracle_chebyshev(dk, A, q, L, mu, r, xi);
    for (int i = 0; i < dv; ++i) {
        double s = 0.0;
        for (int j = 0; j < dk; ++j) s += U[(size_t)i * dk + j] * (alpha * xi[j] + (1.0 - alpha) * q[j]);
        y_ch[i] = s;
    }
    int rc = 0;
    if (y_exact) {
        rc = gka_oracle_cholesky_solve(dk, A, q, xi_exact);
        for (int i = 0; i < dv; ++i) {
            double s = 0.0;
            for (int j = 0; j < dk; ++j) s += U[(size_t)i * dk + j] * (alpha * xi_exact[j] + (1.0 - alpha) * q[j]);
            y_exact[i] = s;
        }
    }
    return rc;
}

/*
 * Forward recurrence over whole sequences.  Nullable: beta (write strength 1), alpha (1), state_in (zero state),
 * out_exact, fro, x_ch (the Chebyshev iterates xi_r, [B,T,heads,d_k]), state_out.
 * threads <= 0 uses the OpenMP default.  Returns 0, or 1 if a Cholesky factorisation failed.
 */
int gka_oracle_fwd(int B, int T, int heads, int dk, int dv,
                   const double *q, const double *k, const double *v,
                   const double *gate, const double *lam, const double *beta, const double *alpha,
                   int lam_mode, int n_iter, const double *state_in,
                   double *out_ch, double *out_exact, double *fro, double *x_ch,
                   double *state_out, int threads)
{
    int rc_all = 0;
    size_t st = (size_t)dk * dk + (size_t)dv * dk;
#ifdef _OPENMP
    if (threads > 0) omp_set_num_threads(threads);
#endif
#pragma omp parallel for schedule(dynamic, 1) reduction(| : rc_all)
    for (int bh = 0; bh < B * heads; ++bh) {
        int b = bh / heads, h = bh % heads;
        double *H = (double *)calloc(st, sizeof(double));
        double *U = H + (size_t)dk * dk;
        double *A = (double *)malloc((size_t)dk * dk * sizeof(double));
        double *xi = (double *)malloc((size_t)dk * sizeof(double));
        double *xe = (double *)malloc((size_t)dk * sizeof(double));
        double *ye = (double *)malloc((size_t)dv * sizeof(double));
        if (state_in) memcpy(H, state_in + (size_t)bh * st, st * sizeof(double));
        for (int t = 0; t < T; ++t) {
            size_t tok = ((size_t)b * T + t) * heads + h;
            double f;
            int rc = gka_token(dk, dv, H, U, A, q + tok * dk, k + tok * dk, v + tok * dv,
                               gate[tok], beta ? beta[tok] : 1.0, alpha ? alpha[tok] : 1.0, lam[tok], lam_mode,
                               n_iter, xi,
                               out_ch + tok * dv, out_exact ? ye : NULL, &f, xe);
            rc_all |= rc;
            if (out_exact) memcpy(out_exact + tok * dv, ye, (size_t)dv * sizeof(double));
            if (fro) fro[tok] = f;
            if (x_ch) memcpy(x_ch + tok * dk, xi, (size_t)dk * sizeof(double));
        }
        if (state_out) memcpy(state_out + (size_t)bh * st, H, st * sizeof(double));
        free(H); free(A); free(xi); free(xe); free(ye);
    }
    return rc_all;
}

/*
 * Recurrent single-token step: the same eq. (CH) applied once per (sequence, head),
 * updating state in place.  q, k: [N, heads, d_k]; v, out: [N, heads, d_v];
 * gate, lam: [N, heads]; state: [N, heads, d_k*d_k + d_v*d_k].
 */
int gka_oracle_decode(int N, int heads, int dk, int dv, double *state,
                      const double *q, const double *k, const double *v,
                      const double *gate, const double *lam, const double *beta, const double *alpha,
                      int lam_mode, int n_iter, double *out_ch, double *out_exact, int threads)
{
    int rc_all = 0;
    size_t st = (size_t)dk * dk + (size_t)dv * dk;
#ifdef _OPENMP
    if (threads > 0) omp_set_num_threads(threads);
#endif
#pragma omp parallel for schedule(static) reduction(| : rc_all)
    for (int nh = 0; nh < N * heads; ++nh) {
        double *H = state + (size_t)nh * st;
        double *U = H + (size_t)dk * dk;
        double *A = (double *)malloc((size_t)dk * dk * sizeof(double));
        double *xi = (double *)malloc((size_t)dk * sizeof(double));
        double *xe = (double *)malloc((size_t)dk * sizeof(double));
        rc_all |= gka_token(dk, dv, H, U, A, q + (size_t)nh * dk, k + (size_t)nh * dk,
                            v + (size_t)nh * dv, gate[nh], beta ? beta[nh] : 1.0, alpha ? alpha[nh] : 1.0, lam[nh],
                            lam_mode, n_iter, xi,
                            out_ch + (size_t)nh * dv,
                            out_exact ? out_exact + (size_t)nh * dv : NULL, NULL, xe);
        free(A); free(xi); free(xe);
    }
    return rc_all;
}

int gka_oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
