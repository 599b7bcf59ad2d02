/*
 * SVD-Cache oracle: a plain, slow, fp64 CPU statement of what the hot path computes.
 *
 * THIS FILE IS TEST INFRASTRUCTURE. Only the test-suite, the smoke check and the
 * benchmark's CPU-baseline leg may build or call it. It shares no code, header, table
 * or helper with the CUDA library, and the CUDA library never calls it.
 *
 * Every routine is the definition written out (the method is exact linear algebra, not
 * an approximation), in the paper's notation:
 *   F   : N x D feature matrix of one DiT block (row = token)            Sec. 3.2
 *   V_k : D x k, the k leading right singular vectors                    Eq. 4, Eq. 5
 *   C   : N x k coefficients F V_k  (= U_k diag(sigma_k))                Eq. 8, Eq. 9
 *   R   : N x D residual F - F_k                                         Eq. 10
 *   Chat: N x k EMA state of the coefficients                            Eq. 11
 * All matrices are row-major, contiguous, double precision. Nothing is blocked, fused
 * or reordered beyond what the formulas state; OpenMP only splits independent rows.
 *
 * Pins (tests/test_oracle_*.py): orthonormality, trace and Eckart-Young identities,
 * one-sided Jacobi SVD on small matrices, numpy's eigh/svd on the same inputs,
 * exact reconstruction at k = D, residual orthogonality, the energy split
 * |F|^2 = |C|^2 + |R|^2, EMA closed forms, and hand-computed fixtures; for the routines beyond
 * the method itself (tests/test_oracle_extensions.py): the residual EMA against its closed
 * forms and against oracle_full_step at beta_r = 0, the forecasts against polynomial sequences
 * (exactness of the Newton form, the known lag of the Taylor form), numpy's polynomial fit, and
 * hand-computed values; the left factors against U diag(sigma) V^T = F_k and U^T U = I on the
 * calibration stack itself.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------------------
 * Gram matrix G = F^T F of a row-stack of features (M x D).  The right singular
 * vectors of the stack (Eq. 4) are the eigenvectors of G and sigma_i^2 its eigenvalues.
 * ---------------------------------------------------------------------------------- */
void oracle_gram(const double *F, int64_t M, int D, double *G)
{
    memset(G, 0, (size_t)D * D * sizeof(double));
#pragma omp parallel for schedule(dynamic, 4)
    for (int i = 0; i < D; ++i) {
        double *gi = G + (size_t)i * D;
        for (int64_t m = 0; m < M; ++m) {
            const double *f = F + (size_t)m * D;
            const double fi = f[i];
            for (int j = i; j < D; ++j) gi[j] += fi * f[j];
        }
    }
    for (int i = 0; i < D; ++i)
        for (int j = 0; j < i; ++j) G[(size_t)i * D + j] = G[(size_t)j * D + i];
}

/* ------------------------------------------------------------------------------------
 * Symmetric eigen-decomposition, textbook route: Householder reduction to tridiagonal
 * form, then implicit-shift QR sweeps with Wilkinson's shift on the tridiagonal matrix,
 * the rotations accumulated into the Householder basis.
 *   A (n x n, symmetric, destroyed)  ->  w (n eigenvalues, DEscending),
 *   Z (n x n, column j = eigenvector of w[j]).
 * Returns 0, or 1 if the QR sweeps did not converge.
 * ---------------------------------------------------------------------------------- */
static void householder_tridiagonal(int n, double *A, double *Z, double *d, double *e)
{
    double *v = (double *)malloc((size_t)n * sizeof(double));
    double *p = (double *)malloc((size_t)n * sizeof(double));
    for (int i = 0; i < n; ++i)
        for (int j = 0; j < n; ++j) Z[(size_t)i * n + j] = (i == j) ? 1.0 : 0.0;

    for (int k = 0; k + 2 < n; ++k) {
        const int len = n - k - 1; /* the reflector acts on indices k+1 .. n-1 */
        double norm2 = 0.0;
        for (int i = 0; i < len; ++i) {
            v[i] = A[(size_t)(k + 1 + i) * n + k];
            norm2 += v[i] * v[i];
        }
        if (norm2 == 0.0) continue;
        const double alpha = (v[0] > 0.0) ? -sqrt(norm2) : sqrt(norm2);
        const double vtv = 2.0 * (norm2 - alpha * v[0]); /* |x - alpha e1|^2 */
        v[0] -= alpha;
        if (vtv == 0.0) continue;
        const double beta = 2.0 / vtv; /* H = I - beta v v^T */

        /* p = beta * A22 v */
#pragma omp parallel for schedule(static)
        for (int i = 0; i < len; ++i) {
            const double *row = A + (size_t)(k + 1 + i) * n + (k + 1);
            double s = 0.0;
            for (int j = 0; j < len; ++j) s += row[j] * v[j];
            p[i] = beta * s;
        }
        double vtp = 0.0;
        for (int i = 0; i < len; ++i) vtp += v[i] * p[i];
        const double K = 0.5 * beta * vtp;
        for (int i = 0; i < len; ++i) p[i] -= K * v[i]; /* p is now w = p - K v */

        /* A22 <- A22 - v w^T - w v^T */
#pragma omp parallel for schedule(static)
        for (int i = 0; i < len; ++i) {
            double *row = A + (size_t)(k + 1 + i) * n + (k + 1);
            for (int j = 0; j < len; ++j) row[j] -= v[i] * p[j] + p[i] * v[j];
        }
        /* column / row k of H A H: (alpha, 0, ..., 0) */
        A[(size_t)(k + 1) * n + k] = alpha;
        A[(size_t)k * n + (k + 1)] = alpha;
        for (int i = 1; i < len; ++i) {
            A[(size_t)(k + 1 + i) * n + k] = 0.0;
            A[(size_t)k * n + (k + 1 + i)] = 0.0;
        }
        /* Z <- Z H  (H touches columns k+1 .. n-1) */
#pragma omp parallel for schedule(static)
        for (int i = 0; i < n; ++i) {
            double *row = Z + (size_t)i * n + (k + 1);
            double s = 0.0;
            for (int j = 0; j < len; ++j) s += row[j] * v[j];
            s *= beta;
            for (int j = 0; j < len; ++j) row[j] -= s * v[j];
        }
    }
    for (int i = 0; i < n; ++i) d[i] = A[(size_t)i * n + i];
    for (int i = 0; i + 1 < n; ++i) e[i] = A[(size_t)(i + 1) * n + i];
    if (n > 0) e[n - 1] = 0.0;
    free(v);
    free(p);
}

static int tridiagonal_qr(int n, double *d, double *e, double *Z)
{
    const double eps = 2.220446049250313e-16;
    int hi = n - 1;
    long budget = 60L * n + 200;
    while (hi > 0) {
        /* deflate negligible sub-diagonal entries */
        for (int i = 0; i < hi; ++i)
            if (fabs(e[i]) <= eps * (fabs(d[i]) + fabs(d[i + 1]))) e[i] = 0.0;
        if (e[hi - 1] == 0.0) { --hi; continue; }
        int lo = hi - 1;
        while (lo > 0 && e[lo - 1] != 0.0) --lo;
        if (--budget < 0) return 1;

        /* Wilkinson shift from the trailing 2 x 2 block of the unreduced part */
        const double dl = 0.5 * (d[hi - 1] - d[hi]);
        const double eh = e[hi - 1];
        const double denom = dl + ((dl >= 0.0) ? 1.0 : -1.0) * hypot(dl, eh);
        const double mu = d[hi] - (eh * eh) / denom;

        double x = d[lo] - mu, z = e[lo];
        for (int k = lo; k < hi; ++k) {
            /* rotation G = [c s; -s c] with G [x; z] = [r; 0]; T <- G T G^T */
            const double r = hypot(x, z);
            const double c = (r == 0.0) ? 1.0 : x / r;
            const double s = (r == 0.0) ? 0.0 : z / r;
            if (k > lo) e[k - 1] = r;
            const double a = d[k], b = e[k], g = d[k + 1];
            d[k] = c * c * a + 2.0 * c * s * b + s * s * g;
            d[k + 1] = s * s * a - 2.0 * c * s * b + c * c * g;
            e[k] = c * s * (g - a) + (c * c - s * s) * b;
            x = e[k];
            if (k + 1 < hi) {
                const double h = e[k + 1];
                z = s * h; /* the bulge at (k+2, k) */
                e[k + 1] = c * h;
            }
            /* Z <- Z G^T on columns k, k+1 */
#pragma omp parallel for schedule(static) if (n > 256)
            for (int i = 0; i < n; ++i) {
                double *row = Z + (size_t)i * n;
                const double zk = row[k], zk1 = row[k + 1];
                row[k] = c * zk + s * zk1;
                row[k + 1] = -s * zk + c * zk1;
            }
        }
    }
    return 0;
}

int oracle_eigh_desc(double *A, int n, double *w, double *Z)
{
    double *e = (double *)malloc((size_t)(n > 0 ? n : 1) * sizeof(double));
    householder_tridiagonal(n, A, Z, w, e);
    const int rc = tridiagonal_qr(n, w, e, Z);
    free(e);
    /* selection sort into descending order, swapping eigenvector columns along */
    for (int i = 0; i < n; ++i) {
        int best = i;
        for (int j = i + 1; j < n; ++j)
            if (w[j] > w[best]) best = j;
        if (best != i) {
            const double t = w[i]; w[i] = w[best]; w[best] = t;
            for (int r = 0; r < n; ++r) {
                const double u = Z[(size_t)r * n + i];
                Z[(size_t)r * n + i] = Z[(size_t)r * n + best];
                Z[(size_t)r * n + best] = u;
            }
        }
    }
    return rc;
}

/* ------------------------------------------------------------------------------------
 * Calibration ("one-time SVD", Sec. 3.3, Eq. 7): top-k right singular vectors of the
 * stack, through the Gram matrix.  Outputs V_k (D x k), lambda (k, = sigma_i^2,
 * descending) and trace(G) = |Fstack|_F^2 = sum of all sigma_i^2 (the denominator of
 * the energy criterion, Eq. 6).  Column signs: the entry of largest magnitude in each
 * column is positive (the SVD leaves the sign free).
 * ---------------------------------------------------------------------------------- */
int oracle_calibrate(const double *Fstack, int64_t M, int D, int k, double *Vk,
                     double *lambda, double *trace, double *lambda_all /* D or NULL */)
{
    double *G = (double *)malloc((size_t)D * D * sizeof(double));
    double *Z = (double *)malloc((size_t)D * D * sizeof(double));
    double *w = (double *)malloc((size_t)D * sizeof(double));
    oracle_gram(Fstack, M, D, G);
    double tr = 0.0;
    for (int i = 0; i < D; ++i) tr += G[(size_t)i * D + i];
    const int rc = oracle_eigh_desc(G, D, w, Z);
    for (int j = 0; j < k; ++j) {
        int arg = 0;
        for (int i = 1; i < D; ++i)
            if (fabs(Z[(size_t)i * D + j]) > fabs(Z[(size_t)arg * D + j])) arg = i;
        const double sgn = (Z[(size_t)arg * D + j] < 0.0) ? -1.0 : 1.0;
        for (int i = 0; i < D; ++i) Vk[(size_t)i * k + j] = sgn * Z[(size_t)i * D + j];
        lambda[j] = w[j];
    }
    if (lambda_all) memcpy(lambda_all, w, (size_t)D * sizeof(double));
    *trace = tr;
    free(G); free(Z); free(w);
    return rc;
}

/* ------------------------------------------------------------------------------------
 * Brute-force second route for tiny matrices: one-sided (Hestenes) Jacobi SVD of A
 * itself (m x n, m >= 1).  Plane rotations make the columns of A V mutually orthogonal;
 * their norms are the singular values.  Outputs sigma (n, descending) and V (n x n,
 * column j = right singular vector of sigma[j]).  Returns the number of sweeps used.
 * ---------------------------------------------------------------------------------- */
int oracle_jacobi_svd(const double *A, int m, int n, double *sigma, double *V)
{
    double *W = (double *)malloc((size_t)m * n * sizeof(double));
    memcpy(W, A, (size_t)m * n * sizeof(double));
    for (int i = 0; i < n; ++i)
        for (int j = 0; j < n; ++j) V[(size_t)i * n + j] = (i == j) ? 1.0 : 0.0;
    int sweeps = 0;
    for (; sweeps < 100; ++sweeps) {
        int rotated = 0;
        for (int p = 0; p + 1 < n; ++p)
            for (int q = p + 1; q < n; ++q) {
                double a = 0.0, b = 0.0, g = 0.0;
                for (int i = 0; i < m; ++i) {
                    const double wp = W[(size_t)i * n + p], wq = W[(size_t)i * n + q];
                    a += wp * wp; b += wq * wq; g += wp * wq;
                }
                if (g == 0.0 || fabs(g) <= 1e-15 * sqrt(a * b)) continue;
                rotated = 1;
                const double zeta = (b - a) / (2.0 * g);
                const double t = ((zeta >= 0.0) ? 1.0 : -1.0) / (fabs(zeta) + sqrt(1.0 + zeta * zeta));
                const double c = 1.0 / sqrt(1.0 + t * t), s = c * t;
                for (int i = 0; i < m; ++i) {
                    const double wp = W[(size_t)i * n + p], wq = W[(size_t)i * n + q];
                    W[(size_t)i * n + p] = c * wp - s * wq;
                    W[(size_t)i * n + q] = s * wp + c * wq;
                }
                for (int i = 0; i < n; ++i) {
                    const double vp = V[(size_t)i * n + p], vq = V[(size_t)i * n + q];
                    V[(size_t)i * n + p] = c * vp - s * vq;
                    V[(size_t)i * n + q] = s * vp + c * vq;
                }
            }
        if (!rotated) break;
    }
    for (int j = 0; j < n; ++j) {
        double a = 0.0;
        for (int i = 0; i < m; ++i) a += W[(size_t)i * n + j] * W[(size_t)i * n + j];
        sigma[j] = sqrt(a);
    }
    for (int i = 0; i < n; ++i) { /* sort descending, columns of V along */
        int best = i;
        for (int j = i + 1; j < n; ++j)
            if (sigma[j] > sigma[best]) best = j;
        if (best != i) {
            const double t = sigma[i]; sigma[i] = sigma[best]; sigma[best] = t;
            for (int r = 0; r < n; ++r) {
                const double u = V[(size_t)r * n + i];
                V[(size_t)r * n + i] = V[(size_t)r * n + best];
                V[(size_t)r * n + best] = u;
            }
        }
    }
    free(W);
    return sweeps;
}

/* ------------------------------------------------------------------------------------
 * Rank selection (Eq. 6): the smallest k whose leading eigenvalues hold at least a
 * fraction tau of the total energy trace = sum_i sigma_i^2.  lambda is descending.
 * Returns n if even all n listed eigenvalues fall short.
 * ---------------------------------------------------------------------------------- */
int oracle_rank_for_energy(const double *lambda, int n, double trace, double tau)
{
    double acc = 0.0;
    for (int k = 1; k <= n; ++k) {
        acc += lambda[k - 1];
        if (acc / trace >= tau) return k;
    }
    return n;
}

/* ------------------------------------------------------------------------------------
 * Full step (Sec. 3.3 - 3.5).  Row by row:
 *   c    = V_k^T f            Eq. 8 with Eq. 9: U_k diag(sigma_k) = F V_k (sigma cancels)
 *   r    = f - V_k c          Eq. 9, Eq. 10
 *   chat = c                          on the first full step (the EMA has no history)
 *        = beta chat + (1-beta) c     afterwards, Eq. 11 written on the coefficients
 * C (N x k) and R (N x D) are outputs; Chat (N x k) is updated in place.
 * ---------------------------------------------------------------------------------- */
void oracle_full_step(const double *F, int64_t N, int D, const double *Vk, int k,
                      double beta, int first, double *Chat, double *R, double *C)
{
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        const double *f = F + (size_t)n * D;
        double *c = C + (size_t)n * k;
        double *r = R + (size_t)n * D;
        double *ch = Chat + (size_t)n * k;
        for (int j = 0; j < k; ++j) {
            double s = 0.0;
            for (int d = 0; d < D; ++d) s += f[d] * Vk[(size_t)d * k + j];
            c[j] = s;
        }
        for (int d = 0; d < D; ++d) {
            double s = 0.0;
            for (int j = 0; j < k; ++j) s += c[j] * Vk[(size_t)d * k + j];
            r[d] = f[d] - s;
        }
        for (int j = 0; j < k; ++j) ch[j] = first ? c[j] : beta * ch[j] + (1.0 - beta) * c[j];
    }
}

/* ------------------------------------------------------------------------------------
 * Cached step (Sec. 3.5): the forecast of the principal part is the EMA state, the
 * residual is reused as stored:  fhat = V_k chat + r.
 * ---------------------------------------------------------------------------------- */
void oracle_cached_step(const double *Chat, const double *Vk, const double *R, int64_t N,
                        int D, int k, double *Fhat)
{
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        const double *ch = Chat + (size_t)n * k;
        const double *r = R + (size_t)n * D;
        double *fh = Fhat + (size_t)n * D;
        for (int d = 0; d < D; ++d) {
            double s = 0.0;
            for (int j = 0; j < k; ++j) s += ch[j] * Vk[(size_t)d * k + j];
            fh[d] = s + r[d];
        }
    }
}

/* ------------------------------------------------------------------------------------
 * Full step with a smoothed residual (the ablation of Sec. 4.5, Fig. 4(c): "EMA on both").
 * As oracle_full_step, except that the stored residual is itself an EMA of the residuals of
 * the full steps:
 *   rhat = r                                  on the first full step
 *        = beta_r rhat + (1 - beta_r) r       afterwards          (r = f - V_k c, Eq. 10)
 * beta_r = 0 is the method itself (Sec. 3.5: the residual is reused as it is); beta = 0
 * together with beta_r = 0 is "reuse on both" (Eq. 3).  Rhat (N x D) is updated in place.
 * ---------------------------------------------------------------------------------- */
void oracle_full_step_residual_ema(const double *F, int64_t N, int D, const double *Vk, int k,
                                   double beta, double beta_r, int first, double *Chat,
                                   double *Rhat, double *C)
{
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        const double *f = F + (size_t)n * D;
        double *c = C + (size_t)n * k;
        double *rh = Rhat + (size_t)n * D;
        double *ch = Chat + (size_t)n * k;
        for (int j = 0; j < k; ++j) {
            double s = 0.0;
            for (int d = 0; d < D; ++d) s += f[d] * Vk[(size_t)d * k + j];
            c[j] = s;
        }
        for (int d = 0; d < D; ++d) {
            double s = 0.0;
            for (int j = 0; j < k; ++j) s += c[j] * Vk[(size_t)d * k + j];
            const double r = f[d] - s;
            rh[d] = first ? r : beta_r * rh[d] + (1.0 - beta_r) * r;
        }
        for (int j = 0; j < k; ++j) ch[j] = first ? c[j] : beta * ch[j] + (1.0 - beta) * c[j];
    }
}

/* ------------------------------------------------------------------------------------
 * Other predictors on the principal coefficients (Sec. 5.3, Fig. 4(b)): the paper pairs its
 * decomposition with predictors of the cited caching methods and does not restate them.  Two
 * forecasts from the coefficients of the last order+1 full steps, hist[0] the newest,
 * hist[i] the one i full steps earlier (each n values), for a cached step that lies
 * u = (steps since the last full step) / (steps between full steps) intervals ahead:
 *   backward differences   D^0 = hist[0],  D^i = D^{i-1}(newest) - D^{i-1}(one step earlier)
 *   kind 1 ("taylor")  out = sum_i  u^i / i!  D^i
 *        a Taylor expansion in the step offset whose derivatives are the backward differences
 *        (the form of the cited cache-then-forecast method);
 *   kind 2 ("newton")  out = sum_i  u (u+1) ... (u+i-1) / i!  D^i
 *        Newton's backward-difference formula: the polynomial of degree `order` through the
 *        last order+1 coefficients, evaluated u intervals past the newest.
 * order = 0 is plain reuse of the newest coefficients (Eq. 3) for both kinds.
 * ---------------------------------------------------------------------------------- */
void oracle_forecast(const double *const *hist, int order, int64_t n, double u, int kind, double *out)
{
#pragma omp parallel for schedule(static)
    for (int64_t e = 0; e < n; ++e) {
        double d[8];                       /* d[j] = current difference anchored j steps back */
        for (int j = 0; j <= order; ++j) d[j] = hist[j][e];
        double acc = d[0], coef = 1.0;
        for (int i = 1; i <= order; ++i) {
            for (int j = 0; j + i <= order; ++j) d[j] = d[j] - d[j + 1];   /* now D^i at j steps back */
            coef *= (kind == 1 ? u : (u + (double)(i - 1))) / (double)i;
            acc += coef * d[0];
        }
        out[e] = acc;
    }
}

/* ------------------------------------------------------------------------------------
 * Left factors of Eq. 8:  U = F V_k diag(sigma_k)^{-1} = C diag(sigma_k)^{-1}, sigma_i the
 * cached singular values (square roots of the Gram eigenvalues, Eq. 7).  A column whose
 * sigma is zero carries no energy; it is set to zero instead of dividing.
 * ---------------------------------------------------------------------------------- */
void oracle_left_factors(const double *C, const double *sigma, int64_t N, int k, double *U)
{
    for (int64_t n = 0; n < N; ++n)
        for (int j = 0; j < k; ++j)
            U[(size_t)n * k + j] = sigma[j] > 0.0 ? C[(size_t)n * k + j] / sigma[j] : 0.0;
}

#ifdef _OPENMP
#include <omp.h>
int oracle_threads(void) { return omp_get_max_threads(); }
void oracle_set_threads(int n) { omp_set_num_threads(n); }
#else
int oracle_threads(void) { return 1; }
void oracle_set_threads(int n) { (void)n; }
#endif
