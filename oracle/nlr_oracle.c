/*
 * CPU oracle for the spectrally normalized nonnegative low-rank (NLR) K-means
 * iteration ("GEM iteration").
 *
 * THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, step-by-step restatement
 * of the method, used only to check the CUDA library and to be timed as a
 * reported CPU baseline.  It shares no code with the CUDA path and nothing in
 * the product may call it.
 *
 * Precision follows the paper's device-buffer table: every buffer (X-hat, U,
 * Theta, q, y/sqrt(n), y-bar, p, s) is FP32; every sum is accumulated in FP64
 * and rounded once into its buffer; the three statistics a, b, h stay FP64.
 * The paper does not fix the evaluation order of the entrywise FP32 update, so
 * it is evaluated in FP64 and rounded once.
 *
 * Rows are split over OpenMP threads in contiguous static chunks; per-thread
 * FP64 partial sums are combined in thread-index order, so a run is
 * reproducible for a fixed thread count.  There is no blocking, fusion or
 * reordering beyond that.
 *
 * Parity pins (tests marked "not gpu"): finite differences of the objective,
 * the movement identity against the direct norm, one step of the unnormalized
 * augmented-Lagrangian method written with the explicit n x n matrix, closed
 * forms on planted assignments, the invariance of X-hat under affine rescaling,
 * library eigenvalues, and brute-force exact K-means on n <= 12.
 * Unpinned by the paper (fixed by this build only): the hyper-parameter values
 * and the distribution of the starting factor -- they are inputs here.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t t;          /* index of the iteration just taken */
    int32_t dual;       /* 1 if the dual-ascent gate fired */
    int32_t stop;       /* 1 if the stopping test fired */
    int32_t status;     /* 0 ok, -4 normalization breakdown, -5 non-finite statistic */
    double a, b, h;     /* ||W||_F^2, ||U_prev||_F^2, <W, U_prev> */
    double c;           /* FP64 value of the FP32 multiplier */
    double Delta;       /* clamped squared movement estimate */
    double delta_hat;   /* sqrt(Delta / K) */
    double rho;         /* ||q||_2 / sqrt(n) of the new iterate */
    double fhat;        /* normalized objective at the iterate the step started from */
} nlr_oracle_info;

static int n_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

int nlr_oracle_threads(void) { return n_threads(); }

static void chunk(int64_t n, int nt, int tid, int64_t *lo, int64_t *hi)
{
    int64_t per = n / nt, rem = n % nt;
    *lo = tid * per + (tid < rem ? tid : rem);
    *hi = *lo + per + (tid < rem ? 1 : 0);
}

/* ------------------------------------------------------------------------- */
/* Data normalization (Section 3: X_c = X - 1 xbar^T, a = ||X_c||_2,          */
/* X-hat = X_c / a).                                                          */
/* ------------------------------------------------------------------------- */

void nlr_oracle_col_mean(const float *X, int64_t n, int32_t d, double *mean)
{
    int nt = n_threads();
    double *part = (double *)calloc((size_t)nt * d, sizeof(double));
#pragma omp parallel num_threads(nt)
    {
#ifdef _OPENMP
        int tid = omp_get_thread_num();
#else
        int tid = 0;
#endif
        int64_t lo, hi;
        chunk(n, nt, tid, &lo, &hi);
        double *m = part + (size_t)tid * d;
        for (int64_t i = lo; i < hi; ++i)
            for (int32_t j = 0; j < d; ++j) m[j] += (double)X[i * d + j];
    }
    for (int32_t j = 0; j < d; ++j) {
        double s = 0.0;
        for (int t = 0; t < nt; ++t) s += part[(size_t)t * d + j];
        mean[j] = s / (double)n;
    }
    free(part);
}

/* G = X_c^T X_c (d x d, FP64), X_c = X - 1 mean^T; mean may be NULL (no centering). */
void nlr_oracle_gram(const float *X, int64_t n, int32_t d, const double *mean, double *G)
{
    int nt = n_threads();
    size_t dd = (size_t)d * d;
    double *part = (double *)calloc((size_t)nt * dd, sizeof(double));
#pragma omp parallel num_threads(nt)
    {
#ifdef _OPENMP
        int tid = omp_get_thread_num();
#else
        int tid = 0;
#endif
        int64_t lo, hi;
        chunk(n, nt, tid, &lo, &hi);
        double *g = part + (size_t)tid * dd;
        double *row = (double *)malloc(sizeof(double) * d);
        for (int64_t i = lo; i < hi; ++i) {
            for (int32_t j = 0; j < d; ++j)
                row[j] = (double)X[i * d + j] - (mean ? mean[j] : 0.0);
            for (int32_t j = 0; j < d; ++j) {
                double xj = row[j];
                double *gj = g + (size_t)j * d;
                for (int32_t k = j; k < d; ++k) gj[k] += xj * row[k];
            }
        }
        free(row);
    }
    for (int32_t j = 0; j < d; ++j)
        for (int32_t k = j; k < d; ++k) {
            double s = 0.0;
            for (int t = 0; t < nt; ++t) s += part[(size_t)t * dd + (size_t)j * d + k];
            G[(size_t)j * d + k] = s;
            G[(size_t)k * d + j] = s;
        }
    free(part);
}

/* Largest eigenvalue of a symmetric d x d matrix by cyclic Jacobi rotations. */
double nlr_oracle_sym_eig_max(const double *Gin, int32_t d)
{
    size_t dd = (size_t)d * d;
    double *A = (double *)malloc(sizeof(double) * dd);
    memcpy(A, Gin, sizeof(double) * dd);
    for (int sweep = 0; sweep < 100; ++sweep) {
        double off = 0.0, diag = 0.0;
        for (int32_t p = 0; p < d; ++p) {
            diag += A[(size_t)p * d + p] * A[(size_t)p * d + p];
            for (int32_t q = p + 1; q < d; ++q) off += A[(size_t)p * d + q] * A[(size_t)p * d + q];
        }
        if (off <= 1e-32 * (diag + off)) break;
        for (int32_t p = 0; p < d - 1; ++p)
            for (int32_t q = p + 1; q < d; ++q) {
                double apq = A[(size_t)p * d + q];
                if (apq == 0.0) continue;
                double app = A[(size_t)p * d + p], aqq = A[(size_t)q * d + q];
                double theta = (aqq - app) / (2.0 * apq);
                double t = (theta >= 0.0 ? 1.0 : -1.0) / (fabs(theta) + sqrt(theta * theta + 1.0));
                double c = 1.0 / sqrt(t * t + 1.0), s = t * c;
                for (int32_t k = 0; k < d; ++k) {   /* columns p, q */
                    double akp = A[(size_t)k * d + p], akq = A[(size_t)k * d + q];
                    A[(size_t)k * d + p] = c * akp - s * akq;
                    A[(size_t)k * d + q] = s * akp + c * akq;
                }
                for (int32_t k = 0; k < d; ++k) {   /* rows p, q */
                    double apk = A[(size_t)p * d + k], aqk = A[(size_t)q * d + k];
                    A[(size_t)p * d + k] = c * apk - s * aqk;
                    A[(size_t)q * d + k] = s * apk + c * aqk;
                }
            }
    }
    double best = A[0];
    for (int32_t p = 1; p < d; ++p)
        if (A[(size_t)p * d + p] > best) best = A[(size_t)p * d + p];
    free(A);
    return best;
}

/* a = ||X_c||_2 = sqrt(lambda_max(X_c^T X_c)); writes the column mean (zeros if !center). */
double nlr_oracle_spectral_norm(const float *X, int64_t n, int32_t d, int32_t center, double *mean)
{
    if (center) nlr_oracle_col_mean(X, n, d, mean);
    else memset(mean, 0, sizeof(double) * d);
    double *G = (double *)malloc(sizeof(double) * (size_t)d * d);
    nlr_oracle_gram(X, n, d, center ? mean : NULL, G);
    double lam = nlr_oracle_sym_eig_max(G, d);
    free(G);
    return sqrt(lam > 0.0 ? lam : 0.0);
}

/* X-hat = FP32((X - 1 mean^T) / a). */
void nlr_oracle_normalize(const float *X, int64_t n, int32_t d, const double *mean, double a,
                          float *Xhat)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i)
        for (int32_t j = 0; j < d; ++j)
            Xhat[i * d + j] = (float)(((double)X[i * d + j] - mean[j]) / a);
}

/* ------------------------------------------------------------------------- */
/* Constraint vectors (Section 4.1): p = U^T 1, q = U p - 1 = g(U).           */
/* ------------------------------------------------------------------------- */

static void col_sums(const float *U, int64_t n, int32_t r, double *p64)
{
    int nt = n_threads();
    double *part = (double *)calloc((size_t)nt * r, sizeof(double));
#pragma omp parallel num_threads(nt)
    {
#ifdef _OPENMP
        int tid = omp_get_thread_num();
#else
        int tid = 0;
#endif
        int64_t lo, hi;
        chunk(n, nt, tid, &lo, &hi);
        double *pp = part + (size_t)tid * r;
        for (int64_t i = lo; i < hi; ++i)
            for (int32_t j = 0; j < r; ++j) pp[j] += (double)U[i * r + j];
    }
    for (int32_t j = 0; j < r; ++j) {
        double s = 0.0;
        for (int t = 0; t < nt; ++t) s += part[(size_t)t * r + j];
        p64[j] = s;
    }
    free(part);
}

void nlr_oracle_residual(const float *U, int64_t n, int32_t r, float *p, float *q)
{
    double *p64 = (double *)malloc(sizeof(double) * r);
    col_sums(U, n, r, p64);
    for (int32_t j = 0; j < r; ++j) p[j] = (float)p64[j];
    free(p64);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        double s = 0.0;
        for (int32_t j = 0; j < r; ++j) s += (double)U[i * r + j] * (double)p[j];
        q[i] = (float)(s - 1.0);
    }
}

/* Theta = X-hat^T U (d x r), FP64 accumulation; Theta64 receives the unrounded sums. */
static void theta_product(const float *Xhat, const float *U, int64_t n, int32_t d, int32_t r,
                          double *Theta64)
{
    int nt = n_threads();
    size_t dr = (size_t)d * r;
    double *part = (double *)calloc((size_t)nt * dr, sizeof(double));
#pragma omp parallel num_threads(nt)
    {
#ifdef _OPENMP
        int tid = omp_get_thread_num();
#else
        int tid = 0;
#endif
        int64_t lo, hi;
        chunk(n, nt, tid, &lo, &hi);
        double *th = part + (size_t)tid * dr;
        double *urow = (double *)malloc(sizeof(double) * r);
        for (int64_t i = lo; i < hi; ++i) {
            for (int32_t k = 0; k < r; ++k) urow[k] = (double)U[i * r + k];
            for (int32_t j = 0; j < d; ++j) {
                double x = (double)Xhat[i * d + j];
                double *tj = th + (size_t)j * r;
                for (int32_t k = 0; k < r; ++k) tj[k] += x * urow[k];
            }
        }
        free(urow);
    }
#pragma omp parallel for schedule(static)
    for (int64_t e = 0; e < (int64_t)dr; ++e) {
        double s = 0.0;
        for (int t = 0; t < nt; ++t) s += part[(size_t)t * dr + e];
        Theta64[e] = s;
    }
    free(part);
}

void nlr_oracle_theta(const float *Xhat, const float *U, int64_t n, int32_t d, int32_t r,
                      float *Theta)
{
    size_t dr = (size_t)d * r;
    double *T64 = (double *)malloc(sizeof(double) * dr);
    theta_product(Xhat, U, n, d, r, T64);
    for (size_t e = 0; e < dr; ++e) Theta[e] = (float)T64[e];
    free(T64);
}

/*
 * Normalized objective (Eq. "normalized"), written with the stored quantities:
 *   f-hat_y(U) = <A-hat, U U^T> + y^T h + (beta/2) ||h||^2,   h = g(U)/sqrt(n)
 *              = -||X-hat^T U||_F^2 + ytilde^T q + (gamma/2) ||q||^2,
 * with ytilde = y/sqrt(n), gamma = beta/n, q = g(U) = U U^T 1 - 1.
 * Everything is evaluated in FP64 from the FP32 inputs (no intermediate rounding).
 */
static double objective_from_theta(const double *Theta64, int32_t d, int32_t r, const float *U,
                                   const float *ytilde, int64_t n, double beta)
{
    double t2 = 0.0;
    for (size_t e = 0; e < (size_t)d * r; ++e) t2 += Theta64[e] * Theta64[e];
    double *p64 = (double *)malloc(sizeof(double) * r);
    col_sums(U, n, r, p64);
    int nt = n_threads();
    double *yq = (double *)calloc(nt, sizeof(double)), *qq = (double *)calloc(nt, sizeof(double));
#pragma omp parallel num_threads(nt)
    {
#ifdef _OPENMP
        int tid = omp_get_thread_num();
#else
        int tid = 0;
#endif
        int64_t lo, hi;
        chunk(n, nt, tid, &lo, &hi);
        double syq = 0.0, sqq = 0.0;
        for (int64_t i = lo; i < hi; ++i) {
            double s = 0.0;
            for (int32_t j = 0; j < r; ++j) s += (double)U[i * r + j] * p64[j];
            double qi = s - 1.0;
            syq += (double)ytilde[i] * qi;
            sqq += qi * qi;
        }
        yq[tid] = syq;
        qq[tid] = sqq;
    }
    double syq = 0.0, sqq = 0.0;
    for (int t = 0; t < nt; ++t) { syq += yq[t]; sqq += qq[t]; }
    free(yq); free(qq); free(p64);
    double gamma = beta / (double)n;
    return -t2 + syq + 0.5 * gamma * sqq;
}

double nlr_oracle_objective(const float *Xhat, const float *U, const float *ytilde, int64_t n,
                            int32_t d, int32_t r, double beta)
{
    size_t dr = (size_t)d * r;
    double *T64 = (double *)malloc(sizeof(double) * dr);
    theta_product(Xhat, U, n, d, r, T64);
    double f = objective_from_theta(T64, d, r, U, ytilde, n, beta);
    free(T64);
    return f;
}

/* ------------------------------------------------------------------------- */
/* One iteration of Algorithm 1, with the argument conventions of Algorithm 2.*/
/*                                                                            */
/* State in/out: U (n x r, in Omega), ytilde = y/sqrt(n) (n), p (r), q (n).   */
/* Buffers out:  Theta (d x r), ybar (n), s (r).                              */
/* Returns info->status (0, or -4 on normalization breakdown, in which case   */
/* U holds the unscaled W, as in the paper's loop which breaks before the     */
/* scaling call).                                                             */
/* ------------------------------------------------------------------------- */
int nlr_oracle_step(const float *Xhat, int64_t n, int32_t d, int32_t r, int32_t K, double alpha,
                    double beta, double eps_d, double eps_c, int32_t T_min, int32_t t, float *U,
                    float *ytilde, float *p, float *q, float *Theta, float *ybar, float *s,
                    nlr_oracle_info *info)
{
    const double gamma = beta / (double)n;           /* stored penalty: beta / n */
    const size_t dr = (size_t)d * r;
    int nt = n_threads();
    memset(info, 0, sizeof(*info));
    info->t = t;

    /* (a) Theta = X-hat^T U */
    double *T64 = (double *)malloc(sizeof(double) * dr);
    theta_product(Xhat, U, n, d, r, T64);
    for (size_t e = 0; e < dr; ++e) Theta[e] = (float)T64[e];
    info->fhat = objective_from_theta(T64, d, r, U, ytilde, n, beta);
    free(T64);

    /* (b) ybar = ytilde + gamma q ;  s = U^T ybar */
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) ybar[i] = (float)((double)ytilde[i] + gamma * (double)q[i]);
    {
        double *part = (double *)calloc((size_t)nt * r, sizeof(double));
#pragma omp parallel num_threads(nt)
        {
#ifdef _OPENMP
            int tid = omp_get_thread_num();
#else
            int tid = 0;
#endif
            int64_t lo, hi;
            chunk(n, nt, tid, &lo, &hi);
            double *sp = part + (size_t)tid * r;
            for (int64_t i = lo; i < hi; ++i) {
                double yb = (double)ybar[i];
                for (int32_t j = 0; j < r; ++j) sp[j] += (double)U[i * r + j] * yb;
            }
        }
        for (int32_t j = 0; j < r; ++j) {
            double acc = 0.0;
            for (int tt = 0; tt < nt; ++tt) acc += part[(size_t)tt * r + j];
            s[j] = (float)acc;
        }
        free(part);
    }

    /* (c) W = [U + 2 alpha X-hat Theta - alpha (ybar p^T + 1 s^T)]_+ in place, with
     *     a = sum w^2, b = sum u^2, h = sum w u in FP64 (Eq. "entrywise-fusion",
     *     Eq. "fused-statistics"). */
    double *Th = (double *)malloc(sizeof(double) * dr);
    for (size_t e = 0; e < dr; ++e) Th[e] = (double)Theta[e];
    double *sa = (double *)calloc(nt, sizeof(double));
    double *sb = (double *)calloc(nt, sizeof(double));
    double *sh = (double *)calloc(nt, sizeof(double));
#pragma omp parallel num_threads(nt)
    {
#ifdef _OPENMP
        int tid = omp_get_thread_num();
#else
        int tid = 0;
#endif
        int64_t lo, hi;
        chunk(n, nt, tid, &lo, &hi);
        double *acc = (double *)malloc(sizeof(double) * r);
        double la = 0.0, lb = 0.0, lh = 0.0;
        for (int64_t i = lo; i < hi; ++i) {
            for (int32_t k = 0; k < r; ++k) acc[k] = 0.0;
            for (int32_t j = 0; j < d; ++j) {
                double x = (double)Xhat[i * d + j];
                const double *tj = Th + (size_t)j * r;
                for (int32_t k = 0; k < r; ++k) acc[k] += x * tj[k];
            }
            double yb = (double)ybar[i];
            for (int32_t k = 0; k < r; ++k) {
                double u = (double)U[i * r + k];
                double v = u + 2.0 * alpha * acc[k] - alpha * yb * (double)p[k] - alpha * (double)s[k];
                float w = (float)(v > 0.0 ? v : 0.0);
                double wd = (double)w;
                la += wd * wd;
                lb += u * u;
                lh += wd * u;
                U[i * r + k] = w;
            }
        }
        sa[tid] = la; sb[tid] = lb; sh[tid] = lh;
        free(acc);
    }
    free(Th);
    double a = 0.0, b = 0.0, h = 0.0;
    for (int tt = 0; tt < nt; ++tt) { a += sa[tt]; b += sb[tt]; h += sh[tt]; }
    free(sa); free(sb); free(sh);
    info->a = a; info->b = b; info->h = h;

    /* (d) projection: nu = sqrt(a); breakdown if nu <= 1e-20; c_f = FP32(sqrt(K)/nu); U <- c_f W */
    if (!isfinite(a) || !isfinite(b) || !isfinite(h)) { info->status = -5; return -5; }
    double nu = sqrt(a);
    if (nu <= 1e-20) { info->status = -4; return -4; }
    float c_f = (float)(sqrt((double)K) / nu);
    double c = (double)c_f;
    info->c = c;
#pragma omp parallel for schedule(static)
    for (int64_t e = 0; e < n * (int64_t)r; ++e) U[e] = c_f * U[e];

    /* (e) movement estimate (Eq. "movement-estimate") and dual gate */
    double Delta = c * c * a + b - 2.0 * c * h;
    if (Delta < 0.0) Delta = 0.0;
    info->Delta = Delta;
    info->delta_hat = sqrt(Delta) / sqrt((double)K);
    int dual = Delta < eps_d * eps_d * (double)K;
    info->dual = dual;

    /* (f) updated residual from the new U */
    nlr_oracle_residual(U, n, r, p, q);

    /* (g) conditional dual ascent, feasibility, stopping test */
    if (dual) {
#pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < n; ++i)
            ytilde[i] = (float)((double)ytilde[i] + gamma * (double)q[i]);
    }
    double *part = (double *)calloc(nt, sizeof(double));
#pragma omp parallel num_threads(nt)
    {
#ifdef _OPENMP
        int tid = omp_get_thread_num();
#else
        int tid = 0;
#endif
        int64_t lo, hi;
        chunk(n, nt, tid, &lo, &hi);
        double acc = 0.0;
        for (int64_t i = lo; i < hi; ++i) acc += (double)q[i] * (double)q[i];
        part[tid] = acc;
    }
    double qq = 0.0;
    for (int tt = 0; tt < nt; ++tt) qq += part[tt];
    free(part);
    info->rho = sqrt(qq) / sqrt((double)n);
    info->stop = dual && info->delta_hat < eps_c && info->rho < eps_c && (t + 1 >= T_min);
    return 0;
}

/*
 * Algorithm 1 as a loop: y = 0, initial p and q, then up to T iterations.
 * ytilde must hold the starting dual (zeros for a fresh run).  Returns the
 * number of iterations taken in *iters; `last` describes the final one.
 */
int nlr_oracle_run(const float *Xhat, int64_t n, int32_t d, int32_t r, int32_t K, double alpha,
                   double beta, double eps_d, double eps_c, int32_t T, int32_t T_min, float *U,
                   float *ytilde, nlr_oracle_info *last, int32_t *iters)
{
    float *p = (float *)malloc(sizeof(float) * r), *s = (float *)malloc(sizeof(float) * r);
    float *q = (float *)malloc(sizeof(float) * n), *ybar = (float *)malloc(sizeof(float) * n);
    float *Theta = (float *)malloc(sizeof(float) * (size_t)d * r);
    nlr_oracle_residual(U, n, r, p, q);
    int rc = 0;
    int32_t t = 0;
    memset(last, 0, sizeof(*last));
    for (; t < T; ++t) {
        rc = nlr_oracle_step(Xhat, n, d, r, K, alpha, beta, eps_d, eps_c, T_min, t, U, ytilde, p, q,
                             Theta, ybar, s, last);
        if (rc != 0) { break; }
        if (last->stop) { ++t; break; }
    }
    *iters = t;
    free(p); free(s); free(q); free(ybar); free(Theta);
    return rc;
}

/* Row-argmax read-out: lowest index among ties; an all-zero row gets label 0. */
void nlr_oracle_labels(const float *U, int64_t n, int32_t r, int32_t *labels)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        int32_t best = 0;
        float bv = U[i * r];
        for (int32_t j = 1; j < r; ++j)
            if (U[i * r + j] > bv) { bv = U[i * r + j]; best = j; }
        labels[i] = best;
    }
}

/* K-means cost of a labelling (Eq. "partition", left-hand form): sum_k sum_{i in G_k} ||x_i - mean_k||^2. */
double nlr_oracle_kmeans_cost(const float *X, int64_t n, int32_t d, const int32_t *labels, int32_t K)
{
    double *mean = (double *)calloc((size_t)K * d, sizeof(double));
    int64_t *cnt = (int64_t *)calloc(K, sizeof(int64_t));
    for (int64_t i = 0; i < n; ++i) {
        int32_t k = labels[i];
        cnt[k]++;
        for (int32_t j = 0; j < d; ++j) mean[(size_t)k * d + j] += (double)X[i * d + j];
    }
    for (int32_t k = 0; k < K; ++k)
        if (cnt[k] > 0)
            for (int32_t j = 0; j < d; ++j) mean[(size_t)k * d + j] /= (double)cnt[k];
    double J = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        int32_t k = labels[i];
        for (int32_t j = 0; j < d; ++j) {
            double df = (double)X[i * d + j] - mean[(size_t)k * d + j];
            J += df * df;
        }
    }
    free(mean); free(cnt);
    return J;
}
