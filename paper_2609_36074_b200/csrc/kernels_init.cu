// Data-informed starting factor (the paper's appendix "Additional Computation Details", paragraph
// "Initialization"):  V = X-hat X-hat^T Z,  V = Q R,  U0 = Proj_Omega(Q), with the orthonormalization as
// Cholesky QR in feature space:
//   M = X-hat^T Z (d x r),  C = X-hat^T X-hat (d x d),  M^T C M = R^T R,  B = M R^{-1},  Q = X-hat B,
//   U0 = sqrt(K) [Q]_+ / ||[Q]_+||_F.
// The two large products are the iteration's own contractions on the generic kernels: M and C are first
// products (C with X-hat in the factor's place), and Q = X-hat B with the clamp, ||[Q]_+||_F^2 and the column
// sums is the fused second product evaluated at u = 0, 2 alpha = 1, ybar = 0, s = 0, whose scalar step then
// yields the multiplier sqrt(K) / ||[Q]_+||_F and p = U0^T 1.  This file adds the FP64 pieces in between:
// the reduction of the split-K partials without rounding to FP32, and the r x r factorization with the
// triangular solve (one CTA; r <= d <= a few hundred in the intended use, cost O(d^2 r + r^3)).
#include "nlr_common.cuh"
#include "device_utils.cuh"

namespace gemnlr {

// out[e] = sum_g part[g][e] in ascending g (FP64, fixed order).
__global__ void __launch_bounds__(256)
k_red_f64(const double* __restrict__ part, int g, int64_t count, double* __restrict__ out)
{
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < count; e += (int64_t)gridDim.x * blockDim.x) {
        double v = 0.0;
        for (int b = 0; b < g; ++b) v += part[(size_t)b * count + e];
        out[e] = v;
    }
}

void launch_red_f64(const Problem& pb, const double* part, int g, int64_t count, double* out)
{
    k_red_f64<<<kSMs, 256, 0, pb.stream>>>(part, g, count, out);
    pb.count(1);
}

// One CTA.  M (d x r), C (d x d) FP64 row-major in; T = C M, G = M^T T, Cholesky G = R^T R in place (upper
// triangle of G), B = M R^{-1} written as FP32 into theta (d x r row-major, what the second product reads).
// A pivot that is not positive relative to the largest diagonal entry of G (the sample has no full column
// rank, or is too ill-conditioned for Cholesky QR) raises GEM_NLR_E_BREAKDOWN and stops the sequence.
// On success the pending multiplier is set to 0, which makes the following fused second product see u = 0.
__global__ void __launch_bounds__(256)
k_init_small(const double* __restrict__ M, const double* __restrict__ C, double* __restrict__ T,
             double* __restrict__ G, float* __restrict__ theta, Ctl* __restrict__ ctl, int d, int r)
{
    __shared__ double s_piv;
    __shared__ int s_bad;
    const int tid = threadIdx.x, nt = blockDim.x;
    for (int e = tid; e < d * r; e += nt) {
        const int i = e / r, j = e % r;
        double v = 0.0;
        for (int k = 0; k < d; ++k) v = fma(C[(size_t)i * d + k], M[(size_t)k * r + j], v);
        T[e] = v;
    }
    __syncthreads();
    for (int e = tid; e < r * r; e += nt) {
        const int i = e / r, j = e % r;
        if (j < i) continue;                                  // upper triangle; G is symmetric
        double v = 0.0;
        for (int k = 0; k < d; ++k) v = fma(M[(size_t)k * r + i], T[(size_t)k * r + j], v);
        G[e] = v;
    }
    __syncthreads();
    double gmax = 0.0;
    for (int i = 0; i < r; ++i) gmax = fmax(gmax, G[(size_t)i * r + i]);     // every thread: the same value
    if (tid == 0) s_bad = 0;
    __syncthreads();
    // right-looking Cholesky on the upper triangle: row k of R, then the trailing update
    for (int k = 0; k < r; ++k) {
        if (tid == 0) {
            const double piv = G[(size_t)k * r + k];
            if (!(piv > 1e-13 * gmax) || !isfinite(piv)) s_bad = 1;
            s_piv = sqrt(piv > 0.0 ? piv : 1.0);
        }
        __syncthreads();
        if (s_bad) break;
        const double rkk = s_piv;
        for (int j = k + tid; j < r; j += nt) G[(size_t)k * r + j] = (j == k) ? rkk : G[(size_t)k * r + j] / rkk;
        __syncthreads();
        const int m = r - k - 1;
        for (int e = tid; e < m * m; e += nt) {
            const int i = k + 1 + e / m, j = k + 1 + e % m;
            if (j >= i) G[(size_t)i * r + j] -= G[(size_t)k * r + i] * G[(size_t)k * r + j];
        }
        __syncthreads();
    }
    if (s_bad) {
        if (tid == 0) { ctl->status = GEM_NLR_E_BREAKDOWN; ctl->stopped = 1; }
        return;
    }
    // B R = M, one row of B per thread: b_j = (m_j - sum_{k<j} b_k R_kj) / R_jj; T is reused for B in FP64
    for (int i = tid; i < d; i += nt) {
        double* b = T + (size_t)i * r;
        for (int j = 0; j < r; ++j) {
            double v = M[(size_t)i * r + j];
            for (int k = 0; k < j; ++k) v -= b[k] * G[(size_t)k * r + j];
            b[j] = v / G[(size_t)j * r + j];
        }
        for (int j = 0; j < r; ++j) theta[(size_t)i * r + j] = (float)b[j];
    }
    if (tid == 0) ctl->c_f = 0.0f;
}

// Enqueues the whole sequence.  On entry the factor buffer holds Z; on completion it holds the unnormalized
// [Q]_+ with the multiplier pending (the caller runs the tail kernel to materialize U0) and p = U0^T 1.
// Returns false when the split-K partial area cannot hold one d x d record.
bool launch_range_init(const Problem& pb)
{
    const auto& P = pb.P;
    const auto& L = pb.L;
    const int d = P.d, r = P.r;
    double* M64 = pb.init();
    double* C64 = M64 + (size_t)d * r;
    double* T64 = C64 + (size_t)d * d;
    double* G64 = T64 + (size_t)d * r;
    // M = X-hat^T Z
    {
        dim3 g1(L.g1x, L.g1y_d * L.g1y_r);
        launch_pass1_partials(pb, pb.X, pb.U, d, r, L.g1y_r, g1);
        k_red_f64<<<kSMs, 256, 0, pb.stream>>>(pb.part1(), L.g1x, (int64_t)d * r, M64);
        pb.count(1);
    }
    // C = X-hat^T X-hat: the same kernel with X-hat in the factor's place (r := d, row pitch d)
    {
        const size_t cap = L.part1_bytes / sizeof(double) / ((size_t)d * d);
        if (cap < 1) return false;
        const int gx = (int)(cap < (size_t)L.g1x ? cap : (size_t)L.g1x);
        dim3 g1(gx, L.g1y_d * L.g1y_d);
        launch_pass1_partials(pb, pb.X, pb.X, d, d, L.g1y_d, g1);
        k_red_f64<<<kSMs, 256, 0, pb.stream>>>(pb.part1(), gx, (int64_t)d * d, C64);
        pb.count(1);
    }
    k_init_small<<<1, 256, 0, pb.stream>>>(M64, C64, T64, G64, pb.theta(), pb.ctl(), d, r);
    pb.count(1);
    // Q = X-hat B through the fused second product at u = 0 (multiplier 0), 2 alpha = 1, ybar = 0, s = 0
    cudaMemsetAsync(pb.ybar(), 0, sizeof(float) * (size_t)P.n, pb.stream);
    cudaMemsetAsync(pb.alpha_s(), 0, sizeof(float) * (size_t)r, pb.stream);
    cudaMemsetAsync(pb.p(), 0, sizeof(float) * (size_t)r, pb.stream);
    launch_generic_pass2_alpha(pb, 0.5f);
    launch_fin2(pb, L.g2x, L.g2y, G2_RT);
    return true;
}

}  // namespace gemnlr
