// Setup of the normalized model (Section 3): X_c = X - 1 xbar^T, a = ||X_c||_2, X-hat = X_c / a.
// The paper does not say how a is computed; here X_c^T X_c is applied implicitly to a unit vector,
// one streaming pass over X per application:  w = sum_i z_i (x_i - xbar),  z_i = (x_i - xbar) . v.
// The host combines the applications (Krylov / Lanczos form of the power iteration, see below).
// All sums are FP64 and combined in a fixed order.
#include "nlr_common.cuh"
#include "device_utils.cuh"
#include <math.h>
#include <vector>

namespace gemnlr {

// Column sums: each CTA owns a contiguous row chunk; thread t handles column (t % cpp) of the
// rows (t / cpp) + k * rpp of the chunk.  part[blockIdx][j].
__global__ void __launch_bounds__(256)
k_colmean(const float* __restrict__ X, int64_t n, int d, double* __restrict__ part)
{
    __shared__ double sm[256];
    const int cpp = d < 256 ? d : 256;
    const int rpp = 256 / cpp;
    const int jt = threadIdx.x % cpp, rt = threadIdx.x / cpp;
    const int64_t rows_per = (n + gridDim.x - 1) / gridDim.x;
    const int64_t r_lo = (int64_t)blockIdx.x * rows_per;
    const int64_t r_hi = (r_lo + rows_per < n) ? r_lo + rows_per : n;
    for (int c0 = 0; c0 < d; c0 += cpp) {
        const int col = c0 + jt;
        double acc = 0.0;
        if (rt < rpp && col < d)
            for (int64_t row = r_lo + rt; row < r_hi; row += rpp) acc += (double)X[row * d + col];
        __syncthreads();
        sm[threadIdx.x] = acc;
        __syncthreads();
        if (threadIdx.x < cpp && col < d) {
            double v = 0.0;
            for (int k = 0; k < rpp; ++k) v += sm[k * cpp + threadIdx.x];
            part[(size_t)blockIdx.x * d + col] = v;
        }
    }
}

__global__ void k_colmean_fin(const double* __restrict__ part, int g, int d, int64_t n,
                              double* __restrict__ mean)
{
    for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < d; j += gridDim.x * blockDim.x) {
        double v = 0.0;
        for (int b = 0; b < g; ++b) v += part[(size_t)b * d + j];
        mean[j] = v / (double)n;
    }
}

// One power-iteration pass: warp per row, lanes stride the columns; per-warp FP64 column
// accumulators live in shared memory ([warps][d]).  part[blockIdx][j] = partial w_j.
constexpr int PI_WARPS = 8;

__global__ void __launch_bounds__(PI_WARPS * 32)
k_pi_pass(const float* __restrict__ X, int64_t n, int d, const double* __restrict__ mean,
          const double* __restrict__ v, double* __restrict__ part)
{
    extern __shared__ double smd[];       // [PI_WARPS][d] accumulators, then [d] v, [d] mean
    double* sv = smd + (size_t)PI_WARPS * d;
    double* smean = sv + d;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    double* acc = smd + (size_t)warp * d;
    for (int j = threadIdx.x; j < d; j += blockDim.x) { sv[j] = v[j]; smean[j] = mean[j]; }
    for (int j = lane; j < d; j += 32) acc[j] = 0.0;
    __syncthreads();
    const int64_t stride = (int64_t)gridDim.x * PI_WARPS;
    for (int64_t row = (int64_t)blockIdx.x * PI_WARPS + warp; row < n; row += stride) {
        const float* x = X + row * d;
        double z = 0.0;
        for (int j = lane; j < d; j += 32) z = fma((double)x[j] - smean[j], sv[j], z);
        z = warp_sum(z);
        for (int j = lane; j < d; j += 32) acc[j] = fma(z, (double)x[j] - smean[j], acc[j]);
    }
    __syncthreads();
    for (int j = threadIdx.x; j < d; j += blockDim.x) {
        double t = 0.0;
        for (int w = 0; w < PI_WARPS; ++w) t += smd[(size_t)w * d + j];
        part[(size_t)blockIdx.x * d + j] = t;
    }
}

// Same pass for d = 4 LPR NCH (LPR a power of two <= 32): LPR lanes share a row, each lane owns NCH
// 16-byte chunks (columns 4 (sub + k LPR) .. +3), so a warp streams 32 / LPR rows per step with
// 16-byte loads and keeps its column accumulators in registers.
template <int LPR, int NCH>
__global__ void __launch_bounds__(PI_WARPS * 32)
k_pi_pass_vec(const float* __restrict__ X, int64_t n, const double* __restrict__ mean,
              const double* __restrict__ v, double* __restrict__ part)
{
    constexpr int D = 4 * LPR * NCH;
    constexpr int RPW = 32 / LPR;                       // rows per warp and step
    __shared__ double sv[D], smean[D];
    __shared__ double sfold[D];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane % LPR, rg = lane / LPR;
    for (int j = threadIdx.x; j < D; j += blockDim.x) { sv[j] = v[j]; smean[j] = mean[j]; }
    __syncthreads();
    double acc[NCH * 4];
#pragma unroll
    for (int k = 0; k < NCH * 4; ++k) acc[k] = 0.0;
    const int64_t stride = (int64_t)gridDim.x * PI_WARPS * RPW;
    // The loop bound is the warp's base row, identical in all 32 lanes: the shuffles below are
    // executed by the whole warp even when only some of its RPW rows exist.
    for (int64_t rbase = ((int64_t)blockIdx.x * PI_WARPS + warp) * RPW; rbase < n; rbase += stride) {
        const int64_t row = rbase + rg;
        const bool valid = row < n;
        double xc[NCH * 4];
        double z = 0.0;
#pragma unroll
        for (int k = 0; k < NCH; ++k) {
            const int col = 4 * (sub + k * LPR);
            const float4 x = valid ? __ldcs(reinterpret_cast<const float4*>(X + row * D + col)) : make_float4(0.f, 0.f, 0.f, 0.f);
            xc[4 * k + 0] = valid ? (double)x.x - smean[col + 0] : 0.0;
            xc[4 * k + 1] = valid ? (double)x.y - smean[col + 1] : 0.0;
            xc[4 * k + 2] = valid ? (double)x.z - smean[col + 2] : 0.0;
            xc[4 * k + 3] = valid ? (double)x.w - smean[col + 3] : 0.0;
            z = fma(xc[4 * k + 0], sv[col + 0], z); z = fma(xc[4 * k + 1], sv[col + 1], z);
            z = fma(xc[4 * k + 2], sv[col + 2], z); z = fma(xc[4 * k + 3], sv[col + 3], z);
        }
#pragma unroll
        for (int o = 1; o < LPR; o <<= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
#pragma unroll
        for (int k = 0; k < NCH * 4; ++k) acc[k] = fma(z, xc[k], acc[k]);
    }
    // fold the row groups of the warp (lanes with equal sub), then the warps one after the other in warp order
    // into one shared record
#pragma unroll
    for (int k = 0; k < NCH * 4; ++k) {
        double t = acc[k];
#pragma unroll
        for (int o = LPR; o < 32; o <<= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
        acc[k] = t;
    }
    for (int w = 0; w < PI_WARPS; ++w) {
        if (warp == w && rg == 0) {
#pragma unroll
            for (int k = 0; k < NCH * 4; ++k) {
                const int j = 4 * (sub + (k >> 2) * LPR) + (k & 3);
                sfold[j] = (w == 0) ? acc[k] : sfold[j] + acc[k];
            }
        }
        __syncthreads();
    }
    for (int j = threadIdx.x; j < D; j += blockDim.x) part[(size_t)blockIdx.x * D + j] = sfold[j];
}

// w = sum of the per-CTA partials in CTA order (the result of one application of X_c^T X_c to v).
__global__ void __launch_bounds__(256)
k_pi_fin(const double* __restrict__ part, int g, int d, double* __restrict__ w)
{
    for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < d; j += gridDim.x * blockDim.x) {
        double t = 0.0;
        for (int b = 0; b < g; ++b) t += part[(size_t)b * d + j];
        w[j] = t;
    }
}

// X-hat = FP32((X - mean) * (1/a)), evaluated in FP64.
__global__ void __launch_bounds__(256)
k_normalize(const float* X, float* Xhat, int64_t total, int d,
            const double* __restrict__ mean, double inv_a)
{
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t nthreads = (int64_t)gridDim.x * blockDim.x;
    if ((d & 3) == 0) {
        const int64_t total4 = total >> 2;
        for (int64_t e4 = tid; e4 < total4; e4 += nthreads) {
            const int col = (int)((e4 << 2) % d);
            float4 x = reinterpret_cast<const float4*>(X)[e4];
            float4 o;
            o.x = (float)(((double)x.x - mean[col + 0]) * inv_a);
            o.y = (float)(((double)x.y - mean[col + 1]) * inv_a);
            o.z = (float)(((double)x.z - mean[col + 2]) * inv_a);
            o.w = (float)(((double)x.w - mean[col + 3]) * inv_a);
            reinterpret_cast<float4*>(Xhat)[e4] = o;
        }
    } else {
        for (int64_t e = tid; e < total; e += nthreads) {
            const int col = (int)(e % d);
            Xhat[e] = (float)(((double)X[e] - mean[col]) * inv_a);
        }
    }
}

// Counter-based standard normals for the starting vector (splitmix64 + Box-Muller), host side.
static inline uint64_t splitmix64(uint64_t x)
{
    x += 0x9E3779B97F4A7C15ull;
    x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
    x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
    return x ^ (x >> 31);
}

// Largest eigenvalue of the symmetric tridiagonal matrix (alpha[0..m-1], beta[0..m-2]) by bisection
// on the Sturm sequence (host).
static double tridiag_max_eig(const std::vector<double>& alpha, const std::vector<double>& beta, int m)
{
    double lo = alpha[0], hi = alpha[0];
    for (int i = 0; i < m; ++i) {
        const double off = (i > 0 ? fabs(beta[i - 1]) : 0.0) + (i + 1 < m ? fabs(beta[i]) : 0.0);
        if (alpha[i] - off < lo) lo = alpha[i] - off;
        if (alpha[i] + off > hi) hi = alpha[i] + off;
    }
    for (int it = 0; it < 200 && hi - lo > 1e-15 * fabs(hi); ++it) {
        const double mid = 0.5 * (lo + hi);
        // number of eigenvalues greater than mid = number of positive terms of the Sturm recurrence
        int greater = 0;
        double q = alpha[0] - mid;
        if (q > 0) ++greater;
        for (int i = 1; i < m; ++i) {
            const double den = (fabs(q) < 1e-300) ? (q < 0 ? -1e-300 : 1e-300) : q;
            q = alpha[i] - mid - beta[i - 1] * beta[i - 1] / den;
            if (q > 0) ++greater;
        }
        if (greater >= 1) lo = mid; else hi = mid;
    }
    return 0.5 * (lo + hi);
}

// a = ||X_c||_2.  Every pass applies X_c^T X_c to a unit vector on the device (k_pi_pass + k_pi_fin: the
// power-iteration kernel pair).  The passes are driven by a Lanczos recurrence on the host (d-vectors,
// full reorthogonalisation): the largest Ritz value of the tridiagonal matrix is the best estimate of
// lambda_max in the span of the iterates v, Av, A^2 v, ... -- never above lambda_max, and it converges in
// far fewer passes than the plain iteration v <- Av / ||Av|| when the leading singular values are close.
int run_spectral_norm(const Problem& pb, const float* X_in, float* Xhat_out, double* a_out,
                      double* host_scratch)
{
    (void)host_scratch;
    const auto& P = pb.P;
    const int d = P.d;
    const int g = pb.L.gs;
    double* mean = pb.setup();              // [d]
    double* v = mean + d;                   // [d]
    double* wdev = v + d;                   // [d]
    double* part = wdev + d;                // [g][d]
    cudaStream_t st = pb.stream;

    std::vector<double> hostv(d);
    if (P.center) {
        k_colmean<<<g, 256, 0, st>>>(X_in, P.n, d, part);
        k_colmean_fin<<<(d + 255) / 256, 256, 0, st>>>(part, g, d, P.n, mean);
        pb.count(2);
        if (pb.shard) {
            // global mean = (sum over ranks of the local column sums) / n_global, summed on the host in rank order
            if (cudaMemcpyAsync(hostv.data(), mean, sizeof(double) * d, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
                cudaStreamSynchronize(st) != cudaSuccess)
                return GEM_NLR_E_CUDA;
            for (int j = 0; j < d; ++j) hostv[j] *= (double)P.n;
            if (pb.shard->host_sum(pb.shard->ctx, hostv.data(), d) != 0) return GEM_NLR_E_CUDA;
            for (int j = 0; j < d; ++j) hostv[j] /= (double)pb.shard->n_global;
            if (cudaMemcpyAsync(mean, hostv.data(), sizeof(double) * d, cudaMemcpyHostToDevice, st) != cudaSuccess ||
                cudaStreamSynchronize(st) != cudaSuccess)
                return GEM_NLR_E_CUDA;
        }
    } else {
        cudaMemsetAsync(mean, 0, sizeof(double) * d, st);
    }
    // seeded Gaussian start, normalized
    std::vector<std::vector<double>> V;
    std::vector<double> vk(d), w(d);
    double nrm2 = 0.0;
    for (int j = 0; j < d; ++j) {
        uint64_t a = splitmix64(P.pi_seed * 0x100000001B3ull + 2 * (uint64_t)j);
        uint64_t b = splitmix64(P.pi_seed * 0x100000001B3ull + 2 * (uint64_t)j + 1);
        double u1 = ((double)(a >> 11) + 1.0) / 9007199254740993.0;
        double u2 = (double)(b >> 11) / 9007199254740992.0;
        vk[j] = sqrt(-2.0 * log(u1)) * cos(6.283185307179586 * u2);
        nrm2 += vk[j] * vk[j];
    }
    for (int j = 0; j < d; ++j) vk[j] /= sqrt(nrm2);

    const size_t smem = sizeof(double) * ((size_t)PI_WARPS * d + 2 * (size_t)d);
    if (smem > 48 * 1024)
        cudaFuncSetAttribute(k_pi_pass, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    int max_it = P.pi_max_iters > 0 ? P.pi_max_iters : 100;
    if (max_it > d) max_it = d;             // the Krylov space is exhausted after d steps
    const double tol = P.pi_tol > 0.0 ? P.pi_tol : 1e-7;
    std::vector<double> alpha, beta;
    double sigma_prev = -1.0, sigma = 0.0;
    int calm = 0;
    for (int it = 0; it < max_it; ++it) {
        if (cudaMemcpyAsync(v, vk.data(), sizeof(double) * d, cudaMemcpyHostToDevice, st) != cudaSuccess)
            return GEM_NLR_E_CUDA;
        switch (d) {
#define PI_CASE(DD, LPR, NCH) case DD: k_pi_pass_vec<LPR, NCH><<<g, PI_WARPS * 32, 0, st>>>(X_in, P.n, mean, v, part); break;
            PI_CASE(16, 4, 1) PI_CASE(32, 8, 1) PI_CASE(64, 16, 1) PI_CASE(128, 32, 1) PI_CASE(256, 32, 2)
            PI_CASE(384, 32, 3) PI_CASE(512, 32, 4) PI_CASE(640, 32, 5) PI_CASE(768, 32, 6)
#undef PI_CASE
            default: k_pi_pass<<<g, PI_WARPS * 32, smem, st>>>(X_in, P.n, d, mean, v, part); break;
        }
        k_pi_fin<<<(d + 255) / 256, 256, 0, st>>>(part, g, d, wdev);
        pb.count(2);
        if (cudaMemcpyAsync(w.data(), wdev, sizeof(double) * d, cudaMemcpyDeviceToHost, st) != cudaSuccess)
            return GEM_NLR_E_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return GEM_NLR_E_CUDA;
        // row-sharded: X_c^T X_c v is the sum of the ranks' products (every rank then runs the same recurrence)
        if (pb.shard && pb.shard->host_sum(pb.shard->ctx, w.data(), d) != 0) return GEM_NLR_E_CUDA;
        double ak = 0.0;
        for (int j = 0; j < d; ++j) ak += vk[j] * w[j];
        if (!isfinite(ak)) return GEM_NLR_E_NONFINITE;
        alpha.push_back(ak);
        V.push_back(vk);
        // w <- w - (projection on all previous Lanczos vectors), twice for numerical orthogonality
        for (int pass = 0; pass < 2; ++pass)
            for (const auto& vj : V) {
                double dot = 0.0;
                for (int j = 0; j < d; ++j) dot += vj[j] * w[j];
                for (int j = 0; j < d; ++j) w[j] -= dot * vj[j];
            }
        double bk = 0.0;
        for (int j = 0; j < d; ++j) bk += w[j] * w[j];
        bk = sqrt(bk);
        const double theta = tridiag_max_eig(alpha, beta, (int)alpha.size());
        sigma = sqrt(theta > 0.0 ? theta : 0.0);
        if (sigma_prev >= 0.0 && fabs(sigma - sigma_prev) <= tol * sigma) { if (++calm >= 2) break; } else calm = 0;
        sigma_prev = sigma;
        if (!(bk > 1e-14 * (fabs(ak) + 1e-300))) break;   // invariant subspace: the Ritz value is exact
        beta.push_back(bk);
        for (int j = 0; j < d; ++j) vk[j] = w[j] / bk;
    }
    if (!(sigma > 0.0)) return GEM_NLR_E_BREAKDOWN;
    *a_out = sigma;
    const int64_t total = P.n * (int64_t)d;
    int64_t blocks = (total / 4 + 255) / 256;
    if (blocks > kSMs * 16) blocks = kSMs * 16;
    if (blocks < 1) blocks = 1;
    k_normalize<<<(int)blocks, 256, 0, st>>>(X_in, Xhat_out, total, d, mean, 1.0 / sigma);
    pb.count();
    if (cudaGetLastError() != cudaSuccess) return GEM_NLR_E_CUDA;
    return GEM_NLR_OK;
}

}  // namespace gemnlr
