// Setup of the normalized model (Section 3): X_c = X - 1 xbar^T, a = ||X_c||_2, X-hat = X_c / a.
// The paper does not say how a is computed; here it is a power iteration on X_c^T X_c applied
// implicitly, one streaming pass over X per iteration:  w = sum_i z_i (x_i - xbar),
// z_i = (x_i - xbar) . v,  sigma = sqrt(||w||) for ||v|| = 1,  v <- w / ||w||.
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

// w = sum of partials; sigma = sqrt(||w||); v <- w / ||w||.  scal[0] = sigma, scal[1] = ||w||.
__global__ void __launch_bounds__(256)
k_pi_fin(const double* __restrict__ part, int g, int d, double* __restrict__ v,
         double* __restrict__ scal)
{
    __shared__ double sred[32];
    double nrm2 = 0.0;
    for (int j = threadIdx.x; j < d; j += blockDim.x) {
        double t = 0.0;
        for (int b = 0; b < g; ++b) t += part[(size_t)b * d + j];
        v[j] = t;
        nrm2 += t * t;
    }
    nrm2 = block_sum<256>(nrm2, sred);
    const double nrm = sqrt(nrm2);
    for (int j = threadIdx.x; j < d; j += blockDim.x) v[j] = (nrm > 0.0) ? v[j] / nrm : 0.0;
    if (threadIdx.x == 0) { scal[0] = sqrt(nrm); scal[1] = nrm; }
}

// X-hat = FP32((X - mean) * (1/a)), evaluated in FP64.
__global__ void __launch_bounds__(256)
k_normalize(const float* __restrict__ X, float* __restrict__ Xhat, int64_t total, int d,
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

int run_spectral_norm(const Problem& pb, const float* X_in, float* Xhat_out, double* a_out,
                      double* host_scratch)
{
    const auto& P = pb.P;
    const int d = P.d;
    const int g = pb.L.gs;
    double* mean = pb.setup();              // [d]
    double* v = mean + d;                   // [d]
    double* scal = v + d;                   // [4]
    double* part = scal + 4;                // [g][d]
    cudaStream_t st = pb.stream;

    if (P.center) {
        k_colmean<<<g, 256, 0, st>>>(X_in, P.n, d, part);
        k_colmean_fin<<<(d + 255) / 256, 256, 0, st>>>(part, g, d, P.n, mean);
        pb.count(2);
    } else {
        cudaMemsetAsync(mean, 0, sizeof(double) * d, st);
    }
    // seeded Gaussian start, normalized
    std::vector<double> v0(d);
    double nrm2 = 0.0;
    for (int j = 0; j < d; ++j) {
        uint64_t a = splitmix64(P.pi_seed * 0x100000001B3ull + 2 * (uint64_t)j);
        uint64_t b = splitmix64(P.pi_seed * 0x100000001B3ull + 2 * (uint64_t)j + 1);
        double u1 = ((double)(a >> 11) + 1.0) / 9007199254740993.0;
        double u2 = (double)(b >> 11) / 9007199254740992.0;
        v0[j] = sqrt(-2.0 * log(u1)) * cos(6.283185307179586 * u2);
        nrm2 += v0[j] * v0[j];
    }
    for (int j = 0; j < d; ++j) v0[j] /= sqrt(nrm2);
    if (cudaMemcpyAsync(v, v0.data(), sizeof(double) * d, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return GEM_NLR_E_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return GEM_NLR_E_CUDA;   // v0 is a local

    const size_t smem = sizeof(double) * ((size_t)PI_WARPS * d + 2 * (size_t)d);
    if (smem > 48 * 1024)
        cudaFuncSetAttribute(k_pi_pass, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    const int max_it = P.pi_max_iters > 0 ? P.pi_max_iters : 100;
    const double tol = P.pi_tol > 0.0 ? P.pi_tol : 1e-7;
    double sigma_prev = -1.0, sigma = 0.0;
    for (int it = 0; it < max_it; ++it) {
        k_pi_pass<<<g, PI_WARPS * 32, smem, st>>>(X_in, P.n, d, mean, v, part);
        k_pi_fin<<<1, 256, 0, st>>>(part, g, d, v, scal);
        pb.count(2);
        if (cudaMemcpyAsync(host_scratch, scal, 2 * sizeof(double), cudaMemcpyDeviceToHost, st) != cudaSuccess)
            return GEM_NLR_E_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return GEM_NLR_E_CUDA;
        sigma = host_scratch[0];
        if (!isfinite(sigma)) return GEM_NLR_E_NONFINITE;
        if (sigma_prev >= 0.0 && fabs(sigma - sigma_prev) <= tol * sigma) break;
        sigma_prev = sigma;
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
