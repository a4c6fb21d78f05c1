// gem_nlr_column_sums_static: p = U^T 1 with no allocation anywhere.
//
// Some callers of this library may not allocate device memory when they need a result: a
// plug-in that runs inside a host application which hands out all device memory at start-up
// and forbids later cudaMalloc calls, a serving loop in which an allocation's implicit
// device-wide synchronization would stall other streams, or code that has already given the
// whole device to a memory pool it does not own.  The regular entry points take their scratch
// from a caller-provided workspace; this one keeps its scratch (the per-block partial column
// sums) in a fixed array that is part of the library image.  Every GPU that loads the library
// holds that array (about 300 KB) until the process exits.
//
// The array is named in host code only to look up its device address: the host-side symbol is
// a stand-in, not something a kernel can be given.  The address is looked up once per device,
// with that device current, on the first call made on it.
#include <cuda_runtime.h>
#include <stdint.h>
#include <mutex>
#include "../../include/gem_nlr.h"

namespace {

constexpr int kWarps = 4;                       // warps per block, one row per warp at a time
constexpr int kMaxBlocks = 296;                 // two blocks per SM of a B200
constexpr int kMaxR = GEM_NLR_STATIC_MAX_R;     // widest factor the fixed scratch can serve
constexpr int kMaxDevices = 64;

// per-block partial column sums: [kMaxBlocks][kMaxR] FP64
static __device__ __align__(256) double g_colsum_scratch[kMaxBlocks * kMaxR];

__global__ void __launch_bounds__(kWarps * 32)
k_colsum_static(const float* __restrict__ U, int64_t n, int r, double* __restrict__ part)
{
    __shared__ double acc[kWarps][kMaxR];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int j = lane; j < r; j += 32) acc[warp][j] = 0.0;
    const int64_t stride = (int64_t)gridDim.x * kWarps;
    for (int64_t row = (int64_t)blockIdx.x * kWarps + warp; row < n; row += stride) {
        const float* u = U + row * r;
        for (int j = lane; j < r; j += 32) acc[warp][j] += (double)u[j];
    }
    __syncthreads();
    // every block overwrites its whole record, so nothing in the scratch has to start at zero
    for (int j = threadIdx.x; j < r; j += blockDim.x) {
        double v = 0.0;
        for (int w = 0; w < kWarps; ++w) v += acc[w][j];
        part[(size_t)blockIdx.x * kMaxR + j] = v;
    }
}

__global__ void k_colsum_static_fin(const double* __restrict__ part, int blocks, int r, float* __restrict__ p)
{
    for (int j = threadIdx.x; j < r; j += blockDim.x) {
        double v = 0.0;
        for (int b = 0; b < blocks; ++b) v += part[(size_t)b * kMaxR + j];   // fixed order
        p[j] = (float)v;
    }
}

std::mutex g_mu;
double* g_scratch_addr[kMaxDevices];   // device address of g_colsum_scratch, per device

// Looks up (once per device, with that device current) where the scratch array lives.
int scratch_for_current_device(double** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return GEM_NLR_E_CUDA;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
        double* ptr = nullptr;
        if (cudaGetSymbolAddress((void**)&ptr, g_colsum_scratch) != cudaSuccess || !ptr) return GEM_NLR_E_CUDA;
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return GEM_NLR_OK;
}

}  // namespace

extern "C" int gem_nlr_column_sums_static(const float* U_dev, int64_t n, int32_t r, float* p_dev,
                                          void* cuda_stream)
{
    if (!U_dev || !p_dev || n < 1 || r < 1) return GEM_NLR_E_INVALID;
    if (r > kMaxR) return GEM_NLR_E_TOO_LARGE;
    double* scratch = nullptr;
    const int rc = scratch_for_current_device(&scratch);
    if (rc != GEM_NLR_OK) return rc;
    int64_t blocks = (n + kWarps - 1) / kWarps;
    if (blocks > kMaxBlocks) blocks = kMaxBlocks;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    k_colsum_static<<<(int)blocks, kWarps * 32, 0, st>>>(U_dev, n, r, scratch);
    k_colsum_static_fin<<<1, 128, 0, st>>>(scratch, (int)blocks, r, p_dev);
    return cudaGetLastError() == cudaSuccess ? GEM_NLR_OK : GEM_NLR_E_CUDA;
}
