// Helpers shared by the warp-level tensor-core kernels (mma.sync TF32 with the 3-product split).
#pragma once
#include "nlr_common.cuh"
#include "pipeline.cuh"
#include "tc_common.cuh"
#include "ffma_family.cuh"

namespace gemnlr {

// wide-factor shapes (kernels_mmaw.cu), reached through mma_plan / mma_launch_* by shape id >= 100
bool mmaw_plan(const Problem& pb, FfmaPlan* pl);
void mmaw_pass1(const Problem& pb, const FfmaPlan& pl);
void mmaw_pass2(const Problem& pb, const FfmaPlan& pl);

namespace mma {

constexpr int NCW = 8;
constexpr int NTHREADS = (NCW + 1) * 32;

template <int TM>
__device__ __forceinline__ uint32_t x_chunk_off(int rl, int c)
{
    return (uint32_t)((c >> 3) * (TM * 128) + rl * 128 + (((c & 7) ^ (rl & 7)) << 4));
}

__device__ __forceinline__ void mma_tf32(float* c, const uint32_t* a, uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t* r)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

__device__ __forceinline__ float lds32(uint32_t addr)
{
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
}

__device__ __forceinline__ void split_tf32(float x, uint32_t& hi, uint32_t& lo)
{
    const float h = tf32_hi(x);
    hi = __float_as_uint(h);
    lo = __float_as_uint(x - h);
}

}  // namespace mma
}  // namespace gemnlr
