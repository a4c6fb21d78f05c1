// tcgen05 / TMEM helpers for the 3xTF32 kernel family (sm_100a only).
#pragma once
#include <stdint.h>
#include "pipeline.cuh"
#include <cuda_fp16.h>

namespace gemnlr {

// FP32 -> (hi, lo) with hi exactly representable in TF32 (low 13 mantissa bits cleared) and
// lo = x - hi (exact in FP32).  x*y is then recovered to about 2^-21 by hi*hi' + lo*hi' + hi*lo'.
__device__ __forceinline__ float tf32_hi(float x) { return __uint_as_float(__float_as_uint(x) & 0xffffe000u); }

// Shared-memory matrix descriptor (64 bit): start address, leading / stride byte offsets
// (all >> 4), descriptor version 1 (sm_100), 128-byte swizzle.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3fffu);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32;
    d |= (uint64_t)1 << 46;          // version
    d |= (uint64_t)2 << 61;          // SWIZZLE_128B
    return d;
}

// Same for the 128-byte swizzle with 32-byte atoms (layout type 1), the only layout MN-major TF32
// operands may use: 128-byte rows along K, the 32-byte chunk index XORed with the row index mod 4.
__device__ __forceinline__ uint64_t umma_desc_sw128_atom32(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3fffu);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32;
    d |= (uint64_t)1 << 46;          // version
    d |= (uint64_t)1 << 61;          // SWIZZLE_128B_BASE32B
    return d;
}

// Instruction descriptor for kind::tf32, FP32 accumulate, M x N tile; a_mn / b_mn: operand is
// MN-major (1) or K-major (0).
__host__ __device__ constexpr uint32_t umma_idesc_tf32(int M, int N, int a_mn, int b_mn)
{
    return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// D[tmem] (+)= A[smem] * B[smem]; issued by one thread.
__device__ __forceinline__ void umma_tf32(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
        : "memory");
}

// The three products of one k-step of the split scheme, D (+)= Ahi*Bhi + Alo*Bhi + Ahi*Blo, from one
// asm block so that the issuing thread spends as few instructions as possible per MMA.
__device__ __forceinline__ void umma_tf32_x3(uint32_t tmem_d, uint64_t a_hi, uint64_t a_lo, uint64_t b_hi,
                                             uint64_t b_lo, uint32_t idesc, uint32_t accumulate_first)
{
    asm volatile(
        "{\n\t.reg .pred p, t;\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "setp.eq.b32 t, %7, %7;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %3, %5, {%7, %7, %7, %7}, p;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %2, %3, %5, {%7, %7, %7, %7}, t;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %4, %5, {%7, %7, %7, %7}, t;\n\t}"
        ::"r"(tmem_d), "l"(a_hi), "l"(a_lo), "l"(b_hi), "l"(b_lo), "r"(idesc), "r"(accumulate_first), "r"(0u)
        : "memory");
}

// Arrive on an mbarrier once all tcgen05.mma issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Whole-warp TMEM allocation of ncols columns (power of two >= 32); the base address is
// written to *dst_smem.
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// 32 lanes x 32 consecutive columns: thread i of the warp receives row (lane base + i).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v)
{
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// 32 lanes x 16 consecutive columns.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v)
{
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// 16 TMEM lanes x 16 columns in the fragment layout of the warp-level MMA accumulators: thread t gets,
// for column block b (8 columns), v[4b], v[4b+1] = (lane t/4, columns 8b + 2 (t%4), + 1) and v[4b+2], v[4b+3] =
// the same columns of lane t/4 + 8.  Four threads hold 8 consecutive columns of a row: one 32-byte sector.
// Completion must be awaited with tmem_ld_wait() before the values are used.
__device__ __forceinline__ void tmem_ld_16x256b_x2(uint32_t taddr, float* v)
{
    uint32_t r[8];
    asm volatile("tcgen05.ld.sync.aligned.16x256b.x2.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr));
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Column sums of a 32-row x 16-column block held one row per lane (v[16]): after the exchange
// lane l holds the sum of column 8 b4 + 4 b3 + 2 b2 + b1 (bits of l) over the 32 rows (both lanes of a
// pair hold the same value).  31 adds and 16 shuffles instead of 80 of each for 16 butterfly sums.
__device__ __forceinline__ float colsum16(const float* v, int lane)
{
    float a8[8], a4[4], a2[2], a1;
    const bool h16 = lane & 16, h8 = lane & 8, h4 = lane & 4, h2 = lane & 2;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float send = h16 ? v[i] : v[i + 8];
        const float keep = h16 ? v[i + 8] : v[i];
        a8[i] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float send = h8 ? a8[i] : a8[i + 4];
        const float keep = h8 ? a8[i + 4] : a8[i];
        a4[i] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const float send = h4 ? a4[i] : a4[i + 2];
        const float keep = h4 ? a4[i + 2] : a4[i];
        a2[i] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
    }
    {
        const float send = h2 ? a2[0] : a2[1];
        const float keep = h2 ? a2[1] : a2[0];
        a1 = keep + __shfl_xor_sync(0xffffffffu, send, 2);
    }
    return a1 + __shfl_xor_sync(0xffffffffu, a1, 1);
}

// ---- two-term FP16 split (x 2^k = h1 + h2, 22 significant bits) on kind::f16 MMAs with K = 16 ----
// Shared-memory matrix descriptor, K-major operand with the 64-byte swizzle: 64-byte rows, groups
// of 8 rows 512 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_k_sw64(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3fffu);
    d |= (uint64_t)(16u >> 4) << 16;
    d |= (uint64_t)(512u >> 4) << 32;
    d |= (uint64_t)1 << 46;          // version
    d |= (uint64_t)4 << 61;          // SWIZZLE_64B
    return d;
}

// Instruction descriptor for kind::f16 with fp16 operands, FP32 accumulate, M x N tile.
__host__ __device__ constexpr uint32_t umma_idesc_f16(int M, int N, int a_mn, int b_mn)
{
    return (1u << 4) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) | ((uint32_t)(N >> 3) << 17) |
           ((uint32_t)(M >> 4) << 24);
}

// D (+)= A1 B1 + A2 B1 + A1 B2 (one k-step of 16 of the two-term fp16 split).
__device__ __forceinline__ void umma_f16_x3(uint32_t tmem_d, uint64_t a1, uint64_t a2, uint64_t b1, uint64_t b2,
                                            uint32_t idesc, uint32_t accumulate_first)
{
    asm volatile(
        "{\n\t.reg .pred p, t;\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "setp.eq.b32 t, %7, %7;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %3, %5, {%7, %7, %7, %7}, p;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %2, %3, %5, {%7, %7, %7, %7}, t;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %4, %5, {%7, %7, %7, %7}, t;\n\t}"
        ::"r"(tmem_d), "l"(a1), "l"(a2), "l"(b1), "l"(b2), "r"(idesc), "r"(accumulate_first), "r"(0u)
        : "memory");
}

// Two MMAs of one k-step when the B images h1 | h2 are contiguous (N = 2 n): D[:, 0..2n) (+)= A1 [B1 | B2],
// then D[:, 0..n) += A2 B1.  Columns 0..n-1 collect h1 h1' + h2 h1', columns n..2n-1 collect h1 h2'; the
// reader of the accumulator adds the two halves.  One MMA instruction fewer per k-step: an instruction costs
// the issuing thread ~130 cycles whatever its N, which is what bounds narrow tiles.
__device__ __forceinline__ void umma_f16_x2(uint32_t tmem_d, uint64_t a1, uint64_t a2, uint64_t b12, uint32_t idesc_2n,
                                            uint32_t idesc_n, uint32_t accumulate_first)
{
    asm volatile(
        "{\n\t.reg .pred p, t;\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "setp.eq.b32 t, %7, %7;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %3, %4, {%7, %7, %7, %7}, p;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %2, %3, %5, {%7, %7, %7, %7}, t;\n\t}"
        ::"r"(tmem_d), "l"(a1), "l"(a2), "l"(b12), "r"(idesc_2n), "r"(idesc_n), "r"(accumulate_first), "r"(0u)
        : "memory");
}

// Eight scaled values (consecutive data rows of one column) -> the two fp16 chunks h1, h2 (16 bytes each).
__device__ __forceinline__ void split_h8(const float* v, uint4& h1, uint4& h2)
{
    uint32_t a[4], b[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __half2 hi = __floats2half2_rn(v[2 * i], v[2 * i + 1]);
        const float2 f = __half22float2(hi);
        const __half2 lo = __floats2half2_rn(v[2 * i] - f.x, v[2 * i + 1] - f.y);
        a[i] = *reinterpret_cast<const uint32_t*>(&hi);
        b[i] = *reinterpret_cast<const uint32_t*>(&lo);
    }
    h1 = make_uint4(a[0], a[1], a[2], a[3]);
    h2 = make_uint4(b[0], b[1], b[2], b[3]);
}

__device__ __forceinline__ void sts128u(uint32_t addr, uint4 v)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

__device__ __forceinline__ float lds32f(uint32_t addr)
{
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
}

// Byte offset inside a K-major image of the 16-byte chunk holding data rows 8 kg .. 8 kg + 7 of MN row m.
__device__ __forceinline__ uint32_t kimg_off(int m, int kg)
{
    return (uint32_t)(m * 64 + ((kg ^ ((m >> 1) & 3)) << 4));
}

// TMA tile store shared -> global (clipped at the tensor bounds), bulk-group completion.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tmap, int x, int y, uint32_t src)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"((uint64_t)tmap), "r"(x), "r"(y), "r"(src) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait() { asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void named_bar_sync(int id, int nthreads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

}  // namespace gemnlr
