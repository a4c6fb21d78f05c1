// Tensor-core first product of the iteration with the vector pass fused in (tcgen05 + TMEM),
//   Theta = X-hat^T U   (d x r),   u = c_f w,  q = u.p - 1,  gated ytilde += gamma q,
//   ybar = ytilde + gamma q,  s = U^T ybar,  sum q^2,  sum ytilde q            (Algorithm 2, call sites 1-3, 8-11)
// for shapes where FP32 FFMA cannot keep up with HBM (r > 16).
//
// FP32 accuracy from FP16 tensor cores: every operand entry is scaled by a power of two and split as
// x 2^k = h1 + h2 with h1 = fp16(x 2^k), h2 = fp16(x 2^k - h1) (22 significant bits), and the product is
// accumulated in FP32 as h1 h1' + h2 h1' + h1 h2' (three MMAs with K = 16); the dropped h2 h2' term is
// below 2^-22 relative.  The scales cannot overflow: |x-hat_ij| <= ||X-hat||_2 = 1 (scale 2^15) and
// |u_ij| <= ||U||_F = sqrt(K) (scale the largest power of two with |u| 2^k <= 2^14).  Against the
// 3xTF32 split of the other kernels this halves the number of MMA instructions per row (K = 16 instead
// of 8), and an MMA instruction costs the same ~130-180 cycles whatever K is: at N = d = 64 the TF32
// version of this kernel was bound by exactly that instruction rate.
//
// The contraction runs over the data rows, so both operands are MN-major: per stage of TR = 32 rows the
// split warps write fp16 images in the canonical MN-major 128-byte-swizzle layout (atoms of 64 columns
// x 8 rows = 8 x 128 bytes, 16-byte chunk index XOR row mod 8; K atoms 1 KB apart, MN atoms 4 KB apart).
// The accumulator is Theta^T: TMEM lane = column j of U (M = 128, columns beyond r are zero), TMEM
// column = feature f (N = d).
//
// One persistent CTA per SM, 14 warps:
//   warp 0       producer: per stage ceil(r/32) U boxes and d/32 X-hat boxes (plain FP32 rows).
//   warps 6-17   vector + split, three teams taking stages round-robin: one warp per row does the row-local
//                vector work on the U boxes, then both operands are converted into the image ring;
//                the raw stage goes back to the producer as soon as the team has read it.
//   warp 1       MMA issuer (2 k-steps x 3 products per stage).  Every FLUSH stages the accumulator is
//                handed to the epilogue and the other TMEM buffer is started from zero.
//   warps 2-5    epilogue: add each handed-over accumulator, rescaled, into this CTA's FP64 partial of
//                Theta^T (thread = column j of U).
// Partials have the layout of the FFMA family's first product, so k_red1_fused reduces them.
// Every mbarrier wait is bounded (GEM_NLR_E_TIMEOUT; the kernel runs to its end and frees its TMEM).
#include "nlr_common.cuh"
#include "device_utils.cuh"
#include "pipeline.cuh"
#include "tc_common.cuh"
#include "tc_family.cuh"
#include <cuda_fp16.h>

namespace gemnlr {
namespace tc1 {

constexpr int TR = 32;                         // data rows per stage (4 k-steps)
constexpr int CHUNK_BYTES = TR * 128;          // one box: TR rows x 32 floats
constexpr int NTEAMS = 3;                      // vector / split teams of four warps, taking stages round-robin
constexpr int NTHREADS = (6 + 4 * NTEAMS) * 32;
constexpr int MAX_RING = 8;
constexpr int FLUSH = 32;                      // stages per accumulation period (1024 rows)
constexpr int ATOM_BYTES = TR * 128;           // one MN atom of an image: 64 columns (128 bytes) x TR rows

// Shared-memory matrix descriptor of an MN-major fp16 operand in the 128-byte-swizzle layout:
// leading byte offset = distance between MN atoms (64 columns), stride byte offset = distance between
// K atoms (8 rows).
__device__ __forceinline__ uint64_t umma_desc_mn_sw128(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3fffu);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32;
    d |= (uint64_t)1 << 46;          // version
    d |= (uint64_t)2 << 61;          // SWIZZLE_128B
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

// v (already scaled) -> (h1, h2) packed for 4 consecutive entries: 8 bytes each.
__device__ __forceinline__ void split_h4(const float4 v, uint2& h1, uint2& h2)
{
    const __half2 a01 = __floats2half2_rn(v.x, v.y), a23 = __floats2half2_rn(v.z, v.w);
    const float2 f01 = __half22float2(a01), f23 = __half22float2(a23);
    const __half2 b01 = __floats2half2_rn(v.x - f01.x, v.y - f01.y), b23 = __floats2half2_rn(v.z - f23.x, v.w - f23.y);
    h1 = make_uint2(*reinterpret_cast<const uint32_t*>(&a01), *reinterpret_cast<const uint32_t*>(&a23));
    h2 = make_uint2(*reinterpret_cast<const uint32_t*>(&b01), *reinterpret_cast<const uint32_t*>(&b23));
}

__device__ __forceinline__ void sts64(uint32_t addr, uint2 v)
{
    asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(addr), "r"(v.x), "r"(v.y) : "memory");
}

// Byte offset of 4 consecutive columns starting at column c (multiple of 4) of row rl inside an image
// (MN atoms of 64 columns ATOM_BYTES apart, 128-byte rows, 16-byte chunk index XOR row mod 8).
__device__ __forceinline__ uint32_t img_off(int rl, int c)
{
    return (uint32_t)((c >> 6) * ATOM_BYTES + rl * 128 + ((((c & 63) >> 3) ^ (rl & 7)) << 4) + (c & 7) * 2);
}

__global__ void __launch_bounds__(NTHREADS, 1)
k_pass1_tc(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmU,
           float* __restrict__ ytilde, float* __restrict__ ybar, Ctl* __restrict__ ctl,
           const float* __restrict__ p, int64_t n, int d, int r, int K, int NSR, int NLO, double gamma,
           double* __restrict__ part)
{
    if (ctl->stopped) return;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t bars[4 * MAX_RING + 4];
    __shared__ uint32_t abort_flag;
    __shared__ uint32_t tmem_base_s;
    __shared__ __align__(16) float sp[128];
    __shared__ double sq[2][4 * NTEAMS];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int NBX = d / 32;                        // X-hat boxes per stage
    const int NBU = (r + 31) / 32;                 // U boxes per stage (M = 128 reads 4; missing ones are never written: see below)
    const int STAGE = (4 + NBX) * CHUNK_BYTES;     // raw stage: 4 U boxes then the X-hat boxes (FP32 rows of 128 bytes)
    const int NXA = (d + 63) / 64;                 // MN atoms of an X-hat image
    const int IMG = (2 * 2 + 2 * NXA) * ATOM_BYTES;   // image stage: U h1 (2 atoms), U h2, X h1, X h2
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < 2 * d) tmem_cols <<= 1;

    const uint32_t smem_base = smem_u32(smem);
    const uint32_t raw0 = smem_base;                                   // NSR raw stages
    const uint32_t img0 = raw0 + (uint32_t)NSR * STAGE;                // NLO image stages

    const uint32_t bar0 = smem_u32(bars);
    auto full = [&](int s) { return bar0 + 8u * s; };
    auto split = [&](int s) { return bar0 + 8u * (MAX_RING + s); };
    auto rawfree = [&](int s) { return bar0 + 8u * (2 * MAX_RING + s); };
    auto lofree = [&](int s) { return bar0 + 8u * (3 * MAX_RING + s); };
    auto accfull = [&](int a) { return bar0 + 8u * (4 * MAX_RING + a); };
    auto accfree = [&](int a) { return bar0 + 8u * (4 * MAX_RING + 2 + a); };

    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_RING; ++s) {
            mbar_init(full(s), 1); mbar_init(split(s), 4); mbar_init(rawfree(s), 4); mbar_init(lofree(s), 1);
        }
        for (int a = 0; a < 2; ++a) { mbar_init(accfull(a), 1); mbar_init(accfree(a), 4); }
        abort_flag = 0;
        fence_barrier_init();
    }
    if (threadIdx.x < 128) sp[threadIdx.x] = (threadIdx.x < r) ? p[threadIdx.x] : 0.f;
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_s), tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;

    // contiguous block of stages per CTA
    const int64_t n_stages = (n + TR - 1) / TR;
    const int64_t base_cnt = n_stages / gridDim.x, rem_cnt = n_stages % gridDim.x;
    const int64_t g_lo = (int64_t)blockIdx.x * base_cnt + ((int64_t)blockIdx.x < rem_cnt ? blockIdx.x : rem_cnt);
    const int my_stages = (int)(base_cnt + ((int64_t)blockIdx.x < rem_cnt ? 1 : 0));
    const int n_periods = (my_stages + FLUSH - 1) / FLUSH;

    const float cf = ctl->c_f;
    const int dual = ctl->dual_pending;
    // power-of-two operand scales (see the header): x-hat 2^15, u 2^eU with |u| 2^eU <= 2^14
    int eU;
    {
        int e;
        frexpf(sqrtf((float)K), &e);                   // |u_ij| <= ||U||_F = sqrt(K) <= 2^e
        eU = 14 - e;
    }
    const float sU = ldexpf(1.0f, eU), sX = 32768.0f;
    const double unscale = ldexp(1.0, -15 - eU);
    double qq = 0.0, yq = 0.0;
    float s_acc[4] = {0.f, 0.f, 0.f, 0.f};         // vector warps: s partial of this lane's 4 columns
    double* const out = part + (size_t)blockIdx.x * ((size_t)d * r + r + 2);

    if (warp == 0) {
        // ------------------------------ producer ------------------------------
        if (lane == 0) {
            for (int g = 0; g < my_stages && !abort_flag; ++g) {
                const int s = g % NSR;
                if (g >= NSR) mbar_wait(rawfree(s), ((g / NSR) - 1) & 1, &abort_flag, ctl);
                const int row0 = (int)((g_lo + g) * TR);
                const uint32_t dst = raw0 + (uint32_t)s * STAGE;
                mbar_expect_tx(full(s), (uint32_t)(NBU + NBX) * CHUNK_BYTES);
                for (int c = 0; c < NBU; ++c) tma_load_2d(dst + c * CHUNK_BYTES, &tmU, c * 32, row0, full(s));
                for (int b = 0; b < NBX; ++b) tma_load_2d(dst + (4 + b) * CHUNK_BYTES, &tmX, b * 32, row0, full(s));
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_f16(128, d, 1, 1);
            // The wait for the next stage sits between the two k-steps of the current one, so the tensor pipe
            // has MMAs queued while this thread polls.
            if (my_stages > 0) mbar_wait(split(0), 0, &abort_flag, ctl);
            for (int g = 0; g < my_stages && !abort_flag; ++g) {
                const int l = g % NLO;
                const int period = g / FLUSH, a = period & 1, in_period = g % FLUSH;
                if (in_period == 0 && period >= 2) mbar_wait(accfree(a), ((period >> 1) - 1) & 1, &abort_flag, ctl);
                tc_fence_after();
                const uint32_t tacc = tmem_base + (uint32_t)(a * d);
                const uint32_t im = img0 + (uint32_t)l * IMG;
                // A = U images (M = 128: 2 MN atoms), B = X-hat images (N = d); MN atoms ATOM_BYTES apart (LBO),
                // K atoms of 8 rows 1 KB apart (SBO); a k-step of 16 rows advances the start address by 2 KB
                const uint64_t da1 = umma_desc_mn_sw128(im, ATOM_BYTES, 1024), da2 = umma_desc_mn_sw128(im + 2 * ATOM_BYTES, ATOM_BYTES, 1024);
                const uint64_t db1 = umma_desc_mn_sw128(im + 4 * ATOM_BYTES, ATOM_BYTES, 1024);
                const uint64_t db2 = umma_desc_mn_sw128(im + (4 + NXA) * ATOM_BYTES, ATOM_BYTES, 1024);
#pragma unroll
                for (int ks = 0; ks < TR / 16; ++ks) {
                    if (ks == 1 && g + 1 < my_stages)
                        mbar_wait(split((g + 1) % NLO), ((g + 1) / NLO) & 1, &abort_flag, ctl);
                    umma_f16_x3(tacc, da1 + 128 * ks, da2 + 128 * ks, db1 + 128 * ks, db2 + 128 * ks, idesc,
                                (in_period | ks) ? 1u : 0u);
                }
                umma_commit(lofree(l));
                if (in_period == FLUSH - 1 || g == my_stages - 1) umma_commit(accfull(a));
            }
        }
    } else if (warp >= 6) {
        // ------------------------------ vector pass + split ------------------------------
        // One warp per row at a time: lane = (U chunk, 16-byte piece), i.e. the 32 lanes read the 4 x 8
        // pieces of one row -- every quarter-warp covers one full 128-byte line, no bank conflicts.
        // NTEAMS teams of four warps take the stages round-robin: a stage costs a team about 3,400 cycles of
        // mostly dependent latency (reductions, FP64 row scalars, conversions) against a budget of ~900, so
        // several stages have to be in flight.
        const int vw = warp - 6;                           // 0 .. 4 NTEAMS - 1
        const int team = vw >> 2, tw = vw & 3;             // team; rows tw + 4 k (k = 0..7) of the team's stages
        const int tt = (vw & 3) * 32 + lane;               // 0..127 inside the team
        const int box = lane >> 3, c = lane & 7;           // U chunk (32 columns) and logical 16-byte piece inside it
        const int col0 = box * 32 + 4 * c;                 // first of this lane's 4 columns of u
        const float4 p4 = *reinterpret_cast<const float4*>(sp + col0);
        // ytilde of this warp's eight rows (lane k < 8 holds row tw + 4 k) is requested one of the team's
        // stages ahead, so its DRAM latency is not paid inside the stage
        float yt_next = 0.f;
        if (team < my_stages) {
            const int64_t row_f = (g_lo + team) * TR + tw + 4 * (lane & 7);
            if (lane < 8 && row_f < n) yt_next = ytilde[row_f];
        }
        for (int g = team; g < my_stages; g += NTEAMS) {
            const int s = g % NSR, l = g % NLO;
            const int64_t srow0 = (g_lo + g) * TR;
            const int64_t myrow = srow0 + tw + 4 * (lane & 7);
            float yt_l = yt_next;
            yt_next = (g + NTEAMS < my_stages && lane < 8 && myrow + NTEAMS * TR < n) ? ytilde[myrow + NTEAMS * TR] : 0.f;
            float yb_l = 0.f;
            mbar_wait(full(s), (g / NSR) & 1, &abort_flag, ctl);
            if (g >= NLO) mbar_wait(lofree(l), ((g / NLO) - 1) & 1, &abort_flag, ctl);
            const uint32_t hi_s = raw0 + (uint32_t)s * STAGE, im = img0 + (uint32_t)l * IMG;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                // four independent rows at a time: loads first, reductions interleaved, then scalars and stores
                uint32_t off[4];
                float4 u4[4];
                float dot[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int rl = tw + 4 * (half * 4 + k);
                    off[k] = (uint32_t)(box * CHUNK_BYTES + rl * 128 + c * 16);
                }
                {
                    float4 w4[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k)      // boxes beyond r are never loaded: their columns are zero
                        w4[k] = (box < NBU) ? lds128(hi_s + off[k]) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        u4[k] = make_float4(cf * w4[k].x, cf * w4[k].y, cf * w4[k].z, cf * w4[k].w);
                        dot[k] = fmaf(u4[k].x, p4.x, fmaf(u4[k].y, p4.y, fmaf(u4[k].z, p4.z, u4[k].w * p4.w)));
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1)
#pragma unroll
                    for (int k = 0; k < 4; ++k) dot[k] += __shfl_xor_sync(0xffffffffu, dot[k], o);
                // row scalars: lane 4 half + k owns row tw + 4 (4 half + k) (dot[] is the same in every lane)
                {
                    const int kk = lane & 3;
                    const float q = (kk == 0) ? dot[0] : (kk == 1) ? dot[1] : (kk == 2) ? dot[2] : dot[3];
                    const float qm1 = q - 1.0f;
                    if ((lane >> 2) == half) {
                        if (dual) yt_l = (float)((double)yt_l + gamma * (double)qm1);
                        yb_l = (float)((double)yt_l + gamma * (double)qm1);
                        if (myrow < n) {
                            qq = fma((double)qm1, (double)qm1, qq);
                            yq = fma((double)yt_l, (double)qm1, yq);
                        }
                    }
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float yb = __shfl_sync(0xffffffffu, yb_l, half * 4 + k);
                    s_acc[0] = fmaf(u4[k].x, yb, s_acc[0]); s_acc[1] = fmaf(u4[k].y, yb, s_acc[1]);   // rows beyond n: u = 0
                    s_acc[2] = fmaf(u4[k].z, yb, s_acc[2]); s_acc[3] = fmaf(u4[k].w, yb, s_acc[3]);
                    // image of u 2^eU (u = c_f w rounded to FP32, as the plain definition has it)
                    uint2 h1, h2;
                    split_h4(make_float4(u4[k].x * sU, u4[k].y * sU, u4[k].z * sU, u4[k].w * sU), h1, h2);
                    const uint32_t io = img_off(tw + 4 * (half * 4 + k), col0);
                    sts64(im + io, h1);
                    sts64(im + 2 * ATOM_BYTES + io, h2);
                }
            }
            if (lane < 8 && myrow < n) {
                if (dual) ytilde[myrow] = yt_l;
                ybar[myrow] = yb_l;
            }
            // ---- X-hat boxes -> fp16 images: 256 float4 per box, two per thread of the team ----
            for (int b = 0; b < NBX; ++b) {
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const int idx = tt + 128 * hh, rr = idx >> 3, f0 = b * 32 + 4 * (idx & 7);
                    const float4 x = lds128(hi_s + (uint32_t)((4 + b) * CHUNK_BYTES) + (uint32_t)idx * 16);
                    uint2 h1, h2;
                    split_h4(make_float4(x.x * sX, x.y * sX, x.z * sX, x.w * sX), h1, h2);
                    const uint32_t io = img_off(rr, f0);
                    sts64(im + 4 * ATOM_BYTES + io, h1);
                    sts64(im + (4 + NXA) * ATOM_BYTES + io, h2);
                }
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(split(l));          // image stage l is ready for the MMAs
                mbar_arrive(rawfree(s));        // and this team is done with the raw stage
            }
        }
        qq = warp_sum(qq);
        yq = warp_sum(yq);
        if (lane == 0) { sq[0][vw] = qq; sq[1][vw] = yq; }
    }
    if (warp >= 2 && warp < 6) {
        // ------------------------------ epilogue: FP64 fold of the accumulator ------------------------------
        // Thread = column j of U (TMEM lane).  Each hand-over adds the FP32
        // accumulator of the period into this CTA's FP64 partial record (Theta^T entry (j, f) lives at
        // out[f * r + j]; every thread owns its addresses, lanes are contiguous in j).
        const int q4 = warp & 3;                          // TMEM lane quarter
        const int j = q4 * 32 + lane;                     // column of U
        for (int period = 0; period < n_periods; ++period) {
            const int a = period & 1;
            mbar_wait(accfull(a), (period >> 1) & 1, &abort_flag, ctl);
            tc_fence_after();
            for (int c = 0; c * 16 < d; ++c) {
                float v[16];
                tmem_ld16(tmem_base + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(a * d + c * 16), v);
                if (j < r) {
                    double* o = out + (size_t)(c * 16) * r + j;
#pragma unroll
                    for (int k = 0; k < 16; ++k) {
                        const double prev = (period == 0) ? 0.0 : o[(size_t)k * r];
                        o[(size_t)k * r] = prev + unscale * (double)v[k];
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(accfree(a));
        }
    }
    // Every MMA has completed (the epilogue waited for the last hand-over): the rings are scratch now.
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, tmem_cols);
    float* sscr = reinterpret_cast<float*>(smem);             // [vector warps][128 columns]
    if (warp >= 6) {
        const int col0 = (lane >> 3) * 32 + 4 * (lane & 7);
#pragma unroll
        for (int k = 0; k < 4; ++k) sscr[(warp - 6) * 128 + col0 + k] = s_acc[k];
    }
    __syncthreads();
    if (threadIdx.x < r) {
        double v = 0.0;
        for (int k = 0; k < 4 * NTEAMS; ++k) v += (double)sscr[k * 128 + threadIdx.x];
        out[(size_t)d * r + threadIdx.x] = v;
    }
    if (threadIdx.x == 0) {
        double a0 = 0.0, a1 = 0.0;
        for (int w = 0; w < 4 * NTEAMS; ++w) { a0 += sq[0][w]; a1 += sq[1][w]; }
        out[(size_t)d * r + r] = a0;
        out[(size_t)d * r + r + 1] = a1;
    }
}

}  // namespace tc1

bool tc1_plan(const Problem& pb, Tc1Plan* pl)
{
    const int d = pb.P.d, r = pb.P.r;
    if (d % 32 != 0 || d > 256 || r % 4 != 0 || r < 8 || r > 128 || pb.P.n < 1024 || pb.P.n > 2000000000ll) return false;
    if ((size_t)d * r > 16384) return false;          // partial records of the shared reduction kernel
    const int NBX = d / 32, NXA = (d + 63) / 64;
    const size_t stage = (size_t)(4 + NBX) * tc1::CHUNK_BYTES;
    const size_t img = (size_t)(4 + 2 * NXA) * tc1::ATOM_BYTES;
    const size_t limit = 227 * 1024 - 2048;
    int NLO = 0, NSR = 0;
    for (int nlo = 4; nlo >= 2 && !NSR; --nlo)
        for (int nsr = 6; nsr >= 3; --nsr)
            if ((size_t)nsr * stage + (size_t)nlo * img + 1024 <= limit) { NSR = nsr; NLO = nlo; break; }
    if (!NSR) return false;
    pl->NSR = NSR; pl->NLO = NLO;
    pl->smem = (size_t)NSR * stage + (size_t)NLO * img + 1024;
    if (pl->smem < (size_t)8 * 128 * 4 + 1024) pl->smem = (size_t)8 * 128 * 4 + 1024;     // s scratch of the tail
    if (!make_tensor_map_2d(&pl->tmX, pb.X, pb.P.n, d, tc1::TR, 32, false, 1)) return false;      // plain rows
    if (!make_tensor_map_2d(&pl->tmU, pb.U, pb.P.n, r, tc1::TR, 32, false, 1)) return false;
    const int64_t stages = (pb.P.n + tc1::TR - 1) / tc1::TR;
    pl->grid = (int)(stages < kSMs ? stages : kSMs);
    if (cudaFuncSetAttribute(tc1::k_pass1_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl->smem) != cudaSuccess)
        return false;
    return true;
}

void tc1_launch_first(const Problem& pb, const Tc1Plan& pl)
{
    tc1::k_pass1_tc<<<pl.grid, tc1::NTHREADS, pl.smem, pb.stream>>>(
        pl.tmX, pl.tmU, pb.ytilde(), pb.ybar(), pb.ctl(), pb.p(), pb.P.n, pb.P.d, pb.P.r, pb.P.K, pl.NSR, pl.NLO, pb.gamma,
        pb.part1());
    pb.count(1);
}

}  // namespace gemnlr
