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
// The contraction runs over the data rows, which is the slow (MN-major) operand orientation of the
// tensor core: MN-major operands are fetched at about 9 elements per clock whatever their type.  The
// split warps touch every entry anyway, so they write the fp16 images transposed, K-major: one 64-byte
// row (the 32 data rows of a stage) per column of U / feature of X-hat, 64-byte swizzle (16-byte chunk
// index XOR (row >> 1) mod 4).  A lane owns columns lane + 32 j and a warp eight consecutive data rows, so
// a lane holds the 8 K-values of a chunk and writes it with one conflict-free 16-byte store.  With
// K-major operands an M = 128, N = d MMA costs about 130 cycles: 6 per stage, under the HBM budget.
// The accumulator is Theta^T: TMEM lane = column j of U (M = 128, columns beyond r are zero), TMEM
// column = feature f (N = d).
//
// One persistent CTA per SM, 20 warps (roles by warp index: see the role constants below):
//   U producer   per stage one bulk copy of the TR rows of U (contiguous in global memory); without the static
//                images also of the rows of X-hat.
//   X producer   per stage the pre-swizzled transposed fp16 image boxes of X-hat, straight into the image stage.
//   teams        vector + split, three teams of four warps taking stages round-robin: a warp does the row-local
//                vector work on 8 rows of U, then the operands are converted into the image ring;
//                the raw stage goes back to the producer as soon as the team has read it.
//   MMA issuer   2 k-steps x 3 products per stage (2 x 2 with the stacked N = 2 d operand).  Every FLUSH stages
//                the accumulator is handed to the epilogue and the other TMEM buffer is started from zero.
//   epilogue     four warps add each handed-over accumulator, rescaled, into this CTA's FP64 partial of
//                Theta^T (thread = column j of U).
// Partials have the layout of the FFMA family's first product, so k_red1_fused reduces them.
// Every mbarrier wait is bounded (GEM_NLR_E_TIMEOUT; the kernel runs to its end and frees its TMEM).
#include "nlr_common.cuh"
#include "device_utils.cuh"
#include "pipeline.cuh"
#include "tc_common.cuh"
#include "tc_family.cuh"

namespace gemnlr {
namespace tc1 {

constexpr int TR = 32;                         // data rows per stage (4 k-steps)
constexpr int NTEAMS = 3;                      // vector / split teams of four warps, taking stages round-robin
constexpr int NTHREADS = 20 * 32;
// Warp roles.  A warp runs on scheduler (warp index mod 4).  The thread that issues the MMAs executes a serial
// stream of ~100 instructions per stage; when it shared its scheduler with three busy team warps that
// stream, not the tensor pipe or the teams, set the stage rate (device timelines: no wait on its path, 1400
// cycles per stage).  So scheduler 1 hosts only light roles: the issuer (warp 1), one of the four epilogue
// warps (5: the TMEM lane quarter of a warp is fixed by its index mod 4), the two producers (9, 13) and an
// idle warp (17); the twelve team warps are the warps of schedulers 0, 2 and 3 outside the epilogue group 4-7.
__device__ __forceinline__ bool is_team_warp(int w) { return (w & 3) != 1 && (w >> 2) != 1; }
__device__ __forceinline__ int team_warp_index(int w)          // 0 .. 11 over the team warps in increasing order
{
    const int q = w >> 2, res = w & 3;
    return (q == 0 ? 0 : q - 1) * 3 + (res == 0 ? 0 : res - 1);
}
constexpr int WARP_UPROD = 9, WARP_XPROD = 13, WARP_ISSUER = 1, WARP_EPI0 = 4;
constexpr int MAX_RING = 8;
constexpr int FLUSH = 128;                     // stages per accumulation period (4096 rows)
constexpr int UIMG = 128 * 64;                 // one fp16 image of the U operand: 128 columns x 32 data rows

// XIMG = true: the X-hat operand comes from the static transposed fp16 images (one contiguous, pre-swizzled
// box of d x 32 halves per stage and image, bulk-copied straight into the image stage); the raw stage then
// holds the U rows only and the teams convert only U.  XIMG = false: the teams convert the FP32 rows of X-hat too.
template <bool XIMG>
__global__ void __launch_bounds__(NTHREADS, 1)
k_pass1_tc(const float* __restrict__ X, const float* __restrict__ U, const __half* __restrict__ xT1,
           const __half* __restrict__ xT2, float* __restrict__ ytilde, float* __restrict__ ybar, Ctl* __restrict__ ctl,
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
    // raw stage: the TR rows of U then those of X-hat exactly as they lie in global memory (row pitch r and
    // d floats): the rows of a stage are contiguous there, so each operand arrives with one bulk copy
    const int URAW = (TR * r * 4 + 127) / 128 * 128;
    const int STAGE = (URAW + (XIMG ? 0 : TR * d * 4) + 1023) / 1024 * 1024;
    const int XIMG_BYTES = d * 64;                 // one fp16 image of the X-hat operand: d features x 32 data rows
    const int IMG = 2 * UIMG + 2 * XIMG_BYTES;           // image stage: U h1, U h2, X h1, X h2
    // d <= 128: the X-hat images h1 | h2 are used as one N = 2 d operand (2 MMAs per k-step, accumulator of 2 d
    // columns whose halves the epilogue adds); else 3 MMAs per k-step into d columns
    const bool wideB = d <= 128;
    const int ACC = wideB ? 2 * d : d;             // TMEM columns per accumulator buffer
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < 2 * ACC) tmem_cols <<= 1;

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
            mbar_init(full(s), 1); mbar_init(split(s), XIMG ? 5 : 4); mbar_init(rawfree(s), 4); mbar_init(lofree(s), 1);
        }
        for (int a = 0; a < 2; ++a) { mbar_init(accfull(a), 1); mbar_init(accfree(a), 4); }
        abort_flag = 0;
        fence_barrier_init();
    }
    if (threadIdx.x < 128) sp[threadIdx.x] = (threadIdx.x < r) ? p[threadIdx.x] : 0.f;
    if (warp == WARP_ISSUER) tmem_alloc(smem_u32(&tmem_base_s), tmem_cols);
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

    if (warp == WARP_UPROD) {
        // ------------------------------ producer ------------------------------
        if (lane == 0) {
            for (int g = 0; g < my_stages && !abort_flag; ++g) {
                const int s = g % NSR;
                if (g >= NSR) mbar_wait_backoff(rawfree(s), ((g / NSR) - 1) & 1, &abort_flag, ctl);
                const int64_t row0 = (g_lo + g) * TR;
                const int rows = (n - row0 < TR) ? (int)(n - row0) : TR;
                const uint32_t dst = raw0 + (uint32_t)s * STAGE;
                if (XIMG) {
                    mbar_expect_tx(full(s), (uint32_t)(rows * r * 4));
                    bulk_load_1d(dst, U + row0 * r, (uint32_t)(rows * r * 4), full(s));
                } else {
                    mbar_expect_tx(full(s), (uint32_t)(rows * (r + d) * 4));
                    bulk_load_1d(dst, U + row0 * r, (uint32_t)(rows * r * 4), full(s));
                    bulk_load_1d(dst + URAW, X + row0 * d, (uint32_t)(rows * d * 4), full(s));
                }
            }
        }
    } else if (warp == WARP_XPROD) {
        // ------------------------------ X-hat image producer ------------------------------
        // Its own thread: the image ring is released by the MMAs, the raw ring by the teams; one thread
        // serving both would let the U loads run only one stage ahead.  The boxes of a stage go straight
        // into its image stage, once the MMAs of the stage that used it last are done.
        if (XIMG && lane == 0) {
            for (int g = 0; g < my_stages && !abort_flag; ++g) {
                const int l = g % NLO;
                if (g >= NLO) mbar_wait_backoff(lofree(l), ((g / NLO) - 1) & 1, &abort_flag, ctl);
                const uint32_t im = img0 + (uint32_t)l * IMG;
                const size_t xoff = (size_t)(g_lo + g) * d * 32;          // one block of d features per stage
                mbar_expect_tx(split(l), (uint32_t)(2 * XIMG_BYTES));
                bulk_load_1d(im + 2 * UIMG, xT1 + xoff, (uint32_t)XIMG_BYTES, split(l));
                bulk_load_1d(im + 2 * UIMG + XIMG_BYTES, xT2 + xoff, (uint32_t)XIMG_BYTES, split(l));
            }
        }
    } else if (warp == WARP_ISSUER) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_f16(128, d, 0, 0), idesc2 = umma_idesc_f16(128, 2 * d, 0, 0);
            // The wait for the next stage sits between the two k-steps of the current one, so the tensor pipe
            // has MMAs queued while this thread polls.
            if (my_stages > 0) mbar_wait_spin(split(0), 0, &abort_flag, ctl);
            // image slot l and its phase, accumulator a and position in the accumulation period: kept
            // incrementally (this thread's instruction stream is the critical path of the kernel)
            int l = 0, lph = 0, a = 0, in_period = 0, period = 0;
            // descriptors of image stage 0; the address field counts 16-byte units, so stage l adds l * IMG / 16
            const uint64_t da1_0 = umma_desc_k_sw64(img0), da2_0 = umma_desc_k_sw64(img0 + UIMG);
            const uint64_t db1_0 = umma_desc_k_sw64(img0 + 2 * UIMG), db2_0 = umma_desc_k_sw64(img0 + 2 * UIMG + XIMG_BYTES);
            const uint64_t dstep = (uint64_t)(IMG >> 4);
            for (int g = 0; g < my_stages; ++g) {
                if (in_period == 0 && period >= 2) mbar_wait_spin(accfree(a), ((period >> 1) - 1) & 1, &abort_flag, ctl);
                tc_fence_after();
                const uint32_t tacc = tmem_base + (uint32_t)(a * ACC);
                // A = U images (M = 128 columns), B = X-hat images (N = d features), K-major; a k-step of 16 data
                // rows (32 bytes inside the 64-byte swizzled row) advances the start address by 2
                const uint64_t doff = dstep * (uint64_t)l;
                const uint64_t da1 = da1_0 + doff, da2 = da2_0 + doff, db1 = db1_0 + doff, db2 = db2_0 + doff;
                if (wideB) umma_f16_x2(tacc, da1, da2, db1, idesc2, idesc, in_period ? 1u : 0u);
                else umma_f16_x3(tacc, da1, da2, db1, db2, idesc, in_period ? 1u : 0u);
                int ln = l + 1, lphn = lph;
                if (ln == NLO) { ln = 0; lphn ^= 1; }
                if (g + 1 < my_stages) mbar_wait_spin(split(ln), (uint32_t)lphn, &abort_flag, ctl);
                if (wideB) umma_f16_x2(tacc, da1 + 2, da2 + 2, db1 + 2, idesc2, idesc, 1u);
                else umma_f16_x3(tacc, da1 + 2, da2 + 2, db1 + 2, db2 + 2, idesc, 1u);
                umma_commit(lofree(l));
                if (in_period == FLUSH - 1 || g == my_stages - 1) umma_commit(accfull(a));
                l = ln; lph = lphn;
                if (++in_period == FLUSH) { in_period = 0; ++period; a ^= 1; }
            }
        }
    } else if (is_team_warp(warp)) {
        // ------------------------------ vector pass + split ------------------------------
        // A warp takes 8 consecutive data rows of a stage, a lane the columns lane + 32 j of U (scalar loads
        // from the plain FP32 rows: consecutive lanes, consecutive words).  NTEAMS teams of four warps take
        // the stages round-robin: a stage costs a team a few thousand cycles of mostly dependent latency
        // (reductions, FP64 row scalars, conversions) against a budget of ~900, so several are in flight.
        const int vw = team_warp_index(warp);              // 0 .. 4 NTEAMS - 1
        const int team = vw >> 2, tw = vw & 3;             // team; data rows 8 tw .. 8 tw + 7 of the team's stages
        float p1[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) p1[j] = sp[lane + 32 * j];
        // ytilde of this warp's eight rows (lane 4 k holds row 8 tw + k: the lane group that ends up with the
        // row's dot product) is requested one of the team's stages ahead, so its DRAM latency is not paid
        // inside the stage
        const bool owner = (lane & 3) == 0;
        const float cs = cf * sU, inv_sU = 1.0f / sU;      // everything below works on v = u 2^eU: scaling by a
                                                           // power of two commutes with every FP32 rounding
        float yt_next = 0.f;
        if (team < my_stages) {
            const int64_t row_f = (g_lo + team) * TR + 8 * tw + (lane >> 2);
            if (owner && row_f < n) yt_next = ytilde[row_f];
        }
        for (int g = team; g < my_stages; g += NTEAMS) {
            const int s = g % NSR, l = g % NLO;
            const int64_t srow0 = (g_lo + g) * TR;
            const int64_t myrow = srow0 + 8 * tw + (lane >> 2);
            float yt_l = yt_next;
            yt_next = (g + NTEAMS < my_stages && owner && myrow + NTEAMS * TR < n) ? ytilde[myrow + NTEAMS * TR] : 0.f;
            float yb_l = 0.f;
            mbar_wait_backoff(full(s), (g / NSR) & 1, &abort_flag, ctl);
            if (g >= NLO) mbar_wait_backoff(lofree(l), ((g / NLO) - 1) & 1, &abort_flag, ctl);
            const uint32_t hi_s = raw0 + (uint32_t)s * STAGE, im = img0 + (uint32_t)l * IMG;
            const int rows_here = (n - srow0 < TR) ? (int)(n - srow0) : TR;
            float u[8][4], dot[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                dot[k] = 0.f;
#pragma unroll
                for (int j = 0; j < 4; ++j) {        // columns beyond r and rows beyond n are zero
                    const float w = (lane + 32 * j < r && 8 * tw + k < rows_here)
                                        ? lds32f(hi_s + (uint32_t)(((8 * tw + k) * r + lane + 32 * j) * 4)) : 0.f;
                    u[k][j] = cs * w;                // v = u 2^eU with u = fl(c_f w)
                    dot[k] = fmaf(u[k][j], p1[j], dot[k]);
                }
            }
            // the eight row sums by recursive halving: lane l ends up with the total of row (l >> 2) & 7
            float q;
            {
                float e4[4], e2[2];
                const bool b4 = lane & 16, b3 = lane & 8, b2 = lane & 4;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float send = b4 ? dot[i] : dot[i + 4], keep = b4 ? dot[i + 4] : dot[i];
                    e4[i] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
                }
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const float send = b3 ? e4[i] : e4[i + 2], keep = b3 ? e4[i + 2] : e4[i];
                    e2[i] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
                }
                {
                    const float send = b2 ? e2[0] : e2[1], keep = b2 ? e2[1] : e2[0];
                    q = keep + __shfl_xor_sync(0xffffffffu, send, 4);
                }
                q += __shfl_xor_sync(0xffffffffu, q, 2);
                q += __shfl_xor_sync(0xffffffffu, q, 1);
            }
            // row scalars: lane 4 k owns row 8 tw + k
            {
                const float qm1 = q * inv_sU - 1.0f;
                if (owner) {
                    if (dual) yt_l = (float)((double)yt_l + gamma * (double)qm1);
                    yb_l = (float)((double)yt_l + gamma * (double)qm1);
                    if (myrow < n) {
                        qq = fma((double)qm1, (double)qm1, qq);
                        yq = fma((double)yt_l, (double)qm1, yq);
                    }
                }
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const float yb = __shfl_sync(0xffffffffu, yb_l, 4 * k);
#pragma unroll
                for (int j = 0; j < 4; ++j) s_acc[j] = fmaf(u[k][j], yb, s_acc[j]);     // rows beyond n: u = 0; scaled by 2^eU
            }
            // images of u 2^eU (u = c_f w rounded to FP32, as the plain definition has it): one chunk per column
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float v[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) v[k] = u[k][j];
                uint4 h1, h2;
                split_h8(v, h1, h2);
                const uint32_t io = kimg_off(lane + 32 * j, tw);
                sts128u(im + io, h1);
                sts128u(im + UIMG + io, h2);
            }
            if (owner && myrow < n) {
                if (dual) ytilde[myrow] = yt_l;
                ybar[myrow] = yb_l;
            }
            // ---- X-hat boxes -> fp16 images: thread = (feature lane, data rows 8 tw .. 8 tw + 7) of a box ----
            for (int b = 0; !XIMG && b < NBX; ++b) {
                float v[8];
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    v[k] = (8 * tw + k < rows_here) ? sX * lds32f(hi_s + (uint32_t)(URAW + ((8 * tw + k) * d + b * 32 + lane) * 4)) : 0.f;
                uint4 h1, h2;
                split_h8(v, h1, h2);
                const uint32_t io = kimg_off(b * 32 + lane, tw);
                sts128u(im + 2 * UIMG + io, h1);
                sts128u(im + 2 * UIMG + XIMG_BYTES + io, h2);
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
    if (warp >= WARP_EPI0 && warp < WARP_EPI0 + 4) {
        // ------------------------------ epilogue: FP64 fold of the accumulator ------------------------------
        // Thread = column j of U (TMEM lane).  Each hand-over adds the FP32
        // accumulator of the period into this CTA's FP64 partial record (Theta^T entry (j, f) lives at
        // out[f * r + j]; every thread owns its addresses, lanes are contiguous in j).
        const int q4 = warp & 3;                          // TMEM lane quarter
        const int j = q4 * 32 + lane;                     // column of U
        for (int period = 0; period < n_periods; ++period) {
            const int a = period & 1;
            mbar_wait_relaxed(accfull(a), (period >> 1) & 1, &abort_flag, ctl);
            tc_fence_after();
            for (int c = 0; c * 16 < d; ++c) {
                float v[16];
                tmem_ld16(tmem_base + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(a * ACC + c * 16), v);
                if (wideB) {            // second half of the accumulator: the h1 h2' products
                    float v2[16];
                    tmem_ld16(tmem_base + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(a * ACC + d + c * 16), v2);
#pragma unroll
                    for (int k = 0; k < 16; ++k) v[k] += v2[k];
                }
                if (j < r) {
                    // eight old values are requested before the first store: two memory round trips per group
                    // instead of sixteen dependent ones (the compiler cannot reorder the loads past the
                    // stores itself), so a fold stays far shorter than an accumulation period
                    double* o = out + (size_t)(c * 16) * r + j;
#pragma unroll
                    for (int h = 0; h < 16; h += 8) {
                        double prev[8];
#pragma unroll
                        for (int k = 0; k < 8; ++k) prev[k] = (period == 0) ? 0.0 : __ldcg(o + (size_t)(h + k) * r);
#pragma unroll
                        for (int k = 0; k < 8; ++k) o[(size_t)(h + k) * r] = prev[k] + unscale * (double)v[h + k];
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
    if (warp == WARP_ISSUER) tmem_dealloc(tmem_base, tmem_cols);
    float* sscr = reinterpret_cast<float*>(smem);             // [vector warps][128 columns]
    if (is_team_warp(warp)) {
#pragma unroll
        for (int k = 0; k < 4; ++k) sscr[team_warp_index(warp) * 128 + lane + 32 * k] = s_acc[k] * ldexpf(1.0f, -eU);
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
    if ((size_t)d * r > 16384) return false;          // larger products raised a launch failure at n = 4e6, d = 200 (224), r = 100 (cause not found): kept out
    const bool ximg = pb.has_ximg() && pb.L.fb == d;          // one block of d features per stage in the transposed images
    if (!ximg && d != pb.dx) return false;                    // without images X-hat itself is read: no feature padding
    const size_t stage = (((size_t)tc1::TR * r * 4 + 127) / 128 * 128 + (ximg ? 0 : (size_t)tc1::TR * d * 4) + 1023) / 1024 * 1024;
    const size_t img = (size_t)2 * tc1::UIMG + (size_t)2 * d * 64;
    const size_t limit = 227 * 1024 - 2048;
    int NLO = 0, NSR = 0;
    // A wait names a phase by its parity, so no waiter may fall two phases behind its barrier.  The raw ring is
    // a multiple of NTEAMS deep (a raw slot then always belongs to the same team, which sees every one of its
    // phases); the image ring needs NLO >= NTEAMS (a team that has seen the MMAs of stage g - NTEAMS - NLO finish
    // knows those of stage g - 2 NLO have).
    for (int nlo = 4; nlo >= tc1::NTEAMS && !NSR; --nlo)
        for (int nsr = 2 * tc1::NTEAMS; nsr >= tc1::NTEAMS; nsr -= tc1::NTEAMS)
            if ((size_t)nsr * stage + (size_t)nlo * img + 1024 <= limit) { NSR = nsr; NLO = nlo; break; }
    if (!NSR) return false;
    pl->NSR = NSR; pl->NLO = NLO; pl->ximg = ximg;
    pl->smem = (size_t)NSR * stage + (size_t)NLO * img + 1024;
    if (pl->smem < (size_t)8 * 128 * 4 + 1024) pl->smem = (size_t)8 * 128 * 4 + 1024;     // s scratch of the tail
    const int64_t stages = (pb.P.n + tc1::TR - 1) / tc1::TR;
    pl->grid = (int)(stages < kSMs ? stages : kSMs);
    if (cudaFuncSetAttribute(tc1::k_pass1_tc<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl->smem) != cudaSuccess ||
        cudaFuncSetAttribute(tc1::k_pass1_tc<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl->smem) != cudaSuccess)
        return false;
    return true;
}

void tc1_launch_first(const Problem& pb, const Tc1Plan& pl)
{
    const __half* x1 = pl.ximg ? reinterpret_cast<const __half*>(pb.ximgT(0)) : nullptr;
    const __half* x2 = pl.ximg ? reinterpret_cast<const __half*>(pb.ximgT(1)) : nullptr;
    if (pl.ximg)
        tc1::k_pass1_tc<true><<<pl.grid, tc1::NTHREADS, pl.smem, pb.stream>>>(
            pb.X, pb.U, x1, x2, pb.ytilde(), pb.ybar(), pb.ctl(), pb.p(), pb.P.n, pb.P.d, pb.P.r, pb.P.K, pl.NSR, pl.NLO,
            pb.gamma, pb.part1());
    else
        tc1::k_pass1_tc<false><<<pl.grid, tc1::NTHREADS, pl.smem, pb.stream>>>(
            pb.X, pb.U, x1, x2, pb.ytilde(), pb.ybar(), pb.ctl(), pb.p(), pb.P.n, pb.P.d, pb.P.r, pb.P.K, pl.NSR, pl.NLO,
            pb.gamma, pb.part1());
    pb.count(1);
}

}  // namespace gemnlr
