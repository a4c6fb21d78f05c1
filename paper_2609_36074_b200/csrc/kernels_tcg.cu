// Tiled 3xTF32 tcgen05 second product for wide problems (d and r too large for the resident-Theta
// kernel: the embedding-sized shape d = 768, r = 1000):
//   acc = X-hat Theta ;  W = [U + 2 alpha acc - alpha (ybar p^T + 1 s^T)]_+ in place ;  FP64 a, b, h ;
//   column sums of W                                               (Eq. "entrywise-fusion", Algorithm 2 call 4)
//
// Work item = (128-row tile, 256-column block).  The K loop streams d in chunks of 16 features:
// a stage holds the X-hat box (128 rows x 64 bytes, TMA with the 64-byte swizzle = K-major UMMA
// operand) and the matching boxes of the pre-split Theta^T images (256 columns x 64 bytes, hi and
// lo, already swizzled in global memory, one bulk copy each).  With M = 128, N = 256 a TF32
// tcgen05.mma runs at the tensor pipe's full rate, and the accumulator (256 TMEM columns) is
// double-buffered, so the epilogue of one item overlaps the MMAs of the next.
//
//   warp 0       producer (TMA / bulk copies, 4-stage ring)
//   warp 1       MMA issuer: per chunk 2 k-steps x 3 products; commits free the stage
//   warps 2-9    epilogue: warp = (TMEM lane quarter, column half); thread = row; 16 columns at a
//                time: tcgen05.ld, old U entries straight from global memory (each thread reads and
//                writes whole 32-byte sectors of its row), FP64 statistics; column sums by a
//                shuffle transpose-reduce, combined across the four quarters in fixed order
//   warps 10-13  split: lo image of the X-hat box (second ring).  The raw box itself is the hi operand:
//                kind::tf32 ignores the low 13 mantissa bits of an FP32 operand (checked: results are
//                unchanged when the box is not rewritten), so hi = trunc(x) needs no storage
// Every mbarrier wait is bounded (error status GEM_NLR_E_TIMEOUT, kernel runs to its end, TMEM freed).
#include "nlr_common.cuh"
#include "device_utils.cuh"
#include "fin_logic.cuh"
#include "pipeline.cuh"
#include "tc_common.cuh"
#include "tc_family.cuh"

namespace gemnlr {
namespace tcg {

constexpr int TILE_M = 128;
constexpr int NBLK = 256;                     // columns per item = MMA N
constexpr int KC = 16;                        // features per chunk (64-byte rows)
constexpr int A_BOX = TILE_M * KC * 4;        // 8 KB
constexpr int B_BOX = NBLK * KC * 4;          // 16 KB
constexpr int STAGE = A_BOX + 2 * B_BOX;      // 40 KB: X-hat raw/hi, Theta^T hi, Theta^T lo
constexpr int NS = 4, NLO = 3;
constexpr int NEPI = 8;                       // epilogue warps
constexpr int NTHREADS = (2 + NEPI + 4) * 32;
constexpr size_t SMEM_RING = (size_t)NS * STAGE + (size_t)NLO * A_BOX;

// Shared-memory matrix descriptor, K-major operand with the 64-byte swizzle: 64-byte rows, groups
// of 8 rows 512 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_sw64(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3fffu);
    d |= (uint64_t)(16u >> 4) << 16;
    d |= (uint64_t)(512u >> 4) << 32;
    d |= (uint64_t)1 << 46;          // version
    d |= (uint64_t)4 << 61;          // SWIZZLE_64B
    return d;
}

// Theta (d x r, FP32 row-major) -> hi / lo images of Theta^T as K-major 64-byte-swizzled boxes:
// box (kb, cb) = features 16 kb .. 16 kb + 15 of columns 256 cb .. 256 cb + 255 (zero beyond r).
__global__ void k_theta_images64(const float* __restrict__ theta, int d, int r, int NCB, const Ctl* __restrict__ ctl,
                                 float* __restrict__ img_hi, float* __restrict__ img_lo)
{
    if (ctl->stopped) return;
    const int64_t total = (int64_t)d * NCB * NBLK;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int j = (int)(e / (NCB * NBLK)), k = (int)(e % (NCB * NBLK));     // feature, column
        const float v = (k < r) ? theta[(size_t)j * r + k] : 0.f;
        const float hi = tf32_hi(v);
        const int kb = j >> 4, jj = j & 15, c = jj >> 2, w = jj & 3;
        const int cb = k >> 8, kr = k & 255;
        const size_t off = ((size_t)(kb * NCB + cb) * NBLK + kr) * KC + (size_t)(((c ^ ((kr >> 1) & 3)) << 2) + w);
        img_hi[off] = hi;
        img_lo[off] = v - hi;
    }
}

__global__ void __launch_bounds__(NTHREADS, 1)
k_pass2_tcg(const __grid_constant__ CUtensorMap tmX, const float* __restrict__ img_hi,
            const float* __restrict__ img_lo, float* __restrict__ U, const float* __restrict__ ybar,
            const float* __restrict__ p, const float* __restrict__ alpha_s, Ctl* __restrict__ ctl, int64_t n, int d,
            int r, int NCB, float alpha, int K, double eps_d, double* __restrict__ part, float* __restrict__ p_out)
{
    if (ctl->stopped) return;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t bars[3 * NS + NLO + 4];
    __shared__ uint32_t abort_flag;
    __shared__ uint32_t tmem_base_s;
    __shared__ double sred[32];
    __shared__ int is_last;
    __shared__ double sc;
    __shared__ int sok;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int KB = d / KC;
    const int RP = NCB * NBLK;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t stage0 = smem_base;
    const uint32_t lo0 = stage0 + (uint32_t)NS * STAGE;
    unsigned char* tail = smem + SMEM_RING;
    float* sp = reinterpret_cast<float*>(tail);                         // [RP] p
    float* sas = sp + RP;                                               // [RP] alpha s
    double* scol = reinterpret_cast<double*>(sas + RP);                 // [RP] running column sums of W
    float* stmp = reinterpret_cast<float*>(scol + RP);                  // [2][4][NBLK] per-quarter column sums of an item

    const uint32_t bar0 = smem_u32(bars);
    auto xfull = [&](int s) { return bar0 + 8u * s; };
    auto xsplit = [&](int s) { return bar0 + 8u * (NS + s); };
    auto xfree = [&](int s) { return bar0 + 8u * (2 * NS + s); };
    auto lofree = [&](int l) { return bar0 + 8u * (3 * NS + l); };
    auto accfull = [&](int a) { return bar0 + 8u * (3 * NS + NLO + a); };
    auto accfree = [&](int a) { return bar0 + 8u * (3 * NS + NLO + 2 + a); };

    if (threadIdx.x == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(xfull(s), 1); mbar_init(xsplit(s), 4); mbar_init(xfree(s), 1); }
        for (int l = 0; l < NLO; ++l) mbar_init(lofree(l), 1);
        for (int a = 0; a < 2; ++a) { mbar_init(accfull(a), 1); mbar_init(accfree(a), NEPI); }
        abort_flag = 0;
        fence_barrier_init();
    }
    for (int j = threadIdx.x; j < RP; j += NTHREADS) {
        sp[j] = (j < r) ? p[j] : 0.f;
        sas[j] = (j < r) ? alpha_s[j] : 0.f;
        scol[j] = 0.0;
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_s), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;

    const int64_t n_tiles = (n + TILE_M - 1) / TILE_M;
    const int64_t n_items = n_tiles * NCB;
    const float cf = ctl->c_f;
    const float two_alpha = 2.0f * alpha;
    double sa = 0.0, sb = 0.0, sh = 0.0;

    if (warp == 0) {
        // ------------------------------ producer ------------------------------
        if (lane == 0) {
            int64_t g = 0;
            for (int64_t w = blockIdx.x; w < n_items && !abort_flag; w += gridDim.x) {
                const int64_t t = w / NCB;
                const int cb = (int)(w % NCB);
                const int row0 = (int)(t * TILE_M);
                for (int kb = 0; kb < KB; ++kb, ++g) {
                    const int s = (int)(g % NS);
                    if (g >= NS) mbar_wait(xfree(s), (uint32_t)((g / NS) - 1) & 1, &abort_flag, ctl);
                    const uint32_t dst = stage0 + (uint32_t)s * STAGE;
                    const size_t boff = ((size_t)(kb * NCB + cb) * NBLK) * KC;
                    mbar_expect_tx(xfull(s), STAGE);
                    tma_load_2d(dst, &tmX, kb * KC, row0, xfull(s));
                    bulk_load_1d(dst + A_BOX, img_hi + boff, B_BOX, xfull(s));
                    bulk_load_1d(dst + A_BOX + B_BOX, img_lo + boff, B_BOX, xfull(s));
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        // Inside an item the wait for the next chunk is placed between the two k-steps of the current chunk,
        // so the tensor pipe has work queued while this thread polls.
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_tf32(TILE_M, NBLK, 0, 0);
            int64_t g = 0;
            int i = 0;
            for (int64_t w = blockIdx.x; w < n_items && !abort_flag; w += gridDim.x, ++i) {
                const int a = i & 1;
                // item boundary: the previous accumulator is already handed over; wait for a free one and for
                // the first chunk
                if (i >= 2) mbar_wait(accfree(a), (uint32_t)((i >> 1) - 1) & 1, &abort_flag, ctl);
                mbar_wait(xsplit((int)(g % NS)), (uint32_t)(g / NS) & 1, &abort_flag, ctl);
                const uint32_t tacc = tmem_base + (uint32_t)(a * NBLK);
                for (int kb = 0; kb < KB; ++kb, ++g) {
                    const int s = (int)(g % NS), l = (int)(g % NLO);
                    tc_fence_after();
                    const uint32_t st = stage0 + (uint32_t)s * STAGE;
                    const uint64_t da_hi = umma_desc_sw64(st), da_lo = umma_desc_sw64(lo0 + (uint32_t)l * A_BOX);
                    const uint64_t db_hi = umma_desc_sw64(st + A_BOX), db_lo = umma_desc_sw64(st + A_BOX + B_BOX);
                    // a k-step (8 features = 32 bytes inside the 64-byte swizzled row) advances the start address by 2
                    umma_tf32_x3(tacc, da_hi, da_lo, db_hi, db_lo, idesc, kb ? 1u : 0u);
                    if (kb + 1 < KB) mbar_wait(xsplit((int)((g + 1) % NS)), (uint32_t)((g + 1) / NS) & 1, &abort_flag, ctl);
                    umma_tf32_x3(tacc, da_hi + 2, da_lo + 2, db_hi + 2, db_lo + 2, idesc, 1u);
                    umma_commit(xfree(s));
                    umma_commit(lofree(l));
                }
                umma_commit(accfull(a));
            }
        }
    } else if (warp >= 2 + NEPI) {
        // ------------------------------ split: lo image of the X-hat box ------------------------------
        const int st = threadIdx.x - (2 + NEPI) * 32;   // 0..127
        int64_t g = 0;
        for (int64_t w = blockIdx.x; w < n_items; w += gridDim.x) {
            for (int kb = 0; kb < KB; ++kb, ++g) {
                const int s = (int)(g % NS), l = (int)(g % NLO);
                mbar_wait(xfull(s), (uint32_t)(g / NS) & 1, &abort_flag, ctl);
                if (g >= NLO) mbar_wait(lofree(l), (uint32_t)((g / NLO) - 1) & 1, &abort_flag, ctl);
                const uint32_t hi_a = stage0 + (uint32_t)s * STAGE, lo_a = lo0 + (uint32_t)l * A_BOX;
                float4 xin[A_BOX / 16 / 128];
#pragma unroll
                for (int k = 0; k < A_BOX / 16 / 128; ++k) xin[k] = lds128(hi_a + (uint32_t)(k * 128 + st) * 16);
#pragma unroll
                for (int k = 0; k < A_BOX / 16 / 128; ++k) {
                    const uint32_t off = (uint32_t)(k * 128 + st) * 16;
                    const float4 x = xin[k];
                    const float4 hi = make_float4(tf32_hi(x.x), tf32_hi(x.y), tf32_hi(x.z), tf32_hi(x.w));
                    sts128(lo_a + off, make_float4(x.x - hi.x, x.y - hi.y, x.z - hi.z, x.w - hi.w));
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(xsplit(s));
            }
        }
    } else {
        // ------------------------------ epilogue (warps 2..9) ------------------------------
        // Warp = (TMEM lane quarter q, column half).  Accumulators are read in the 16x256b fragment layout:
        // a thread holds rows q*32 + g + {0, 8, 16, 24} (g = lane / 4) and, per 16-column group, the column
        // pairs 8 b + 2 tq, + 1 (tq = lane % 4, b = 0, 1), so that the 4 lanes of a group read and write one
        // full 32-byte sector of a row of U.
        const int q = warp & 3;
        const int half = (warp - 2) >> 2;
        const int g4 = lane >> 2, tq = lane & 3;
        const int et = (warp - 2) * 32 + lane;            // 0..255 among the epilogue threads
        int i = 0;
        for (int64_t w = blockIdx.x; w < n_items; w += gridDim.x, ++i) {
            const int a = i & 1;
            const int64_t t = w / NCB;
            const int cb = (int)(w % NCB);
            bool valid[4];
            float nay[4];
            float* urow[4];
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const int64_t row = t * TILE_M + q * 32 + g4 + 8 * x;
                valid[x] = row < n;
                nay[x] = valid[x] ? -alpha * ybar[row] : 0.f;
                urow[x] = U + (valid[x] ? row : 0) * (int64_t)r;
            }
            float* my_tmp = stmp + (size_t)(a * 4 + q) * NBLK + half * 128;
            mbar_wait(accfull(a), (uint32_t)(i >> 1) & 1, &abort_flag, ctl);
            tc_fence_after();
#pragma unroll 1
            for (int jj = 0; jj < 8; ++jj) {
                const int col0 = cb * NBLK + half * 128 + jj * 16;
                // acc[x2][...]: x2 = 0: rows g4, g4 + 8; x2 = 1: rows g4 + 16, g4 + 24
                float acc[2][8];
                const uint32_t tcol = (uint32_t)(a * NBLK + half * 128 + jj * 16);
                tmem_ld_16x256b_x2(tmem_base + ((uint32_t)(q * 32) << 16) + tcol, acc[0]);
                tmem_ld_16x256b_x2(tmem_base + ((uint32_t)(q * 32 + 16) << 16) + tcol, acc[1]);
                float2 wold[4][2];
#pragma unroll
                for (int x = 0; x < 4; ++x)
#pragma unroll
                    for (int b = 0; b < 2; ++b) {
                        const int c = col0 + 8 * b + 2 * tq;
                        wold[x][b] = (valid[x] && c < r) ? __ldcs(reinterpret_cast<const float2*>(urow[x] + c))
                                                         : make_float2(0.f, 0.f);
                    }
                tmem_ld_wait();
                float cs[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
#pragma unroll
                for (int b = 0; b < 2; ++b) {
                    const int c = col0 + 8 * b + 2 * tq;
                    const float2 p2 = *reinterpret_cast<const float2*>(sp + c);
                    const float2 s2 = *reinterpret_cast<const float2*>(sas + c);
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        const bool live = valid[x] && c < r;
                        // rows g4 + 8 x: x = 0, 1 from the first load (registers 4b + 0..1 / 4b + 2..3), x = 2, 3 from the second
                        const float a0 = acc[x >> 1][4 * b + 2 * (x & 1)], a1 = acc[x >> 1][4 * b + 2 * (x & 1) + 1];
                        const float u0 = live ? cf * wold[x][b].x : 0.f, u1 = live ? cf * wold[x][b].y : 0.f;
                        float v0 = fmaf(two_alpha, a0, u0), v1 = fmaf(two_alpha, a1, u1);
                        v0 = fmaf(nay[x], p2.x, v0); v1 = fmaf(nay[x], p2.y, v1);
                        v0 -= s2.x; v1 -= s2.y;
                        const float w0 = live ? fmaxf(v0, 0.f) : 0.f, w1 = live ? fmaxf(v1, 0.f) : 0.f;
                        const double wd0 = (double)w0, ud0 = (double)u0, wd1 = (double)w1, ud1 = (double)u1;
                        sa = fma(wd0, wd0, sa); sb = fma(ud0, ud0, sb); sh = fma(wd0, ud0, sh);
                        sa = fma(wd1, wd1, sa); sb = fma(ud1, ud1, sb); sh = fma(wd1, ud1, sh);
                        cs[b][0] += w0; cs[b][1] += w1;
                        if (live) *reinterpret_cast<float2*>(urow[x] + c) = make_float2(w0, w1);
                    }
                }
                // column sums over the 32 rows of the quarter: the 8 row groups g4 of the warp
#pragma unroll
                for (int b = 0; b < 2; ++b)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        float v = cs[b][e];
                        v += __shfl_xor_sync(0xffffffffu, v, 4);
                        v += __shfl_xor_sync(0xffffffffu, v, 8);
                        v += __shfl_xor_sync(0xffffffffu, v, 16);
                        if (lane < 4) my_tmp[jj * 16 + 8 * b + 2 * tq + e] = v;
                    }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(accfree(a));
            // the four quarters of a column, combined in fixed order by the thread that owns the column
            named_bar_sync(1, NEPI * 32);
            {
                const float* t4 = stmp + (size_t)(a * 4) * NBLK + et;
                const double v = (((double)t4[0] + (double)t4[NBLK]) + (double)t4[2 * NBLK]) + (double)t4[3 * NBLK];
                scol[cb * NBLK + et] += v;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, 512);

    // ---- CTA partial: a, b, h and the column sums of W ----
    const int PS = 4 + r;
    sa = block_sum<NTHREADS>(sa, sred);
    sb = block_sum<NTHREADS>(sb, sred);
    sh = block_sum<NTHREADS>(sh, sred);
    double* out = part + (size_t)blockIdx.x * PS;
    if (threadIdx.x == 0) { out[0] = sa; out[1] = sb; out[2] = sh; out[3] = 0.0; }
    for (int j = threadIdx.x; j < r; j += NTHREADS) out[4 + j] = scol[j];
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned prev = atomicAdd(&ctl->counter[1], 1u);
        is_last = (prev == gridDim.x - 1) ? 1 : 0;
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    const int G = gridDim.x;
    double a = 0.0, b = 0.0, hh = 0.0;
    for (int i = threadIdx.x; i < G; i += NTHREADS) {
        a += __ldcg(part + (size_t)i * PS + 0);
        b += __ldcg(part + (size_t)i * PS + 1);
        hh += __ldcg(part + (size_t)i * PS + 2);
    }
    a = block_sum<NTHREADS>(a, sred);
    b = block_sum<NTHREADS>(b, sred);
    hh = block_sum<NTHREADS>(hh, sred);
    if (threadIdx.x == 0) {
        double c;
        sok = fin2_scalars(ctl, a, b, hh, K, eps_d, &c) ? 1 : 0;
        sc = c;
        ctl->counter[1] = 0;
    }
    __syncthreads();
    if (!sok) return;
    for (int j = threadIdx.x; j < r; j += NTHREADS) {
        double v = 0.0;
        for (int i = 0; i < G; ++i) v += __ldcg(part + (size_t)i * PS + 4 + j);
        p_out[j] = (float)(sc * v);
    }
}


// ================================================================================================
// First product for the same wide problems:  Theta = c_f X-hat^T W  as Theta^T tiles.
//
// Work item (one CTA each, all resident at once) = (128 columns of U, up to 256 features, one of
// NSPLIT contiguous row ranges).  The contraction runs over the data rows, so both operands are
// MN-major: TMA boxes of 16 rows x 32 columns with the 128-byte swizzle of 32-byte atoms (A = 4 boxes
// of U, B = up to 8 boxes of X-hat per stage).  Two teams of four warps take alternate stages and
// write the lo images (x - trunc(x)) into a second ring; the raw boxes serve as the hi operands (the
// tensor core ignores the low 13 mantissa bits) and the pending multiplier c_f is applied to the
// reduced Theta instead of to every entry of U;
// the MMA issuer runs 2 k-steps x 3 products per stage into one of two TMEM accumulators, which is
// handed to the epilogue every FLUSH stages and folded into the FP64 partial of this row range
// (layout [feature][column] like the generic first product, so the same reduction kernel follows).
// The row-local vector work cannot be fused here (a CTA sees 128 of the r columns): it runs as the
// separate vector pass before this kernel.
// ================================================================================================
constexpr int TR1 = 16;                        // rows per stage (2 k-steps)
constexpr int CH1 = TR1 * 128;                 // one box: 16 rows x 32 floats = 2 KB
constexpr int NS1 = 5, NLO1 = 3;               // a raw slot lives from the TMA issue to the last MMA, a lo slot from the split on
constexpr int FLUSH1 = 256;                    // stages per accumulation period (4096 rows)
constexpr int NTH1 = 14 * 32;                  // producer, MMA, 4 epilogue, 8 split warps

__global__ void __launch_bounds__(NTH1, 1)
k_pass1_tcg(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmU, Ctl* __restrict__ ctl,
            int64_t n, int d, int r, int NMT, int NNB, int NSPLIT, double* __restrict__ part)
{
    if (ctl->stopped) return;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t bars[3 * NS1 + NLO1 + 4];
    __shared__ uint32_t abort_flag;
    __shared__ uint32_t tmem_base_s;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // item of this CTA
    const int mt = blockIdx.x % NMT, nb = (blockIdx.x / NMT) % NNB, sp = blockIdx.x / (NMT * NNB);
    const int f0 = nb * 256;
    const int Nb = (d - f0 < 256) ? d - f0 : 256;          // features of this item (multiple of 32)
    const int NBX = Nb / 32;
    const int STAGE1 = (4 + 8) * CH1;                       // U boxes then up to 8 X-hat boxes

    const uint32_t smem_base = smem_u32(smem);
    const uint32_t raw0 = smem_base, lo0 = raw0 + (uint32_t)NS1 * STAGE1;
    const uint32_t bar0 = smem_u32(bars);
    auto full = [&](int s) { return bar0 + 8u * s; };
    auto split = [&](int s) { return bar0 + 8u * (NS1 + s); };
    auto rawfree = [&](int s) { return bar0 + 8u * (2 * NS1 + s); };
    auto lofree = [&](int l) { return bar0 + 8u * (3 * NS1 + l); };
    auto accfull = [&](int a) { return bar0 + 8u * (3 * NS1 + NLO1 + a); };
    auto accfree = [&](int a) { return bar0 + 8u * (3 * NS1 + NLO1 + 2 + a); };
    if (threadIdx.x == 0) {
        for (int s = 0; s < NS1; ++s) { mbar_init(full(s), 1); mbar_init(split(s), 4); mbar_init(rawfree(s), 1); }
        for (int l = 0; l < NLO1; ++l) mbar_init(lofree(l), 1);
        for (int a = 0; a < 2; ++a) { mbar_init(accfull(a), 1); mbar_init(accfree(a), 4); }
        abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_s), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;

    // contiguous block of stages of this row range
    const int64_t n_stages = (n + TR1 - 1) / TR1;
    const int64_t base_cnt = n_stages / NSPLIT, rem_cnt = n_stages % NSPLIT;
    const int64_t g_lo = (int64_t)sp * base_cnt + (sp < rem_cnt ? sp : rem_cnt);
    const int my_stages = (int)(base_cnt + (sp < rem_cnt ? 1 : 0));
    const int n_periods = (my_stages + FLUSH1 - 1) / FLUSH1;

    if (warp == 0) {
        if (lane == 0) {
            for (int g = 0; g < my_stages && !abort_flag; ++g) {
                const int s = g % NS1;
                if (g >= NS1) mbar_wait(rawfree(s), ((g / NS1) - 1) & 1, &abort_flag, ctl);
                const int row0 = (int)((g_lo + g) * TR1);
                const uint32_t dst = raw0 + (uint32_t)s * STAGE1;
                mbar_expect_tx(full(s), (uint32_t)(4 + NBX) * CH1);
                for (int c = 0; c < 4; ++c) tma_load_2d(dst + c * CH1, &tmU, mt * 128 + c * 32, row0, full(s));
                for (int b = 0; b < NBX; ++b) tma_load_2d(dst + (4 + b) * CH1, &tmX, f0 + b * 32, row0, full(s));
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_tf32(128, Nb, 1, 1);
            // the wait for the next stage sits between the two k-steps of the current one
            if (my_stages > 0) mbar_wait(split(0), 0, &abort_flag, ctl);
            for (int g = 0; g < my_stages && !abort_flag; ++g) {
                const int s = g % NS1, l = g % NLO1;
                const int period = g / FLUSH1, a = period & 1, in_period = g % FLUSH1;
                if (in_period == 0 && period >= 2) mbar_wait(accfree(a), ((period >> 1) - 1) & 1, &abort_flag, ctl);
                tc_fence_after();
                const uint32_t tacc = tmem_base + (uint32_t)(a * 256);
                const uint32_t hi_s = raw0 + (uint32_t)s * STAGE1, lo_s = lo0 + (uint32_t)l * STAGE1;
                // chunks are CH1 bytes apart (LBO); 4-row swizzle periods of 512 bytes along K (SBO); a k-step is 1 KB
                const uint64_t da_hi = umma_desc_sw128_atom32(hi_s, CH1, 512), da_lo = umma_desc_sw128_atom32(lo_s, CH1, 512);
                const uint64_t db_hi = umma_desc_sw128_atom32(hi_s + 4 * CH1, CH1, 512);
                const uint64_t db_lo = umma_desc_sw128_atom32(lo_s + 4 * CH1, CH1, 512);
                umma_tf32_x3(tacc, da_hi, da_lo, db_hi, db_lo, idesc, in_period ? 1u : 0u);
                if (g + 1 < my_stages) mbar_wait(split((g + 1) % NS1), ((g + 1) / NS1) & 1, &abort_flag, ctl);
                umma_tf32_x3(tacc, da_hi + 64, da_lo + 64, db_hi + 64, db_lo + 64, idesc, 1u);
                umma_commit(rawfree(s));
                umma_commit(lofree(l));
                if (in_period == FLUSH1 - 1 || g == my_stages - 1) umma_commit(accfull(a));
            }
        }
    } else if (warp >= 6) {
        // ------------------------------ split (two teams on alternate stages) ------------------------------
        const int vw = warp - 6, team = vw >> 2;
        const int tt = (vw & 3) * 32 + lane;               // 0..127 inside the team
        const int nq = (4 + NBX) * (CH1 / 16) / 128;       // float4 per thread and stage (U boxes first)
        for (int g = team; g < my_stages; g += 2) {
            const int s = g % NS1, l = g % NLO1;
            mbar_wait(full(s), (g / NS1) & 1, &abort_flag, ctl);
            if (g >= NLO1) mbar_wait(lofree(l), ((g / NLO1) - 1) & 1, &abort_flag, ctl);
            const uint32_t hi_s = raw0 + (uint32_t)s * STAGE1, lo_s = lo0 + (uint32_t)l * STAGE1;
            // lo = x - trunc(x) of every piece (12 per thread at most, all requested up front); the raw boxes
            // are the hi operands as they are
            float4 xin[12];
#pragma unroll
            for (int k = 0; k < 12; ++k)
                if (k < nq) xin[k] = lds128(hi_s + (uint32_t)(k * 128 + tt) * 16);
#pragma unroll
            for (int k = 0; k < 12; ++k)
                if (k < nq) {
                    const float4 x = xin[k];
                    sts128(lo_s + (uint32_t)(k * 128 + tt) * 16,
                           make_float4(x.x - tf32_hi(x.x), x.y - tf32_hi(x.y), x.z - tf32_hi(x.z), x.w - tf32_hi(x.w)));
                }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(split(s));
        }
    } else {
        // ------------------------------ epilogue: FP64 fold of the accumulator ------------------------------
        // thread = column j of U (TMEM lane); entry (feature f, column j) of this row range's partial
        const int q4 = warp & 3;
        const int j = mt * 128 + q4 * 32 + lane;
        double* const out = part + (size_t)sp * ((size_t)d * r);
        for (int period = 0; period < n_periods; ++period) {
            const int a = period & 1;
            mbar_wait(accfull(a), (period >> 1) & 1, &abort_flag, ctl);
            tc_fence_after();
            for (int c = 0; c * 16 < Nb; ++c) {
                float v[16];
                tmem_ld16(tmem_base + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(a * 256 + c * 16), v);
                if (j < r) {
                    double* o = out + (size_t)(f0 + c * 16) * r + j;
                    double prev[16];
#pragma unroll
                    for (int k = 0; k < 16; ++k) prev[k] = (period == 0) ? 0.0 : __ldcg(o + (size_t)k * r);
#pragma unroll
                    for (int k = 0; k < 16; ++k) o[(size_t)k * r] = prev[k] + (double)v[k];
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(accfree(a));
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, 512);
}

}  // namespace tcg

bool tcg_plan(const Problem& pb, TcgPlan* pl, float* img_storage)
{
    const int d = pb.P.d, r = pb.P.r;
    if (d % tcg::KC != 0 || r % 4 != 0 || r < 16 || pb.P.n < 1024 || pb.P.n > 2000000000ll) return false;
    const int NCB = (r + tcg::NBLK - 1) / tcg::NBLK;
    const int RP = NCB * tcg::NBLK;
    if (RP > 2048) return false;
    pl->NCB = NCB;
    pl->smem2 = tcg::SMEM_RING + (size_t)RP * (4 + 4 + 8) + (size_t)2 * 4 * tcg::NBLK * 4 + 1024;
    if (pl->smem2 > 227 * 1024 - 1024) return false;
    pl->img_hi = img_storage;
    pl->img_lo = img_storage + (size_t)d * RP;
    if (!make_tensor_map_2d(&pl->tmX, pb.X, pb.P.n, d, tcg::TILE_M, tcg::KC, false, 64)) return false;
    const int64_t items = (pb.P.n + tcg::TILE_M - 1) / tcg::TILE_M * NCB;
    pl->g2 = (int)(items < kSMs ? items : kSMs);
    if (cudaFuncSetAttribute(tcg::k_pass2_tcg, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl->smem2) != cudaSuccess)
        return false;
    return true;
}

bool tcg1_plan(const Problem& pb, Tcg1Plan* pl)
{
    const int d = pb.P.d, r = pb.P.r;
    if (d % 32 != 0 || r % 4 != 0 || r < 16 || pb.P.n < 4096 || pb.P.n > 2000000000ll) return false;
    pl->NMT = (r + 127) / 128;
    pl->NNB = (d + 255) / 256;
    const int tiles = pl->NMT * pl->NNB;
    if (tiles > kSMs) return false;
    pl->NSPLIT = kSMs / tiles;
    if (pl->NSPLIT > 8) pl->NSPLIT = 8;                     // partial records are sized for 8 row ranges
    pl->grid = tiles * pl->NSPLIT;
    pl->smem = (size_t)(tcg::NS1 + tcg::NLO1) * 12 * tcg::CH1 + 1024;
    if (!make_tensor_map_2d(&pl->tmX, pb.X, pb.P.n, d, tcg::TR1, 32, true)) return false;
    if (!make_tensor_map_2d(&pl->tmU, pb.U, pb.P.n, r, tcg::TR1, 32, true)) return false;
    if (cudaFuncSetAttribute(tcg::k_pass1_tcg, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl->smem) != cudaSuccess)
        return false;
    return true;
}

void tcg_launch_first(const Problem& pb, const Tcg1Plan& pl)
{
    tcg::k_pass1_tcg<<<pl.grid, tcg::NTH1, pl.smem, pb.stream>>>(pl.tmX, pl.tmU, pb.ctl(), pb.P.n, pb.P.d, pb.P.r,
                                                                 pl.NMT, pl.NNB, pl.NSPLIT, pb.part1());
    pb.count(1);
    launch_red1(pb, pl.NSPLIT, 0, 1);
}

void tcg_launch_second(const Problem& pb, const TcgPlan& pl)
{
    const int d = pb.P.d, r = pb.P.r;
    tcg::k_theta_images64<<<kSMs * 4, 256, 0, pb.stream>>>(pb.theta(), d, r, pl.NCB, pb.ctl(), pl.img_hi, pl.img_lo);
    tcg::k_pass2_tcg<<<pl.g2, tcg::NTHREADS, pl.smem2, pb.stream>>>(
        pl.tmX, pl.img_hi, pl.img_lo, pb.U, pb.ybar(), pb.p(), pb.alpha_s(), pb.ctl(), pb.P.n, d, r, pl.NCB,
        pb.P.alpha, pb.P.K, pb.P.eps_d, pb.part2(), pb.p());
    pb.count(2);
}

}  // namespace gemnlr
