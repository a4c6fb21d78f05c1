// Warp-level tensor-core variant of the skinny-shape family (d in {64, 128}, r in {8, 16}).
//
// Same structure as the FFMA family (persistent CTAs, producer warp + 8 consumer warps, TMA tile
// loads with 128-byte swizzle into an mbarrier ring, vector work fused into the first product,
// last-block reductions), but the inner products run on mma.sync.m16n8k8 TF32 with the 3-product
// split (x = hi + lo, hi exactly representable in TF32; hi*hi' + lo*hi' + hi*lo'), which keeps FP32
// accuracy.  At r = 16 the tcgen05 path cannot help (an MMA instruction costs ~130 cycles whatever
// its N), while the FFMA kernels are bound by shared-memory operand traffic and issue slots; with
// register fragments one ldmatrix feeds 6 MMAs of 1024 MACs each.
//
//  * First product (k_pass1_mma): a warp owns RW rows of the tile (RW / 8 k-steps).  After the
//    row-local vector phase it accumulates Theta = X-hat^T U for its rows: A = X-hat^T (features
//    on M, D/16 tiles; fragments by transposed scalar loads from the swizzled tile), B = U
//    (columns on N, R/8 tiles), FP32 accumulators in registers for the whole kernel.
//  * Second product (k_pass2_mma): a warp owns 16 rows (one M tile); A = X-hat rows via ldmatrix,
//    B = Theta^T hi / lo images built once per CTA in shared memory (row stride D + 4 floats: no
//    bank conflicts), epilogue of Eq. "entrywise-fusion" on the accumulator fragments.
#include "nlr_common.cuh"
#include "device_utils.cuh"
#include "fin_logic.cuh"
#include "pipeline.cuh"
#include "tc_common.cuh"
#include "ffma_family.cuh"
#include "mma_common.cuh"

namespace gemnlr {
namespace mma {

// ------------------------------------------------------------------------------------------------
template <int D, int R, int TM, int NST>
__global__ void __launch_bounds__(NTHREADS, 1)
k_pass1_mma(const __grid_constant__ CUtensorMap tmX, const float* __restrict__ U,
            float* __restrict__ ytilde, float* __restrict__ ybar, Ctl* __restrict__ ctl,
            const float* __restrict__ p, int64_t n, double gamma, double* __restrict__ part)
{
    constexpr int RW = TM / NCW;            // rows of a tile owned by one warp
    constexpr int LPR = 32 / RW;            // lanes per row in the vector phase
    constexpr int CPL = R / LPR;            // columns per lane in the vector phase
    constexpr int MT = D / 16, NT = R / 8, KS = RW / 8;
    constexpr int XB = TM * D * 4, UB = TM * R * 4, STAGE = XB + UB;
    static_assert(RW % 8 == 0 && LPR >= 1 && LPR * RW == 32 && CPL % 4 == 0 && CPL * LPR == R, "mapping");
    static_assert(XB % 1024 == 0 && UB % 1024 == 0 && D % 32 == 0 && R % 8 == 0, "stage alignment");
    static_assert(NCW * D * R * 4 <= NST * STAGE, "reduction scratch fits in the stage ring");

    grid_dep_launch();
    grid_dep_wait();                        // the previous kernel's U, p and control block
    if (ctl->stopped) return;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t bars[2 * NST];
    __shared__ uint32_t abort_flag;
    __shared__ double sred_s[NCW][R];
    __shared__ double sred_q[2][NCW];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bar_base = smem_u32(bars);
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (NST + s); };
    if (threadIdx.x == 0) {
        for (int s = 0; s < NST; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), NCW); }
        abort_flag = 0;
        fence_barrier_init();
    }
    __syncthreads();

    const int64_t n_tiles = (n + TM - 1) / TM;
    const float cf = ctl->c_f;
    const int dual = ctl->dual_pending;

    float acc[MT][NT][4];
    float s_acc[CPL];
    double qq = 0.0, yq = 0.0;
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int nn = 0; nn < NT; ++nn)
#pragma unroll
            for (int k = 0; k < 4; ++k) acc[m][nn][k] = 0.f;
#pragma unroll
    for (int c = 0; c < CPL; ++c) s_acc[c] = 0.f;

    if (warp == NCW) {
        if (lane == 0) {
            int it = 0;
            for (int64_t t = blockIdx.x; t < n_tiles; t += gridDim.x, ++it) {
                const int s = it % NST;
                if (it >= NST) mbar_wait(empty_bar(s), ((it / NST) - 1) & 1, &abort_flag, ctl);
                if (abort_flag) break;
                const int64_t row0 = t * TM;
                const int rows = (n - row0 < TM) ? (int)(n - row0) : TM;
                const uint32_t dst = smem_base + (uint32_t)s * STAGE;
                mbar_expect_tx(full_bar(s), (uint32_t)(XB + rows * R * 4));
#pragma unroll
                for (int b = 0; b < D / 32; ++b)
                    tma_load_2d(dst + b * (TM * 128), &tmX, b * 32, (int)row0, full_bar(s));
                bulk_load_1d(dst + XB, U + row0 * R, (uint32_t)(rows * R * 4), full_bar(s));
            }
        }
    } else {
        const int v_row = lane / LPR, v_sub = lane % LPR;
        const int g = lane >> 2, tq = lane & 3;                 // MMA fragment coordinates
        float preg[CPL];
#pragma unroll
        for (int c = 0; c < CPL; ++c) preg[c] = p[v_sub * CPL + c];
        float yt_next;
        {
            const int64_t row_f = (int64_t)blockIdx.x * TM + warp * RW + v_row;
            yt_next = (row_f < n) ? ytilde[row_f] : 0.f;
        }
        int it = 0;
        for (int64_t t = blockIdx.x; t < n_tiles; t += gridDim.x, ++it) {
            const int s = it % NST;
            const uint32_t xs = smem_base + (uint32_t)s * STAGE;
            const uint32_t us = xs + XB;
            const int rl_v = warp * RW + v_row;
            const int64_t row_v = t * TM + rl_v;
            const bool valid = row_v < n;
            // ytilde of this tile was requested one tile ago (its DRAM latency would otherwise stall
            // every warp once per tile); request the next tile's now
            float yt = yt_next;
            {
                const int64_t row_n = row_v + (int64_t)gridDim.x * TM;
                yt_next = (row_n < n) ? ytilde[row_n] : 0.f;
            }
            mbar_wait(full_bar(s), (it / NST) & 1, &abort_flag, ctl);

            // ---- vector phase on the warp's own rows (u written back into the stage) ----
            {
                const uint32_t ua = us + (uint32_t)(rl_v * R + v_sub * CPL) * 4;
                float u[CPL];
#pragma unroll
                for (int c4 = 0; c4 < CPL / 4; ++c4) {
                    float4 w = lds128(ua + 16 * c4);
                    u[4 * c4 + 0] = valid ? cf * w.x : 0.f;
                    u[4 * c4 + 1] = valid ? cf * w.y : 0.f;
                    u[4 * c4 + 2] = valid ? cf * w.z : 0.f;
                    u[4 * c4 + 3] = valid ? cf * w.w : 0.f;
                }
                float dot = 0.f;
#pragma unroll
                for (int c = 0; c < CPL; ++c) dot = fmaf(u[c], preg[c], dot);
#pragma unroll
                for (int o = 1; o < LPR; o <<= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
                const float q = dot - 1.0f;
                if (dual) yt = (float)((double)yt + gamma * (double)q);
                const float yb = (float)((double)yt + gamma * (double)q);
                if (valid && v_sub == 0) {
                    if (dual) ytilde[row_v] = yt;
                    ybar[row_v] = yb;
                    qq = fma((double)q, (double)q, qq);
                    yq = fma((double)yt, (double)q, yq);
                }
#pragma unroll
                for (int c = 0; c < CPL; ++c) s_acc[c] = fmaf(u[c], yb, s_acc[c]);
#pragma unroll
                for (int c4 = 0; c4 < CPL / 4; ++c4)
                    sts128(ua + 16 * c4, make_float4(u[4 * c4], u[4 * c4 + 1], u[4 * c4 + 2], u[4 * c4 + 3]));
            }
            __syncwarp();

            // ---- Theta phase: per k-step of 8 rows, A = X-hat^T (M = features), B = u (N = columns) ----
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                // The 8 rows of a k-step may sit on the MMA's k index in any order as long as A and B agree:
                // k = tq -> row ka, k = tq + 4 -> row kb with ka in {0, 3, 4, 7}, kb in {1, 2, 5, 6}, which
                // makes the transposed A loads hit 32 distinct banks of the swizzled tile.
                const int ka = warp * RW + ks * 8 + 2 * tq + (tq & 1);
                const int kb = warp * RW + ks * 8 + 2 * tq + 1 - (tq & 1);
                // B fragments: b0 = u[row ka][col g], b1 = u[row kb][col g]
                uint32_t bh[NT][2], bl[NT][2];
#pragma unroll
                for (int nn = 0; nn < NT; ++nn) {
                    split_tf32(lds32(us + (uint32_t)(ka * R + 8 * nn + g) * 4), bh[nn][0], bl[nn][0]);
                    split_tf32(lds32(us + (uint32_t)(kb * R + 8 * nn + g) * 4), bh[nn][1], bl[nn][1]);
                }
                // A fragment (16 features x 8 rows): a0 = x[row ka][f g], a1 = x[row ka][f g + 8],
                //                                    a2 = x[row kb][f g], a3 = x[row kb][f g + 8].
                // M tiles go in pairs and the three products are issued product by product, so that
                // MMAs on the same accumulator are 2 NT instructions apart (their latency is ~4 issue slots).
                constexpr int MP = (MT >= 2) ? 2 : 1;
#pragma unroll
                for (int m0 = 0; m0 < MT; m0 += MP) {
                    uint32_t ah[MP][4], al[MP][4];
#pragma unroll
                    for (int mm = 0; mm < MP; ++mm) {
                        const int f0 = 16 * (m0 + mm) + g, f1 = f0 + 8;
                        split_tf32(lds32(xs + x_chunk_off<TM>(ka, f0 >> 2) + (f0 & 3) * 4), ah[mm][0], al[mm][0]);
                        split_tf32(lds32(xs + x_chunk_off<TM>(ka, f1 >> 2) + (f1 & 3) * 4), ah[mm][1], al[mm][1]);
                        split_tf32(lds32(xs + x_chunk_off<TM>(kb, f0 >> 2) + (f0 & 3) * 4), ah[mm][2], al[mm][2]);
                        split_tf32(lds32(xs + x_chunk_off<TM>(kb, f1 >> 2) + (f1 & 3) * 4), ah[mm][3], al[mm][3]);
                    }
#pragma unroll
                    for (int mm = 0; mm < MP; ++mm)
#pragma unroll
                        for (int nn = 0; nn < NT; ++nn) mma_tf32(acc[m0 + mm][nn], ah[mm], bh[nn][0], bh[nn][1]);
#pragma unroll
                    for (int mm = 0; mm < MP; ++mm)
#pragma unroll
                        for (int nn = 0; nn < NT; ++nn) mma_tf32(acc[m0 + mm][nn], al[mm], bh[nn][0], bh[nn][1]);
#pragma unroll
                    for (int mm = 0; mm < MP; ++mm)
#pragma unroll
                        for (int nn = 0; nn < NT; ++nn) mma_tf32(acc[m0 + mm][nn], ah[mm], bl[nn][0], bl[nn][1]);
                }
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_bar(s));
        }
    }
    __syncthreads();

    // ---- CTA partials: Theta (sum over warps), s, sum q^2, sum ytilde q ----
    float* red = reinterpret_cast<float*>(smem);       // [NCW][D * R]
    if (warp < NCW) {
        const int g = lane >> 2, tq = lane & 3;
        // accumulator fragment: c0, c1 = (row g, cols 2 tq, 2 tq + 1); c2, c3 = (row g + 8, same cols)
#pragma unroll
        for (int m = 0; m < MT; ++m)
#pragma unroll
            for (int nn = 0; nn < NT; ++nn) {
                float* o = red + (size_t)warp * (D * R);
                o[(16 * m + g) * R + 8 * nn + 2 * tq] = acc[m][nn][0];
                o[(16 * m + g) * R + 8 * nn + 2 * tq + 1] = acc[m][nn][1];
                o[(16 * m + g + 8) * R + 8 * nn + 2 * tq] = acc[m][nn][2];
                o[(16 * m + g + 8) * R + 8 * nn + 2 * tq + 1] = acc[m][nn][3];
            }
        const int v_sub = lane % LPR;
#pragma unroll
        for (int c = 0; c < CPL; ++c) {
            float v = s_acc[c];
#pragma unroll
            for (int o = LPR; o < 32; o <<= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if (lane < LPR) sred_s[warp][v_sub * CPL + c] = (double)v;
        }
        qq = warp_sum(qq);
        yq = warp_sum(yq);
        if (lane == 0) { sred_q[0][warp] = qq; sred_q[1][warp] = yq; }
    }
    __syncthreads();
    double* out = part + (size_t)blockIdx.x * (D * R + R + 2);
    for (int e = threadIdx.x; e < D * R; e += NTHREADS) {
        double v = 0.0;
#pragma unroll
        for (int w = 0; w < NCW; ++w) v += (double)red[(size_t)w * (D * R) + e];
        out[e] = v;
    }
    if (threadIdx.x < R) {
        double v = 0.0;
#pragma unroll
        for (int w = 0; w < NCW; ++w) v += sred_s[w][threadIdx.x];
        out[D * R + threadIdx.x] = v;
    }
    if (threadIdx.x == 0) {
        double a = 0.0, b = 0.0;
#pragma unroll
        for (int w = 0; w < NCW; ++w) { a += sred_q[0][w]; b += sred_q[1][w]; }
        out[D * R + R] = a;
        out[D * R + R + 1] = b;
    }
}

// ------------------------------------------------------------------------------------------------
template <int D, int R, int NST>
__global__ void __launch_bounds__(NTHREADS, 1)
k_pass2_mma(const __grid_constant__ CUtensorMap tmX, const float* __restrict__ theta,
            float* __restrict__ U, const float* __restrict__ ybar, const float* __restrict__ p,
            const float* __restrict__ alpha_s, Ctl* __restrict__ ctl, int64_t n, float alpha, int K,
            double eps_d, double* __restrict__ part, float* __restrict__ p_out)
{
    constexpr int TM = NCW * 16;               // one 16-row M tile per consumer warp
    constexpr int NT = R / 8;
    constexpr int XB = TM * D * 4;
    constexpr int TS = D + 4;                  // row stride (floats) of the Theta^T images: conflict-free ldmatrix rows
    constexpr int PS = 4 + R;
    static_assert(XB % 1024 == 0 && D % 32 == 0 && R % 8 == 0 && NT <= 2, "shape");

    grid_dep_launch();
    grid_dep_wait();                        // Theta, s and the control block of the reduction kernel before this one
    if (ctl->stopped) return;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t bars[2 * NST];
    __shared__ uint32_t abort_flag;
    __shared__ double sred[32];
    __shared__ double scol[NCW][R];
    __shared__ int is_last;
    __shared__ double sc;
    __shared__ int sok;
    float* th_hi = reinterpret_cast<float*>(smem + (size_t)NST * XB);      // [16 rows (cols of Theta, zero beyond R)][TS]
    float* th_lo = th_hi + 16 * TS;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t thh = smem_u32(th_hi), thl = smem_u32(th_lo);
    const uint32_t bar_base = smem_u32(bars);
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (NST + s); };
    if (threadIdx.x == 0) {
        for (int s = 0; s < NST; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), NCW); }
        abort_flag = 0;
        fence_barrier_init();
    }
    for (int e = threadIdx.x; e < 16 * D; e += NTHREADS) {
        const int col = e / D, f = e % D;
        const float v = (col < R) ? theta[(size_t)f * R + col] : 0.f;
        const float h = tf32_hi(v);
        th_hi[col * TS + f] = h;
        th_lo[col * TS + f] = v - h;
    }
    __syncthreads();

    const int64_t n_tiles = (n + TM - 1) / TM;
    const float cf = ctl->c_f;
    const float two_alpha = 2.0f * alpha;
    double sa = 0.0, sb = 0.0, sh = 0.0;
    double csum[NT][2];
#pragma unroll
    for (int nn = 0; nn < NT; ++nn) { csum[nn][0] = 0.0; csum[nn][1] = 0.0; }

    if (warp == NCW) {
        if (lane == 0) {
            int it = 0;
            for (int64_t t = blockIdx.x; t < n_tiles; t += gridDim.x, ++it) {
                const int s = it % NST;
                if (it >= NST) mbar_wait(empty_bar(s), ((it / NST) - 1) & 1, &abort_flag, ctl);
                if (abort_flag) break;
                const uint32_t dst = smem_base + (uint32_t)s * XB;
                mbar_expect_tx(full_bar(s), (uint32_t)XB);
#pragma unroll
                for (int b = 0; b < D / 32; ++b)
                    tma_load_2d(dst + b * (TM * 128), &tmX, b * 32, (int)(t * TM), full_bar(s));
            }
        }
    } else {
        const int g = lane >> 2, tq = lane & 3;
        // ldmatrix row addresses: lane l supplies row (l & 7) of matrix l >> 3
        const int a_row = warp * 16 + (lane & 7) + 8 * ((lane >> 3) & 1);   // A: matrices (rows 0-7 | 8-15) x (chunk c | c + 1)
        const int a_cadd = lane >> 4;
        // B: matrices (n-tile 0 | 1) x (k 0-3 | 4-7): Theta^T row = 8 (l >> 4) + (l & 7), feature offset 4 ((l >> 3) & 1)
        const uint32_t b_off = (uint32_t)(((8 * (lane >> 4) + (lane & 7)) * TS + 4 * ((lane >> 3) & 1)) * 4);
        float pk[NT][2], ask[NT][2];
#pragma unroll
        for (int nn = 0; nn < NT; ++nn)
#pragma unroll
            for (int e = 0; e < 2; ++e) { pk[nn][e] = p[8 * nn + 2 * tq + e]; ask[nn][e] = alpha_s[8 * nn + 2 * tq + e]; }
        int it = 0;
        for (int64_t t = blockIdx.x; t < n_tiles; t += gridDim.x, ++it) {
            const int s = it % NST;
            const uint32_t xs = smem_base + (uint32_t)s * XB;
            const int64_t row0 = t * TM + warp * 16 + g, row1 = row0 + 8;
            const bool v0 = row0 < n, v1 = row1 < n;
            // old factor entries (cols 8 nn + 2 tq, + 1 of rows row0, row1) and ybar, issued before the wait
            float2 w0[NT], w1[NT];
#pragma unroll
            for (int nn = 0; nn < NT; ++nn) {
                w0[nn] = v0 ? __ldcg(reinterpret_cast<const float2*>(U + row0 * R + 8 * nn + 2 * tq)) : make_float2(0.f, 0.f);
                w1[nn] = v1 ? __ldcg(reinterpret_cast<const float2*>(U + row1 * R + 8 * nn + 2 * tq)) : make_float2(0.f, 0.f);
            }
            const float yb0 = v0 ? ybar[row0] : 0.f;
            const float yb1 = v1 ? ybar[row1] : 0.f;
            mbar_wait(full_bar(s), (it / NST) & 1, &abort_flag, ctl);
            const bool dead = abort_flag != 0;          // a wait ran out: the tile's data cannot be trusted, U is left as it is
            // one accumulator per product (hi*hi, lo*hi, hi*lo) and N tile: 3 NT independent MMA chains
            float acc[NT][4], acc1[NT][4], acc2[NT][4];
#pragma unroll
            for (int nn = 0; nn < NT; ++nn)
#pragma unroll
                for (int k = 0; k < 4; ++k) acc[nn][k] = acc1[nn][k] = acc2[nn][k] = 0.f;
#pragma unroll 4
            for (int ks = 0; ks < D / 8; ++ks) {
                uint32_t a[4], ah[4], al[4], bh[4], bl[4];
                ldmatrix_x4(xs + x_chunk_off<TM>(a_row, 2 * ks + a_cadd), a);
                ldmatrix_x4(thh + b_off + (uint32_t)ks * 32, bh);
                ldmatrix_x4(thl + b_off + (uint32_t)ks * 32, bl);
#pragma unroll
                for (int k = 0; k < 4; ++k) split_tf32(__uint_as_float(a[k]), ah[k], al[k]);
#pragma unroll
                for (int nn = 0; nn < NT; ++nn) mma_tf32(acc[nn], ah, bh[2 * nn], bh[2 * nn + 1]);
#pragma unroll
                for (int nn = 0; nn < NT; ++nn) mma_tf32(acc1[nn], al, bh[2 * nn], bh[2 * nn + 1]);
#pragma unroll
                for (int nn = 0; nn < NT; ++nn) mma_tf32(acc2[nn], ah, bl[2 * nn], bl[2 * nn + 1]);
            }
#pragma unroll
            for (int nn = 0; nn < NT; ++nn)
#pragma unroll
                for (int k = 0; k < 4; ++k) acc[nn][k] += acc1[nn][k] + acc2[nn][k];
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_bar(s));

            // ---- epilogue: accumulator fragment c0, c1 = (row0, cols 2 tq, +1), c2, c3 = (row1, same cols) ----
            const float nay0 = -alpha * yb0, nay1 = -alpha * yb1;
#pragma unroll
            for (int nn = 0; nn < NT; ++nn) {
                const float wold[4] = {w0[nn].x, w0[nn].y, w1[nn].x, w1[nn].y};
                float wn[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const bool live = (k < 2) ? v0 : v1;
                    const float u = cf * wold[k];
                    float v = fmaf(two_alpha, acc[nn][k], u);
                    v = fmaf((k < 2) ? nay0 : nay1, pk[nn][k & 1], v);
                    v -= ask[nn][k & 1];
                    const float w = live ? fmaxf(v, 0.f) : 0.f;
                    const double wd = (double)w, ud = (double)u;
                    sa = fma(wd, wd, sa);
                    sb = fma(ud, ud, sb);
                    sh = fma(wd, ud, sh);
                    csum[nn][k & 1] += wd;
                    wn[k] = w;
                }
                if (v0 && !dead) __stcg(reinterpret_cast<float2*>(U + row0 * R + 8 * nn + 2 * tq), make_float2(wn[0], wn[1]));
                if (v1 && !dead) __stcg(reinterpret_cast<float2*>(U + row1 * R + 8 * nn + 2 * tq), make_float2(wn[2], wn[3]));
            }
        }
    }
    __syncthreads();

    // ---- CTA partial: a, b, h and the column sums of W ----
    sa = block_sum<NTHREADS>(sa, sred);
    sb = block_sum<NTHREADS>(sb, sred);
    sh = block_sum<NTHREADS>(sh, sred);
    if (warp < NCW) {
        const int tq = lane & 3;
#pragma unroll
        for (int nn = 0; nn < NT; ++nn)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                double v = csum[nn][e];
                v += __shfl_xor_sync(0xffffffffu, v, 4);      // over the 8 row groups g of the warp
                v += __shfl_xor_sync(0xffffffffu, v, 8);
                v += __shfl_xor_sync(0xffffffffu, v, 16);
                if (lane < 4) scol[warp][8 * nn + 2 * tq + e] = v;
            }
    }
    __syncthreads();
    double* out = part + (size_t)blockIdx.x * PS;
    if (threadIdx.x == 0) { out[0] = sa; out[1] = sb; out[2] = sh; out[3] = 0.0; }
    if (threadIdx.x < R) {
        double v = 0.0;
#pragma unroll
        for (int w = 0; w < NCW; ++w) v += scol[w][threadIdx.x];
        out[4 + threadIdx.x] = v;
    }
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
    double a = 0.0, b = 0.0, h = 0.0;
    for (int i = threadIdx.x; i < G; i += NTHREADS) {
        a += __ldcg(part + (size_t)i * PS + 0);
        b += __ldcg(part + (size_t)i * PS + 1);
        h += __ldcg(part + (size_t)i * PS + 2);
    }
    a = block_sum<NTHREADS>(a, sred);
    b = block_sum<NTHREADS>(b, sred);
    h = block_sum<NTHREADS>(h, sred);
    if (threadIdx.x == 0) {
        double c;
        sok = fin2_scalars(ctl, a, b, h, K, eps_d, &c) ? 1 : 0;
        sc = c;
        ctl->counter[1] = 0;
    }
    __syncthreads();
    if (!sok) return;
    if (threadIdx.x < R) {
        double v = 0.0;
        for (int i = 0; i < G; ++i) v += __ldcg(part + (size_t)i * PS + 4 + threadIdx.x);
        p_out[threadIdx.x] = (float)(sc * v);
    }
}

// ------------------------------------------------------------------------------------------------
template <int D, int R, int TM1, int NST1, int NST2>
struct Shape {
    static constexpr int TM2 = NCW * 16;
    static constexpr size_t smem1 = (size_t)NST1 * (TM1 * D * 4 + TM1 * R * 4) + 1024;
    static constexpr size_t smem2 = (size_t)NST2 * (TM2 * D * 4) + (size_t)2 * 16 * (D + 4) * 4 + 1024;
    static bool plan(const Problem& pb, FfmaPlan* pl)
    {
        if (!make_tensor_map_2d(&pl->tm1, pb.X, pb.P.n, D, TM1, 32)) return false;
        if (!make_tensor_map_2d(&pl->tm2, pb.X, pb.P.n, D, TM2, 32)) return false;
        const int64_t t1 = (pb.P.n + TM1 - 1) / TM1, t2 = (pb.P.n + TM2 - 1) / TM2;
        pl->g1 = (int)(t1 < kSMs ? t1 : kSMs);
        pl->g2 = (int)(t2 < kSMs ? t2 : kSMs);
        if (cudaFuncSetAttribute(k_pass1_mma<D, R, TM1, NST1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem1) != cudaSuccess) return false;
        if (cudaFuncSetAttribute(k_pass2_mma<D, R, NST2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem2) != cudaSuccess) return false;
        return true;
    }
    static void pass1(const Problem& pb, const FfmaPlan& pl)
    {
        launch_pdl(k_pass1_mma<D, R, TM1, NST1>, dim3(pl.g1), dim3(NTHREADS), smem1, pb.stream,
                   pl.tm1, pb.U, pb.ytilde(), pb.ybar(), pb.ctl(), pb.p(), pb.P.n, pb.gamma, pb.part1());
    }
    static void pass2(const Problem& pb, const FfmaPlan& pl)
    {
        launch_pdl(k_pass2_mma<D, R, NST2>, dim3(pl.g2), dim3(NTHREADS), smem2, pb.stream,
                   pl.tm2, pb.theta(), pb.U, pb.ybar(), pb.p(), pb.alpha_s(), pb.ctl(), pb.P.n, pb.P.alpha, pb.P.K,
                   pb.P.eps_d, pb.part2(), pb.p());
    }
};

//                   D    R   TM1 NST1 NST2
using S_128_16 = Shape<128, 16, 64,  5,  3>;
using S_64_16  = Shape<64,  16, 128, 4,  6>;
using S_64_8   = Shape<64,  8,  128, 5,  6>;
using S_128_8  = Shape<128, 8,  128, 3,  3>;

}  // namespace mma


bool mma_plan(const Problem& pb, FfmaPlan* pl)
{
    const int d = pb.P.d, r = pb.P.r;
    int id = -1;
    if (d == 128 && r == 16) id = 0;
    else if (d == 64 && r == 16) id = 1;
    else if (d == 64 && r == 8) id = 2;
    else if (d == 128 && r == 8) id = 3;
    // wide factors: r in a multiple-of-4 window below the instantiated N-tile count
    if (id < 0 && r % 4 == 0) {
        const int nt = (r + 7) / 8;
        if (d == 64 && nt == 13) id = 100;
        else if (d == 64 && nt == 8) id = 101;
        else if (d == 32 && nt == 13) id = 102;
    }
    if (id < 0 || pb.P.n < 1024 || pb.P.n > 2000000000ll) return false;
    pl->shape_id = id;
    if (id >= 100) return mmaw_plan(pb, pl);
    using namespace mma;
    switch (id) {
        case 0: return S_128_16::plan(pb, pl);
        case 1: return S_64_16::plan(pb, pl);
        case 2: return S_64_8::plan(pb, pl);
        case 3: return S_128_8::plan(pb, pl);
    }
    return false;
}

void mma_launch_first(const Problem& pb, const FfmaPlan& pl, int mode)
{
    if (pl.shape_id >= 100) { mmaw_pass1(pb, pl); pb.count(1); red1_fused_launch(pb, pl.g1, mode); return; }
    using namespace mma;
    switch (pl.shape_id) {
        case 0: S_128_16::pass1(pb, pl); break;
        case 1: S_64_16::pass1(pb, pl); break;
        case 2: S_64_8::pass1(pb, pl); break;
        case 3: S_128_8::pass1(pb, pl); break;
    }
    pb.count(1);
    red1_fused_launch(pb, pl.g1, mode);
}

void mma_launch_second(const Problem& pb, const FfmaPlan& pl)
{
    if (pl.shape_id >= 100) { mmaw_pass2(pb, pl); pb.count(1); return; }
    using namespace mma;
    switch (pl.shape_id) {
        case 0: S_128_16::pass2(pb, pl); break;
        case 1: S_64_16::pass2(pb, pl); break;
        case 2: S_64_8::pass2(pb, pl); break;
        case 3: S_128_8::pass2(pb, pl); break;
    }
    pb.count(1);
}

}  // namespace gemnlr
