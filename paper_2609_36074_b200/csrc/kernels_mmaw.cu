// Warp-level tensor-core kernels for wide factors (r up to 104 in N tiles of 8 columns; U rows keep
// their stride of r floats): mma.sync.m16n8k8 TF32 with the 3-product split, 64-row tiles holding
// the X-hat rows (TMA, 128-byte swizzle) and the matching U rows (one bulk copy: the rows of a tile
// are contiguous in global memory).
//
//  * First product (k_pass1_mmaw): the 8 consumer warps share the row-local vector phase of a tile
//    (a warp takes 8 rows, lanes over columns: q = u.p - 1, ytilde / ybar, s += u ybar; the scaled u
//    is written back into the stage).  For the contraction a warp is (row group, N quarter): it holds
//    Theta[all features][its 3-4 N tiles] for the rows of its half of every tile, so an X-hat^T
//    fragment serves 3-4 N tiles and a U fragment D/16 M tiles.  Vector phase and contraction meet
//    through an mbarrier per stage (arrive after the vector phase, wait before the MMAs of that
//    stage) and the vector phase runs one tile ahead, so no warp waits for the slowest one.
//  * Second product (k_pass2_mmaw): a warp is (16-row group, N half); A fragments by ldmatrix from
//    the swizzled tile, B fragments by ldmatrix from Theta^T hi / lo images built once per CTA; the
//    old factor entries come from the stage, the new ones go to global memory from the accumulator
//    fragments (each 4-lane group writes one full 32-byte sector).
#include "nlr_common.cuh"
#include "device_utils.cuh"
#include "fin_logic.cuh"
#include "mma_common.cuh"

namespace gemnlr {
namespace mmaw {
using namespace mma;

constexpr int TM = 64;

__device__ __forceinline__ float2 lds64(uint32_t addr)
{
    float2 v;
    asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr));
    return v;
}

__device__ __forceinline__ void sts32(uint32_t addr, float v)
{
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}

// ------------------------------------------------------------------------------------------------
template <int D, int NT, int NST>
__global__ void __launch_bounds__(NTHREADS, 1)
k_pass1_mmaw(const __grid_constant__ CUtensorMap tmX, const float* __restrict__ U,
             float* __restrict__ ytilde, float* __restrict__ ybar, Ctl* __restrict__ ctl,
             const float* __restrict__ p, int64_t n, int r, double gamma, double* __restrict__ part)
{
    constexpr int RP = NT * 8;
    constexpr int MT = D / 16;
    constexpr int RG = 2, NQ = 4;                  // row groups x N quarters = 8 warps
    constexpr int NTQ = (NT + NQ - 1) / NQ;        // N tiles of the largest quarter
    constexpr int ROWS_G = TM / RG, KS = ROWS_G / 8;
    constexpr int RPW = TM / NCW;                  // rows per warp in the vector phase
    constexpr int NJ = (RP + 31) / 32;             // columns per lane in the vector phase
    constexpr int XB = TM * D * 4, UB = (TM * RP * 4 + 1023) / 1024 * 1024, STAGE = XB + UB;
    static_assert(RG * NQ == NCW && RPW == 8 && NT >= NQ, "mapping");
    static_assert(XB % 1024 == 0 && D % 32 == 0, "stage alignment");
    static_assert(RG * D * RP * 4 <= NST * STAGE, "reduction scratch fits in the stage ring");

    if (ctl->stopped) return;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t bars[3 * NST];
    __shared__ uint32_t abort_flag;
    __shared__ double sred_s[NCW][NJ * 32];
    __shared__ double sred_q[2][NCW];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bar_base = smem_u32(bars);
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (NST + s); };
    auto uready_bar = [&](int s) { return bar_base + 8u * (2 * NST + s); };
    if (threadIdx.x == 0) {
        for (int s = 0; s < NST; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), NCW);
            mbar_init(uready_bar(s), NCW);
        }
        abort_flag = 0;
        fence_barrier_init();
    }
    __syncthreads();

    const int64_t n_tiles = (n + TM - 1) / TM;
    const float cf = ctl->c_f;
    const int dual = ctl->dual_pending;

    float acc[MT][NTQ][4];
    float s_acc[NJ];
    double qq = 0.0, yq = 0.0;
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int e = 0; e < NTQ; ++e)
#pragma unroll
            for (int k = 0; k < 4; ++k) acc[m][e][k] = 0.f;
#pragma unroll
    for (int j = 0; j < NJ; ++j) s_acc[j] = 0.f;

    // contraction role of this warp: row group rg, N tiles [t0, t0 + ntq); the quarter with the extra
    // tile sits on a different scheduler in the two row groups
    const int rg = warp >> 2, qd = ((warp & 3) + rg) & 3;
    const int t0 = qd * (NT / NQ) + (qd < NT % NQ ? qd : NT % NQ);
    const int ntq = NT / NQ + (qd < NT % NQ ? 1 : 0);

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
                mbar_expect_tx(full_bar(s), (uint32_t)(XB + rows * r * 4));
#pragma unroll
                for (int b = 0; b < D / 32; ++b)
                    tma_load_2d(dst + b * (TM * 128), &tmX, b * 32, (int)row0, full_bar(s));
                bulk_load_1d(dst + XB, U + row0 * r, (uint32_t)(rows * r * 4), full_bar(s));
            }
        }
    } else {
        const int g = lane >> 2, tq = lane & 3;
        float preg[NJ];
#pragma unroll
        for (int j = 0; j < NJ; ++j) preg[j] = (lane + 32 * j < r) ? p[lane + 32 * j] : 0.f;

        // per-thread address constants of the contraction phase
        const uint32_t r4 = (uint32_t)r * 4, r32 = 8 * r4;
        const uint32_t a_base = (uint32_t)(rg * ROWS_G * 128);
        const uint32_t b_base = (uint32_t)(((rg * ROWS_G + 2 * tq) * r + 8 * t0 + g) * 4);
        uint32_t sw_a[4];       // (row ka | kb) x (feature g | g + 8) of M tile 0, relative to the row group's first row
        {
            const int gh = g >> 2, wd = (g & 3) * 4;
            const int ra = 2 * tq, rb = 2 * tq + 1;
            sw_a[0] = (uint32_t)(ra * 128 + (((gh) ^ ra) << 4) + wd);
            sw_a[1] = (uint32_t)(ra * 128 + (((gh + 2) ^ ra) << 4) + wd);
            sw_a[2] = (uint32_t)(rb * 128 + (((gh) ^ rb) << 4) + wd);
            sw_a[3] = (uint32_t)(rb * 128 + (((gh + 2) ^ rb) << 4) + wd);
        }
        uint32_t jmask = 0;     // columns lane + 32 j below r
#pragma unroll
        for (int j = 0; j < NJ; ++j)
            if (lane + 32 * j < r) jmask |= 1u << j;
        uint32_t okmask = 0;
#pragma unroll
        for (int e = 0; e < NTQ; ++e)
            if (e < ntq && 8 * (t0 + e) + g < r) okmask |= 1u << e;

        // vector phase of tile t (ring position it): this warp's 8 rows, 4 at a time, lanes over columns
        auto vector_phase = [&](int64_t t, int it) {
            const int s = it % NST;
            const uint32_t us = smem_base + (uint32_t)s * STAGE + XB;
            const int64_t vrow = t * TM + warp * RPW + lane;       // lane i < 8 keeps row i's ytilde / ybar
            const bool vlive = lane < RPW && vrow < n;
            float my_yt = vlive ? ytilde[vrow] : 0.f, my_yb = 0.f;
            mbar_wait(full_bar(s), (it / NST) & 1, &abort_flag, ctl);
            const uint32_t vb = us + (uint32_t)(warp * RPW * r + lane) * 4;
            const int rows_left = (n - t * TM - warp * RPW > RPW) ? RPW : (int)(n - t * TM - warp * RPW);   // may be <= 0
#pragma unroll 1
            for (int rb = 0; rb < RPW; rb += 4) {
                float u[4][NJ], dot[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const bool valid = rb + i < rows_left;
                    dot[i] = 0.f;
#pragma unroll
                    for (int j = 0; j < NJ; ++j) {
                        const bool ok = valid && ((jmask >> j) & 1);
                        const float w = ok ? lds32(vb + (uint32_t)(rb + i) * r4 + 128 * j) : 0.f;
                        u[i][j] = cf * w;
                        dot[i] = fmaf(u[i][j], preg[j], dot[i]);
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1)
#pragma unroll
                    for (int i = 0; i < 4; ++i) dot[i] += __shfl_xor_sync(0xffffffffu, dot[i], o);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const bool valid = rb + i < rows_left;
                    const float q = dot[i] - 1.0f;
                    float yt = __shfl_sync(0xffffffffu, my_yt, rb + i);
                    if (dual) yt = (float)((double)yt + gamma * (double)q);
                    const float yb = (float)((double)yt + gamma * (double)q);
                    if (lane == rb + i) { my_yt = yt; my_yb = yb; }
                    if (valid && lane == 0) {
                        qq = fma((double)q, (double)q, qq);
                        yq = fma((double)yt, (double)q, yq);
                    }
#pragma unroll
                    for (int j = 0; j < NJ; ++j) {
                        s_acc[j] = fmaf(u[i][j], yb, s_acc[j]);
                        if ((jmask >> j) & 1) sts32(vb + (uint32_t)(rb + i) * r4 + 128 * j, u[i][j]);
                    }
                }
            }
            if (vlive) {
                if (dual) ytilde[vrow] = my_yt;
                ybar[vrow] = my_yb;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(uready_bar(s));
        };

        int it = 0;
        if ((int64_t)blockIdx.x < n_tiles) vector_phase(blockIdx.x, 0);
        for (int64_t t = blockIdx.x; t < n_tiles; t += gridDim.x, ++it) {
            const int s = it % NST;
            const uint32_t xs = smem_base + (uint32_t)s * STAGE;
            const uint32_t us = xs + XB;
            if (t + gridDim.x < n_tiles) vector_phase(t + gridDim.x, it + 1);
            mbar_wait(uready_bar(s), (it / NST) & 1, &abort_flag, ctl);

            // ---- Theta phase: all features x N tiles [t0, t0 + ntq), rows of row group rg ----
            // k index tq -> row ka = 8 ks + 2 tq, tq + 4 -> row kb = ka + 1 (within the row group):
            // conflict-free transposed A loads from the swizzled tile, conflict-free B loads when the U
            // row stride is 4 mod 8 floats.  The swizzle term depends on (row & 7) only, so every address
            // is a per-thread constant plus ks * 1024 (A) or ks * 8 r floats (B).
            const uint32_t xa = xs + a_base, ua = us + b_base;
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                uint32_t bh[NTQ][2], bl[NTQ][2];
#pragma unroll
                for (int e = 0; e < NTQ; ++e) {
                    const bool ok = (okmask >> e) & 1;
                    split_tf32(ok ? lds32(ua + (uint32_t)ks * r32 + 32 * e) : 0.f, bh[e][0], bl[e][0]);
                    split_tf32(ok ? lds32(ua + (uint32_t)ks * r32 + r4 + 32 * e) : 0.f, bh[e][1], bl[e][1]);
                }
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                    // features f0 = 16 m + g, f1 = f0 + 8: 16-byte chunk 4 m + (g >> 2) (+ 2), i.e. box m >> 1,
                    // chunk-in-box bits toggled by 4 (m & 1) and 2 through the XOR swizzle
                    uint32_t ah[4], al[4];
                    const uint32_t box = (uint32_t)((m >> 1) * (TM * 128) + ks * 1024);
                    split_tf32(lds32(xa + box + (sw_a[0] ^ (64u * (m & 1)))), ah[0], al[0]);
                    split_tf32(lds32(xa + box + (sw_a[1] ^ (64u * (m & 1)))), ah[1], al[1]);
                    split_tf32(lds32(xa + box + (sw_a[2] ^ (64u * (m & 1)))), ah[2], al[2]);
                    split_tf32(lds32(xa + box + (sw_a[3] ^ (64u * (m & 1)))), ah[3], al[3]);
#pragma unroll
                    for (int e = 0; e < NTQ; ++e) if (e < ntq) mma_tf32(acc[m][e], ah, bh[e][0], bh[e][1]);
#pragma unroll
                    for (int e = 0; e < NTQ; ++e) if (e < ntq) mma_tf32(acc[m][e], al, bh[e][0], bh[e][1]);
#pragma unroll
                    for (int e = 0; e < NTQ; ++e) if (e < ntq) mma_tf32(acc[m][e], ah, bl[e][0], bl[e][1]);
                }
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_bar(s));
        }
    }
    __syncthreads();

    // ---- CTA partials: Theta (sum over row groups), s, sum q^2, sum ytilde q ----
    float* red = reinterpret_cast<float*>(smem);       // [RG][D * RP]
    if (warp < NCW) {
        const int g = lane >> 2, tq = lane & 3;
        float* o = red + (size_t)rg * (D * RP);
#pragma unroll
        for (int m = 0; m < MT; ++m)
#pragma unroll
            for (int e = 0; e < NTQ; ++e)
                if (e < ntq) {
                    const int c = 8 * (t0 + e) + 2 * tq;
                    o[(16 * m + g) * RP + c] = acc[m][e][0];
                    o[(16 * m + g) * RP + c + 1] = acc[m][e][1];
                    o[(16 * m + g + 8) * RP + c] = acc[m][e][2];
                    o[(16 * m + g + 8) * RP + c + 1] = acc[m][e][3];
                }
#pragma unroll
        for (int j = 0; j < NJ; ++j) sred_s[warp][lane + 32 * j] = (double)s_acc[j];
        qq = warp_sum(qq);
        yq = warp_sum(yq);
        if (lane == 0) { sred_q[0][warp] = qq; sred_q[1][warp] = yq; }
    }
    __syncthreads();
    double* out = part + (size_t)blockIdx.x * ((size_t)D * r + r + 2);
    for (int e = threadIdx.x; e < D * r; e += NTHREADS) {
        const int f = e / r, c = e - f * r;
        double v = 0.0;
#pragma unroll
        for (int w = 0; w < RG; ++w) v += (double)red[(size_t)w * (D * RP) + f * RP + c];
        out[e] = v;
    }
    for (int c = threadIdx.x; c < r; c += NTHREADS) {
        double v = 0.0;
#pragma unroll
        for (int w = 0; w < NCW; ++w) v += sred_s[w][c];
        out[D * r + c] = v;
    }
    if (threadIdx.x == 0) {
        double a = 0.0, b = 0.0;
#pragma unroll
        for (int w = 0; w < NCW; ++w) { a += sred_q[0][w]; b += sred_q[1][w]; }
        out[D * r + r] = a;
        out[D * r + r + 1] = b;
    }
}

// ------------------------------------------------------------------------------------------------
template <int D, int NT, int NST>
__global__ void __launch_bounds__(NTHREADS, 1)
k_pass2_mmaw(const __grid_constant__ CUtensorMap tmX, const float* __restrict__ theta,
             float* __restrict__ U, const float* __restrict__ ybar, const float* __restrict__ p,
             const float* __restrict__ alpha_s, Ctl* __restrict__ ctl, int64_t n, int r, float alpha, int K,
             double eps_d, double* __restrict__ part, float* __restrict__ p_out)
{
    constexpr int RP = NT * 8;
    constexpr int NH0 = (NT + 1) / 2;              // N tiles of the first half (the second takes NT - NH0)
    constexpr int NPH = (NH0 + 1) / 2;             // ldmatrix pairs per half
    constexpr int IMG_ROWS = (NH0 + 2 * NPH) * 8;  // a pair of the second half may reach one tile past NT
    constexpr int XB = TM * D * 4, UB = (TM * RP * 4 + 1023) / 1024 * 1024, STAGE = XB + UB;
    constexpr int TS = D + 4;                      // image row stride (floats): conflict-free ldmatrix rows
    static_assert(XB % 1024 == 0 && D % 32 == 0, "shape");

    if (ctl->stopped) return;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t bars[2 * NST];
    __shared__ uint32_t abort_flag;
    __shared__ double sred[32];
    __shared__ double scol[NCW][NH0 * 8];
    __shared__ float sp[RP + 8], sas[RP + 8];
    __shared__ int is_last;
    __shared__ double sc;
    __shared__ int sok;
    float* th_hi = reinterpret_cast<float*>(smem + (size_t)NST * STAGE);   // [IMG_ROWS (columns of Theta, zero beyond r)][TS]
    float* th_lo = th_hi + IMG_ROWS * TS;

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
    for (int e = threadIdx.x; e < IMG_ROWS * D; e += NTHREADS) {
        const int col = e / D, f = e % D;
        const float v = (col < r) ? theta[(size_t)f * r + col] : 0.f;
        const float h = tf32_hi(v);
        th_hi[col * TS + f] = h;
        th_lo[col * TS + f] = v - h;
    }
    for (int c = threadIdx.x; c < NCW * NH0 * 8; c += NTHREADS) scol[c / (NH0 * 8)][c % (NH0 * 8)] = 0.0;
    for (int c = threadIdx.x; c < RP + 8; c += NTHREADS) {
        sp[c] = (c < r) ? p[c] : 0.f;
        sas[c] = (c < r) ? alpha_s[c] : 0.f;
    }
    __syncthreads();

    const int64_t n_tiles = (n + TM - 1) / TM;
    const float cf = ctl->c_f;
    const float two_alpha = 2.0f * alpha;
    // role: 16-row group rgp, N half nh (halves alternate over the schedulers)
    const int rgp = warp >> 1, nh = (warp ^ (warp >> 2)) & 1;
    const int t0 = nh ? NH0 : 0, cnt = nh ? NT - NH0 : NH0;
    double sa = 0.0, sb = 0.0, sh = 0.0;
    // Column sums of W: FP32 over the 8 entries a thread meets in 4 tiles, then FP64 (shuffle tree over
    // the warp's row groups, accumulators in shared memory)
    float csf[NH0][2];
#pragma unroll
    for (int e = 0; e < NH0; ++e) { csf[e][0] = 0.f; csf[e][1] = 0.f; }
    auto flush_colsums = [&]() {
#pragma unroll
        for (int e = 0; e < NH0; ++e)
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                double v = (double)csf[e][x];
                v += __shfl_xor_sync(0xffffffffu, v, 4);
                v += __shfl_xor_sync(0xffffffffu, v, 8);
                v += __shfl_xor_sync(0xffffffffu, v, 16);
                if (lane < 4) scol[warp][8 * e + 2 * lane + x] += v;
                csf[e][x] = 0.f;
            }
    };

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
                mbar_expect_tx(full_bar(s), (uint32_t)(XB + rows * r * 4));
#pragma unroll
                for (int b = 0; b < D / 32; ++b)
                    tma_load_2d(dst + b * (TM * 128), &tmX, b * 32, (int)row0, full_bar(s));
                bulk_load_1d(dst + XB, U + row0 * r, (uint32_t)(rows * r * 4), full_bar(s));
            }
        }
    } else {
        const int g = lane >> 2, tq = lane & 3;
        // ldmatrix row addresses: lane l supplies row (l & 7) of matrix l >> 3
        const int a_row = rgp * 16 + (lane & 7) + 8 * ((lane >> 3) & 1);   // A: (rows 0-7 | 8-15) x (chunk c | c + 1)
        const int a_cadd = lane >> 4;
        // B: (tile tb | tb + 1) x (k 0-3 | 4-7): image row 8 (tb + (l >> 4)) + (l & 7), feature offset 4 ((l >> 3) & 1)
        const uint32_t b_off = (uint32_t)(((8 * (t0 + (lane >> 4)) + (lane & 7)) * TS + 4 * ((lane >> 3) & 1)) * 4);
        int it = 0;
        for (int64_t t = blockIdx.x; t < n_tiles; t += gridDim.x, ++it) {
            const int s = it % NST;
            const uint32_t xs = smem_base + (uint32_t)s * STAGE;
            const uint32_t us = xs + XB;
            const int rl0 = rgp * 16 + g, rl1 = rl0 + 8;
            const int64_t row0 = t * TM + rl0, row1 = row0 + 8;
            const bool v0 = row0 < n, v1 = row1 < n;
            const float yb0 = v0 ? ybar[row0] : 0.f;
            const float yb1 = v1 ? ybar[row1] : 0.f;
            mbar_wait(full_bar(s), (it / NST) & 1, &abort_flag, ctl);
            const bool dead = abort_flag != 0;          // a wait ran out: the tile's data cannot be trusted, U is left as it is
            float acc[NH0][4];
#pragma unroll
            for (int e = 0; e < NH0; ++e)
#pragma unroll
                for (int k = 0; k < 4; ++k) acc[e][k] = 0.f;
#pragma unroll 2
            for (int ks = 0; ks < D / 8; ++ks) {
                uint32_t a[4], ah[4], al[4];
                ldmatrix_x4(xs + x_chunk_off<TM>(a_row, 2 * ks + a_cadd), a);
                uint32_t bh[NPH][4], bl[NPH][4];
#pragma unroll
                for (int pe = 0; pe < NPH; ++pe)
                    if (2 * pe < cnt) {
                        ldmatrix_x4(thh + b_off + (uint32_t)(pe * 16 * TS * 4 + ks * 32), bh[pe]);
                        ldmatrix_x4(thl + b_off + (uint32_t)(pe * 16 * TS * 4 + ks * 32), bl[pe]);
                    }
#pragma unroll
                for (int k = 0; k < 4; ++k) split_tf32(__uint_as_float(a[k]), ah[k], al[k]);
                // product by product: MMAs on the same accumulator are cnt instructions apart
#pragma unroll
                for (int e = 0; e < NH0; ++e)
                    if (e < cnt) mma_tf32(acc[e], ah, bh[e >> 1][2 * (e & 1)], bh[e >> 1][2 * (e & 1) + 1]);
#pragma unroll
                for (int e = 0; e < NH0; ++e)
                    if (e < cnt) mma_tf32(acc[e], al, bh[e >> 1][2 * (e & 1)], bh[e >> 1][2 * (e & 1) + 1]);
#pragma unroll
                for (int e = 0; e < NH0; ++e)
                    if (e < cnt) mma_tf32(acc[e], ah, bl[e >> 1][2 * (e & 1)], bl[e >> 1][2 * (e & 1) + 1]);
            }
            // old factor entries of this warp's fragment positions, then the stage can be refilled
            float2 w0[NH0], w1[NH0];
#pragma unroll
            for (int e = 0; e < NH0; ++e) {
                const int c = 8 * (t0 + e) + 2 * tq;
                const bool ok = e < cnt && c < r;
                w0[e] = (ok && v0) ? lds64(us + (uint32_t)(rl0 * r + c) * 4) : make_float2(0.f, 0.f);
                w1[e] = (ok && v1) ? lds64(us + (uint32_t)(rl1 * r + c) * 4) : make_float2(0.f, 0.f);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_bar(s));

            // ---- epilogue: c0, c1 = (row0, cols c, c + 1), c2, c3 = (row1, same cols) ----
            const float nay0 = -alpha * yb0, nay1 = -alpha * yb1;
#pragma unroll
            for (int e = 0; e < NH0; ++e) {
                const int c = 8 * (t0 + e) + 2 * tq;
                const bool cok = e < cnt && c < r;
                const float wold[4] = {w0[e].x, w0[e].y, w1[e].x, w1[e].y};
                const float pk[2] = {sp[c], sp[c + 1]}, ak[2] = {sas[c], sas[c + 1]};
                float wn[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const bool live = ((k < 2) ? v0 : v1) && cok;
                    const float u = cf * wold[k];
                    float v = fmaf(two_alpha, acc[e][k], u);
                    v = fmaf((k < 2) ? nay0 : nay1, pk[k & 1], v);
                    v -= ak[k & 1];
                    const float w = live ? fmaxf(v, 0.f) : 0.f;
                    const double wd = (double)w, ud = (double)u;
                    sa = fma(wd, wd, sa);
                    sb = fma(ud, ud, sb);
                    sh = fma(wd, ud, sh);
                    csf[e][k & 1] += w;
                    wn[k] = w;
                }
                if (v0 && cok && !dead) *reinterpret_cast<float2*>(U + row0 * r + c) = make_float2(wn[0], wn[1]);
                if (v1 && cok && !dead) *reinterpret_cast<float2*>(U + row1 * r + c) = make_float2(wn[2], wn[3]);
            }
            if ((it & 3) == 3) flush_colsums();
        }
    }
    __syncthreads();

    sa = block_sum<NTHREADS>(sa, sred);
    sb = block_sum<NTHREADS>(sb, sred);
    sh = block_sum<NTHREADS>(sh, sred);
    if (warp < NCW) flush_colsums();
    __syncthreads();
    const int PS = 4 + r;
    double* out = part + (size_t)blockIdx.x * PS;
    if (threadIdx.x == 0) { out[0] = sa; out[1] = sb; out[2] = sh; out[3] = 0.0; }
    if (threadIdx.x < r) {
        // column c lives in the warps of its N half, at offset c - 8 * (first tile of the half)
        const int c = threadIdx.x, half = (c >= NH0 * 8) ? 1 : 0, off = c - half * NH0 * 8;
        double v = 0.0;
#pragma unroll
        for (int w = 0; w < NCW; ++w)
            if ((((w ^ (w >> 2)) & 1)) == half) v += scol[w][off];
        out[4 + c] = v;
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
    if (threadIdx.x < r) {
        double v = 0.0;
        for (int i = 0; i < G; ++i) v += __ldcg(part + (size_t)i * PS + 4 + threadIdx.x);
        p_out[threadIdx.x] = (float)(sc * v);
    }
}

// ------------------------------------------------------------------------------------------------
template <int D, int NT, int NST1, int NST2>
struct ShapeW {
    static constexpr int RP = NT * 8;
    static constexpr int NH0 = (NT + 1) / 2, NPH = (NH0 + 1) / 2, IMG_ROWS = (NH0 + 2 * NPH) * 8;
    static constexpr size_t stage = (size_t)TM * D * 4 + (TM * RP * 4 + 1023) / 1024 * 1024;
    static constexpr size_t smem1 = NST1 * stage + 1024;
    static constexpr size_t smem2 = NST2 * stage + (size_t)2 * IMG_ROWS * (D + 4) * 4 + 1024;
    static bool plan(const Problem& pb, FfmaPlan* pl)
    {
        if (!make_tensor_map_2d(&pl->tm1, pb.X, pb.P.n, D, TM, 32)) return false;
        pl->tm2 = pl->tm1;
        const int64_t t1 = (pb.P.n + TM - 1) / TM;
        pl->g1 = pl->g2 = (int)(t1 < kSMs ? t1 : kSMs);
        if (cudaFuncSetAttribute(k_pass1_mmaw<D, NT, NST1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem1) != cudaSuccess) return false;
        if (cudaFuncSetAttribute(k_pass2_mmaw<D, NT, NST2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem2) != cudaSuccess) return false;
        return true;
    }
    static void pass1(const Problem& pb, const FfmaPlan& pl)
    {
        k_pass1_mmaw<D, NT, NST1><<<pl.g1, NTHREADS, smem1, pb.stream>>>(
            pl.tm1, pb.U, pb.ytilde(), pb.ybar(), pb.ctl(), pb.p(), pb.P.n, pb.P.r, pb.gamma, pb.part1());
    }
    static void pass2(const Problem& pb, const FfmaPlan& pl)
    {
        k_pass2_mmaw<D, NT, NST2><<<pl.g2, NTHREADS, smem2, pb.stream>>>(
            pl.tm2, pb.theta(), pb.U, pb.ybar(), pb.p(), pb.alpha_s(), pb.ctl(), pb.P.n, pb.P.r, pb.P.alpha,
            pb.P.K, pb.P.eps_d, pb.part2(), pb.p());
    }
};

//                     D   NT NST1 NST2
using W_64_13 = ShapeW<64, 13, 4,  3>;
using W_64_8  = ShapeW<64, 8,  5,  4>;
using W_32_13 = ShapeW<32, 13, 5,  4>;

}  // namespace mmaw

bool mmaw_plan(const Problem& pb, FfmaPlan* pl)
{
    switch (pl->shape_id) {
        case 100: return mmaw::W_64_13::plan(pb, pl);
        case 101: return mmaw::W_64_8::plan(pb, pl);
        case 102: return mmaw::W_32_13::plan(pb, pl);
    }
    return false;
}

void mmaw_pass1(const Problem& pb, const FfmaPlan& pl)
{
    switch (pl.shape_id) {
        case 100: mmaw::W_64_13::pass1(pb, pl); break;
        case 101: mmaw::W_64_8::pass1(pb, pl); break;
        case 102: mmaw::W_32_13::pass1(pb, pl); break;
    }
}

void mmaw_pass2(const Problem& pb, const FfmaPlan& pl)
{
    switch (pl.shape_id) {
        case 100: mmaw::W_64_13::pass2(pb, pl); break;
        case 101: mmaw::W_64_8::pass2(pb, pl); break;
        case 102: mmaw::W_32_13::pass2(pb, pl); break;
    }
}

}  // namespace gemnlr
