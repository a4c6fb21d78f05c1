// Generic kernel family of the NLR iteration: works for every (n, d, r), plain global loads,
// shared-memory tiles and FP32 FFMA.  It is the fallback for shapes the specialised families
// do not cover and the reference the specialised families are cross-checked against on the GPU.
//
// Reductions are deterministic: every partial sum has a fixed owner and partials are combined
// in a fixed order (FP64), so two runs on the same inputs give the same bits.
#include "nlr_common.cuh"
#include "device_utils.cuh"
#include "fin_logic.cuh"

namespace gemnlr {

// ------------------------------------------------------------------------------------------
// Vector pass (Algorithm 2, call sites 2, 3, 8-11 in one sweep over U): one warp per row.
//   u_i = c_f * w_i ; q_i = u_i . p - 1 ; if gate pending: ytilde_i += gamma q_i ;
//   ybar_i = ytilde_i + gamma q_i ; s += u_i ybar_i ; sum q_i^2 ; sum ytilde_i q_i.
// MATERIALIZE additionally writes u_i back (the scaling call U <- c W).
// Output: part[blockIdx][0..r-1] = s partial, [r] = sum q^2, [r+1] = sum ytilde q.
// ------------------------------------------------------------------------------------------
constexpr int RV_WARPS = 4;

template <bool MATERIALIZE>
__global__ void __launch_bounds__(RV_WARPS * 32)
k_rowvec(float* __restrict__ U, float* __restrict__ ytilde, float* __restrict__ ybar,
         const Ctl* __restrict__ ctl, const float* __restrict__ p, int64_t n, int r, double gamma,
         double* __restrict__ part, int ignore_stop)
{
    if (!ignore_stop && ctl->stopped) return;
    extern __shared__ double sm_s[];              // [RV_WARPS][r]
    __shared__ double sm_red[2][RV_WARPS];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float cf = ctl->c_f;
    const int dual = ctl->dual_pending;
    double* my_s = sm_s + (size_t)warp * r;
    for (int j = lane; j < r; j += 32) my_s[j] = 0.0;
    double qq = 0.0, yq = 0.0;
    const int64_t stride = (int64_t)gridDim.x * RV_WARPS;
    for (int64_t row = (int64_t)blockIdx.x * RV_WARPS + warp; row < n; row += stride) {
        float* urow = U + row * r;
        float acc = 0.f;
        for (int j = lane; j < r; j += 32) {
            float u = cf * urow[j];
            acc = fmaf(u, p[j], acc);
        }
        acc = warp_sum(acc);
        const float q = acc - 1.0f;
        float yt = ytilde[row];
        if (dual) yt = (float)((double)yt + gamma * (double)q);
        const float yb = (float)((double)yt + gamma * (double)q);
        if (lane == 0) {
            if (dual) ytilde[row] = yt;
            ybar[row] = yb;
            qq += (double)q * (double)q;
            yq += (double)yt * (double)q;
        }
        for (int j = lane; j < r; j += 32) {
            float u = cf * urow[j];
            my_s[j] += (double)u * (double)yb;
            if (MATERIALIZE) urow[j] = u;
        }
    }
    if (lane == 0) { sm_red[0][warp] = qq; sm_red[1][warp] = yq; }
    __syncthreads();
    double* out = part + (size_t)blockIdx.x * (r + 2);
    for (int j = threadIdx.x; j < r; j += blockDim.x) {
        double v = 0.0;
        for (int w = 0; w < RV_WARPS; ++w) v += sm_s[(size_t)w * r + j];
        out[j] = v;
    }
    if (threadIdx.x == 0) {
        double a = 0.0, b = 0.0;
        for (int w = 0; w < RV_WARPS; ++w) { a += sm_red[0][w]; b += sm_red[1][w]; }
        out[r] = a;
        out[r + 1] = b;
    }
}

// Vector pass for factors with 32 < r <= 1024, r a multiple of 4: a warp takes 8 / NK rows at a time, a lane
// NK 16-byte pieces of each (NK = 1, 2, 4, 8 for r <= 128, 256, 512, 1024), all requested at once; s is
// accumulated in FP32 over 16 rows and then folded into per-warp FP64 sums.  Same outputs as k_rowvec.
constexpr int RVW_WARPS = 8;
template <bool MATERIALIZE, int NK>
__global__ void __launch_bounds__(RVW_WARPS * 32)
k_rowvec_wide(float* __restrict__ U, float* __restrict__ ytilde, float* __restrict__ ybar,
              const Ctl* __restrict__ ctl, const float* __restrict__ p, int64_t n, int r, double gamma,
              double* __restrict__ part, int ignore_stop)
{
    constexpr int ROWS = 8 / NK;
    if (!ignore_stop && ctl->stopped) return;
    extern __shared__ double sm_s[];              // [RVW_WARPS][r]
    __shared__ double sm_red[2][RVW_WARPS];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float cf = ctl->c_f;
    const int dual = ctl->dual_pending;
    const int r4 = r >> 2;
    double* my_s = sm_s + (size_t)warp * r;
    for (int j = lane; j < r; j += 32) my_s[j] = 0.0;
    float4 p4[NK], sacc[NK];
#pragma unroll
    for (int k = 0; k < NK; ++k) {
        const int c4 = lane + 32 * k;
        p4[k] = (c4 < r4) ? reinterpret_cast<const float4*>(p)[c4] : make_float4(0.f, 0.f, 0.f, 0.f);
        sacc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    auto flush = [&]() {
#pragma unroll
        for (int k = 0; k < NK; ++k) {
            const int c4 = lane + 32 * k;
            if (c4 < r4) {
                double* o = my_s + 4 * c4;
                o[0] += (double)sacc[k].x; o[1] += (double)sacc[k].y; o[2] += (double)sacc[k].z; o[3] += (double)sacc[k].w;
            }
            sacc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
    };
    double qq = 0.0, yq = 0.0;
    int since = 0;
    const int64_t stride = (int64_t)gridDim.x * RVW_WARPS * ROWS;
    for (int64_t row0 = ((int64_t)blockIdx.x * RVW_WARPS + warp) * ROWS; row0 < n; row0 += stride) {
        float4 u[ROWS][NK];
        float yt[ROWS];
#pragma unroll
        for (int i = 0; i < ROWS; ++i) {           // rows beyond n and pieces beyond r read as zero
            const float4* urow = reinterpret_cast<const float4*>(U + (row0 + i) * r);
#pragma unroll
            for (int k = 0; k < NK; ++k) {
                const int c4 = lane + 32 * k;
                u[i][k] = (c4 < r4 && row0 + i < n) ? __ldcs(urow + c4) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            yt[i] = (row0 + i < n) ? ytilde[row0 + i] : 0.f;
        }
#pragma unroll
        for (int i = 0; i < ROWS; ++i) {
            float acc = 0.f;
#pragma unroll
            for (int k = 0; k < NK; ++k) {
                u[i][k].x *= cf; u[i][k].y *= cf; u[i][k].z *= cf; u[i][k].w *= cf;
                acc = fmaf(u[i][k].x, p4[k].x, acc); acc = fmaf(u[i][k].y, p4[k].y, acc);
                acc = fmaf(u[i][k].z, p4[k].z, acc); acc = fmaf(u[i][k].w, p4[k].w, acc);
            }
            acc = warp_sum(acc);
            const float q = acc - 1.0f;
            float y = yt[i];
            if (dual) y = (float)((double)y + gamma * (double)q);
            const float yb = (float)((double)y + gamma * (double)q);
            if (lane == 0 && row0 + i < n) {
                if (dual) ytilde[row0 + i] = y;
                ybar[row0 + i] = yb;
                qq += (double)q * (double)q;
                yq += (double)y * (double)q;
            }
            float4* urow = reinterpret_cast<float4*>(U + (row0 + i) * r);
#pragma unroll
            for (int k = 0; k < NK; ++k) {
                sacc[k].x = fmaf(u[i][k].x, yb, sacc[k].x); sacc[k].y = fmaf(u[i][k].y, yb, sacc[k].y);
                sacc[k].z = fmaf(u[i][k].z, yb, sacc[k].z); sacc[k].w = fmaf(u[i][k].w, yb, sacc[k].w);
                if (MATERIALIZE && lane + 32 * k < r4 && row0 + i < n) urow[lane + 32 * k] = u[i][k];
            }
        }
        since += ROWS;
        if (since >= 16) { flush(); since = 0; }
    }
    flush();
    if (lane == 0) { sm_red[0][warp] = qq; sm_red[1][warp] = yq; }
    __syncthreads();
    double* out = part + (size_t)blockIdx.x * (r + 2);
    for (int j = threadIdx.x; j < r; j += blockDim.x) {
        double v = 0.0;
        for (int w = 0; w < RVW_WARPS; ++w) v += sm_s[(size_t)w * r + j];
        out[j] = v;
    }
    if (threadIdx.x == 0) {
        double a = 0.0, b = 0.0;
        for (int w = 0; w < RVW_WARPS; ++w) { a += sm_red[0][w]; b += sm_red[1][w]; }
        out[r] = a;
        out[r + 1] = b;
    }
}

// Column sums of c_f * U for 32 < r <= 1024, r a multiple of 4: the block sweeps groups of 256 / (r / 4) rows,
// thread t owning the 16-byte piece t % (r / 4) of row t / (r / 4) of each group (so a group is one contiguous
// span and a thread always meets the same four columns), eight groups requested at once, FP64 sums in
// registers.  part[blockIdx][0..r-1].
__global__ void __launch_bounds__(256)
k_colsum_vec(const float* __restrict__ U, const Ctl* __restrict__ ctl, int64_t n, int r, double* __restrict__ part)
{
    __shared__ double sm[1024];                   // [rows of a group][r]
    const int r4 = r >> 2;
    const int per = 256 / r4;                     // rows of a group
    const int t = threadIdx.x;
    const bool active = t < per * r4;
    const int my_row = t / r4;
    const float cf = ctl->c_f;
    double acc[4] = {0.0, 0.0, 0.0, 0.0};
    const float4* U4 = reinterpret_cast<const float4*>(U);
    for (int64_t g0 = (int64_t)blockIdx.x * 8; g0 * per < n; g0 += (int64_t)gridDim.x * 8) {
        float4 w[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int64_t row = (g0 + k) * per + my_row;
            w[k] = (active && row < n) ? __ldcs(U4 + (g0 + k) * per * r4 + t) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            acc[0] += (double)(cf * w[k].x); acc[1] += (double)(cf * w[k].y);
            acc[2] += (double)(cf * w[k].z); acc[3] += (double)(cf * w[k].w);
        }
    }
    if (active) {
#pragma unroll
        for (int c = 0; c < 4; ++c) sm[4 * t + c] = acc[c];      // = sm[my_row][4 (t % r4) + c]
    }
    __syncthreads();
    double* out = part + (size_t)blockIdx.x * (r + 2);
    for (int j = t; j < r; j += 256) {
        double v = 0.0;
        for (int i = 0; i < per; ++i) v += sm[i * r + j];
        out[j] = v;
    }
}

// Column sums of c_f * U (p = U^T 1 for a freshly loaded factor): part[blockIdx][0..r-1].
__global__ void __launch_bounds__(RV_WARPS * 32)
k_colsum(const float* __restrict__ U, const Ctl* __restrict__ ctl, int64_t n, int r,
         double* __restrict__ part)
{
    extern __shared__ double sm_s[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float cf = ctl->c_f;
    double* my_s = sm_s + (size_t)warp * r;
    for (int j = lane; j < r; j += 32) my_s[j] = 0.0;
    const int64_t stride = (int64_t)gridDim.x * RV_WARPS;
    for (int64_t row = (int64_t)blockIdx.x * RV_WARPS + warp; row < n; row += stride) {
        const float* urow = U + row * r;
        for (int j = lane; j < r; j += 32) my_s[j] += (double)(cf * urow[j]);
    }
    __syncthreads();
    double* out = part + (size_t)blockIdx.x * (r + 2);
    for (int j = threadIdx.x; j < r; j += blockDim.x) {
        double v = 0.0;
        for (int w = 0; w < RV_WARPS; ++w) v += sm_s[(size_t)w * r + j];
        out[j] = v;
    }
}

__global__ void k_fin_colsum(const double* __restrict__ part, int g, int r, float* __restrict__ p)
{
    for (int j = threadIdx.x; j < r; j += blockDim.x) {
        double v = 0.0;
        for (int b = 0; b < g; ++b) v += part[(size_t)b * (r + 2) + j];
        p[j] = (float)v;
    }
}

// ------------------------------------------------------------------------------------------
// First product, Theta = X-hat^T U, as split-K partials: CTA (gx, tile) accumulates the
// G_DT x G_RT tile of Theta over its contiguous row chunk.  Per row tile the sums run in FP32
// registers and are then folded into FP64 running sums, so the FP32 chains stay G_TM long.
// part[gx][j * r + k] (FP64).
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
k_pass1_generic(const float* __restrict__ X, const float* __restrict__ U,
                const Ctl* __restrict__ ctl, int64_t n, int d, int r, int tiles_r,
                double* __restrict__ part, int ignore_stop)
{
    if (!ignore_stop && ctl->stopped) return;
    __shared__ __align__(16) float Xs[G_TM][G_DT];
    __shared__ __align__(16) float Us[G_TM][G_RT];
    const float cf = ctl->c_f;
    const int tile = blockIdx.y;
    const int j0 = (tile / tiles_r) * G_DT, k0 = (tile % tiles_r) * G_RT;
    const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
    const int64_t rows_per = (n + gridDim.x - 1) / gridDim.x;
    const int64_t r_lo = (int64_t)blockIdx.x * rows_per;
    const int64_t r_hi = (r_lo + rows_per < n) ? r_lo + rows_per : n;
    double acc64[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc64[a][b] = 0.0;
    for (int64_t m0 = r_lo; m0 < r_hi; m0 += G_TM) {
        for (int idx = threadIdx.x; idx < G_TM * G_DT; idx += 256) {
            int m = idx / G_DT, jj = idx % G_DT;
            int64_t row = m0 + m;
            int col = j0 + jj;
            Xs[m][jj] = (row < r_hi && col < d) ? X[row * d + col] : 0.f;
        }
        for (int idx = threadIdx.x; idx < G_TM * G_RT; idx += 256) {
            int m = idx / G_RT, kk = idx % G_RT;
            int64_t row = m0 + m;
            int col = k0 + kk;
            Us[m][kk] = (row < r_hi && col < r) ? cf * U[row * r + col] : 0.f;
        }
        __syncthreads();
        float acc[4][4];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
#pragma unroll 8
        for (int m = 0; m < G_TM; ++m) {
            const float4 xv = *reinterpret_cast<const float4*>(&Xs[m][ty * 4]);
            const float4 uv = *reinterpret_cast<const float4*>(&Us[m][tx * 4]);
            const float xa[4] = {xv.x, xv.y, xv.z, xv.w};
            const float ua[4] = {uv.x, uv.y, uv.z, uv.w};
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(xa[a], ua[b], acc[a][b]);
        }
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) acc64[a][b] += (double)acc[a][b];
        __syncthreads();
    }
    double* out = part + (size_t)blockIdx.x * ((size_t)d * r);
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        int j = j0 + ty * 4 + a;
        if (j >= d) continue;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            int k = k0 + tx * 4 + b;
            if (k < r) out[(size_t)j * r + k] = acc64[a][b];
        }
    }
}

// Theta[e] = FP32(scale * sum_g part[g][e]) in ascending g (four interleaved slices combined in order);
// red[blockIdx] = this block's share of ||Theta||_F^2 (from the unrounded sums).  scale is the pending
// multiplier c_f when the partials were formed from the unscaled factor (scale_cf), else 1.
__global__ void __launch_bounds__(256)
k_red1(const double* __restrict__ part, int g, int64_t dr, const Ctl* __restrict__ ctl,
       float* __restrict__ theta, double* __restrict__ red, int ignore_stop, int scale_cf)
{
    if (!ignore_stop && ctl->stopped) return;
    const double scale = scale_cf ? (double)ctl->c_f : 1.0;
    __shared__ double sl[4][64];
    __shared__ double sred[32];
    const int e_local = threadIdx.x & 63, slice = threadIdx.x >> 6;
    const int64_t e = (int64_t)blockIdx.x * 64 + e_local;
    double v = 0.0;
    if (e < dr)
        for (int b = slice; b < g; b += 4) v += part[(size_t)b * dr + e];
    sl[slice][e_local] = v;
    __syncthreads();
    double t2 = 0.0;
    if (slice == 0 && e < dr) {
        const double tot = scale * (((sl[0][e_local] + sl[1][e_local]) + sl[2][e_local]) + sl[3][e_local]);
        theta[e] = (float)tot;
        t2 = tot * tot;
    }
    t2 = block_sum<256>(t2, sred);
    if (threadIdx.x == 0) red[blockIdx.x] = t2;
}

// Scalars after the vector pass (and the Theta reduction): s, alpha*s, sum q^2, sum ytilde q,
// ||Theta||^2; finishes the previous iteration (rho, stop test, history record).
// mode 0: start of an iteration, 1: tail (also resets the multiplier after the U buffer was
// rescaled), 2: objective evaluation only.
__global__ void __launch_bounds__(1024)
k_fin1(Ctl* __restrict__ ctl, const double* __restrict__ part1v, int gv, const double* __restrict__ red,
       int nred, int r, int64_t n, float alpha, double gamma, double eps_c, int T_min,
       float* __restrict__ s, float* __restrict__ alpha_s, gem_nlr_iter_info* __restrict__ hist, int mode)
{
    if (mode == 0 && ctl->stopped) return;
    __shared__ double sred[32];
    for (int j = threadIdx.x; j < r; j += blockDim.x) {
        double v = 0.0;
        int b = 0;
        for (; b + 8 <= gv; b += 8) {             // eight records requested at once, added in record order
            double t[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) t[k] = __ldcg(part1v + (size_t)(b + k) * (r + 2) + j);
#pragma unroll
            for (int k = 0; k < 8; ++k) v += t[k];
        }
        for (; b < gv; ++b) v += __ldcg(part1v + (size_t)b * (r + 2) + j);
        float sf = (float)v;
        s[j] = sf;
        alpha_s[j] = alpha * sf;
    }
    double qq = 0.0, yq = 0.0, t2 = 0.0;
    for (int b = threadIdx.x; b < gv; b += blockDim.x) {
        qq += part1v[(size_t)b * (r + 2) + r];
        yq += part1v[(size_t)b * (r + 2) + r + 1];
    }
    if (mode != 1)
        for (int b = threadIdx.x; b < nred; b += blockDim.x) t2 += red[b];
    qq = block_sum<1024>(qq, sred);
    yq = block_sum<1024>(yq, sred);
    t2 = block_sum<1024>(t2, sred);
    if (threadIdx.x == 0) fin1_scalars(ctl, qq, yq, t2, n, gamma, eps_c, T_min, hist, mode);
}

// ------------------------------------------------------------------------------------------
// Second product with the fused epilogue (Eq. "entrywise-fusion"): for a G2_TM x G2_RT output
// tile, acc = (X-hat Theta)_ij, u = c_f * U_ij,
//   w = max{ u + 2 alpha acc - alpha ybar_i p_j - alpha s_j, 0 },  U_ij <- w,
// with FP64 sums of w^2, u^2, w u and of the columns of w.  CTAs walk row tiles with a grid
// stride; part[(gx * tiles_r + ty)][0..2] = a, b, h partials, [3..3+G2_RT) = column sums.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
k_pass2_generic(const float* __restrict__ X, const float* __restrict__ theta, float* __restrict__ U,
                const float* __restrict__ ybar, const float* __restrict__ p,
                const float* __restrict__ alpha_s, const Ctl* __restrict__ ctl, int64_t n, int d,
                int r, float alpha, double* __restrict__ part)
{
    if (ctl->stopped) return;
    __shared__ __align__(16) float Xs[G2_TM][G2_DT + 1];
    __shared__ __align__(16) float Ts[G2_DT][G2_RT];
    __shared__ double sred[32];
    __shared__ double scol[16][G2_RT];
    const float cf = ctl->c_f;
    const float two_alpha = 2.0f * alpha;
    const int k0 = blockIdx.y * G2_RT;
    const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
    const int64_t n_tiles = (n + G2_TM - 1) / G2_TM;
    double sa = 0.0, sb = 0.0, sh = 0.0;
    double csum[4] = {0.0, 0.0, 0.0, 0.0};
    float pk[4], ask[4];
#pragma unroll
    for (int b = 0; b < 4; ++b) {
        int k = k0 + tx * 4 + b;
        pk[b] = (k < r) ? p[k] : 0.f;
        ask[b] = (k < r) ? alpha_s[k] : 0.f;
    }
    for (int64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const int64_t m0 = tile * G2_TM;
        float acc[4][4];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
        for (int j0 = 0; j0 < d; j0 += G2_DT) {
            for (int idx = threadIdx.x; idx < G2_TM * G2_DT; idx += 256) {
                int m = idx / G2_DT, jj = idx % G2_DT;
                int64_t row = m0 + m;
                int col = j0 + jj;
                Xs[m][jj] = (row < n && col < d) ? X[row * d + col] : 0.f;
            }
            for (int idx = threadIdx.x; idx < G2_DT * G2_RT; idx += 256) {
                int jj = idx / G2_RT, kk = idx % G2_RT;
                int j = j0 + jj, k = k0 + kk;
                Ts[jj][kk] = (j < d && k < r) ? theta[(size_t)j * r + k] : 0.f;
            }
            __syncthreads();
#pragma unroll 8
            for (int jj = 0; jj < G2_DT; ++jj) {
                const float4 tv = *reinterpret_cast<const float4*>(&Ts[jj][tx * 4]);
                const float ta[4] = {tv.x, tv.y, tv.z, tv.w};
#pragma unroll
                for (int a = 0; a < 4; ++a) {
                    const float x = Xs[ty * 4 + a][jj];
#pragma unroll
                    for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(x, ta[b], acc[a][b]);
                }
            }
            __syncthreads();
        }
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            const int64_t row = m0 + ty * 4 + a;
            if (row >= n) continue;
            const float nay = -alpha * ybar[row];
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int k = k0 + tx * 4 + b;
                if (k >= r) continue;
                const float u = cf * U[row * r + k];
                float v = fmaf(two_alpha, acc[a][b], u);
                v = fmaf(nay, pk[b], v);
                v -= ask[b];
                const float w = fmaxf(v, 0.f);
                const double wd = (double)w, ud = (double)u;
                sa = fma(wd, wd, sa);
                sb = fma(ud, ud, sb);
                sh = fma(wd, ud, sh);
                csum[b] += wd;
                U[row * r + k] = w;
            }
        }
    }
    sa = block_sum<256>(sa, sred);
    sb = block_sum<256>(sb, sred);
    sh = block_sum<256>(sh, sred);
#pragma unroll
    for (int b = 0; b < 4; ++b) scol[ty][tx * 4 + b] = csum[b];
    __syncthreads();
    double* out = part + ((size_t)blockIdx.x * gridDim.y + blockIdx.y) * (3 + G2_RT);
    if (threadIdx.x == 0) { out[0] = sa; out[1] = sb; out[2] = sh; }
    if (threadIdx.x < G2_RT) {
        double v = 0.0;
        for (int y = 0; y < 16; ++y) v += scol[y][threadIdx.x];
        out[3 + threadIdx.x] = v;
    }
}

// Scalars after the second product (Algorithm 2, steps (d)-(e)): a, b, h, the multiplier,
// the movement estimate, the dual gate, and p = U^T 1 of the new iterate as c * (column sums
// of W).  nparts = gx * gy records of stride (3 + cols_per); column j lives in record
// (gx, j / cols_per) at 3 + j % cols_per.
__global__ void __launch_bounds__(256)
k_fin2(Ctl* __restrict__ ctl, const double* __restrict__ part, int gx, int gy, int cols_per, int r,
       int K, double eps_d, float* __restrict__ p)
{
    if (ctl->stopped) return;
    __shared__ double sred[32];
    __shared__ double sc;
    __shared__ int sbad;
    const int stride = 3 + cols_per;
    const int nparts = gx * gy;
    double a = 0.0, b = 0.0, h = 0.0;
    for (int i = threadIdx.x; i < nparts; i += blockDim.x) {
        a += part[(size_t)i * stride + 0];
        b += part[(size_t)i * stride + 1];
        h += part[(size_t)i * stride + 2];
    }
    a = block_sum<256>(a, sred);
    b = block_sum<256>(b, sred);
    h = block_sum<256>(h, sred);
    if (threadIdx.x == 0) {
        double c;
        sbad = fin2_scalars(ctl, a, b, h, K, eps_d, &c) ? 0 : 1;
        sc = c;
    }
    __syncthreads();
    if (sbad) return;
    const double c = sc;
    for (int j = threadIdx.x; j < r; j += blockDim.x) {
        const int yy = j / cols_per, jj = j % cols_per;
        double v = 0.0;
        for (int x = 0; x < gx; ++x) v += part[((size_t)x * gy + yy) * stride + 3 + jj];
        p[j] = (float)(c * v);
    }
}

// Row-argmax read-out: smallest index among maxima of c_f * U_i (c_f > 0 does not change it).
__global__ void k_labels(const float* __restrict__ U, int64_t n, int r, int32_t* __restrict__ labels)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    if (r <= 32) {
        // one thread per row
        for (int64_t row = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; row < n;
             row += (int64_t)gridDim.x * blockDim.x) {
            const float* u = U + row * r;
            float bv = u[0];
            int best = 0;
            for (int j = 1; j < r; ++j) {
                float v = u[j];
                if (v > bv) { bv = v; best = j; }
            }
            labels[row] = best;
        }
        return;
    }
    for (int64_t row = warp; row < n; row += nwarps) {
        const float* u = U + row * r;
        float bv = -INFINITY;
        int best = 0x7fffffff;
        for (int j = lane; j < r; j += 32) {
            float v = u[j];
            if (v > bv) { bv = v; best = j; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            int ob = __shfl_xor_sync(0xffffffffu, best, o);
            if (ov > bv || (ov == bv && ob < best)) { bv = ov; best = ob; }
        }
        if (lane == 0) labels[row] = best;
    }
}

// Row-argmax read-out with 16-byte loads (r a multiple of 4).  Narrow factors (r <= 32): a thread takes two rows
// at a time, all their pieces requested before the first comparison.  Wider ones (r <= 1024): a warp takes
// 8 / NK rows at a time, a lane NK pieces of each (as in k_rowvec_wide); elements are visited in increasing
// column order inside a lane and the lanes are combined on (value, index), so ties go to the smallest index.
__global__ void __launch_bounds__(256)
k_labels_small4(const float* __restrict__ U, int64_t n, int r4, int32_t* __restrict__ labels)
{
    const float4* U4 = reinterpret_cast<const float4*>(U);
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t row = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; row < n; row += 2 * stride) {
        const int64_t row1 = row + stride;
        float4 a[8], b[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            a[c] = (c < r4) ? __ldcs(U4 + row * r4 + c) : make_float4(0.f, 0.f, 0.f, 0.f);
            b[c] = (c < r4 && row1 < n) ? __ldcs(U4 + row1 * r4 + c) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        float bva = a[0].x, bvb = b[0].x;
        int ba = 0, bb = 0;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            if (c < r4) {
                const float va[4] = {a[c].x, a[c].y, a[c].z, a[c].w}, vb[4] = {b[c].x, b[c].y, b[c].z, b[c].w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (va[e] > bva) { bva = va[e]; ba = 4 * c + e; }
                    if (vb[e] > bvb) { bvb = vb[e]; bb = 4 * c + e; }
                }
            }
        }
        labels[row] = ba;
        if (row1 < n) labels[row1] = bb;
    }
}

template <int NK>
__global__ void __launch_bounds__(256)
k_labels_wide(const float* __restrict__ U, int64_t n, int r, int32_t* __restrict__ labels)
{
    constexpr int ROWS = 8 / NK;
    const int lane = threadIdx.x & 31, r4 = r >> 2;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t row0 = warp * ROWS; row0 < n; row0 += nwarps * ROWS) {
        float4 u[ROWS][NK];
#pragma unroll
        for (int i = 0; i < ROWS; ++i)
#pragma unroll
            for (int k = 0; k < NK; ++k) {
                const int c4 = lane + 32 * k;
                u[i][k] = (c4 < r4 && row0 + i < n) ? __ldcs(reinterpret_cast<const float4*>(U + (row0 + i) * r) + c4)
                                                     : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        float bv[ROWS];
        int best[ROWS];
#pragma unroll
        for (int i = 0; i < ROWS; ++i) {
            bv[i] = -INFINITY;
            best[i] = 0x7fffffff;
#pragma unroll
            for (int k = 0; k < NK; ++k) {
                const int c4 = lane + 32 * k;
                if (c4 < r4) {
                    const float v[4] = {u[i][k].x, u[i][k].y, u[i][k].z, u[i][k].w};
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if (v[e] > bv[i]) { bv[i] = v[e]; best[i] = 4 * c4 + e; }
                }
            }
        }
        auto merge = [](float& v, int& b, float ov, int ob) {
            if (ov > v || (ov == v && ob < b)) { v = ov; b = ob; }
        };
        if constexpr (ROWS == 8) {
            // the eight rows' candidates by recursive halving: after the exchanges over lane bits 4, 3, 2 a lane
            // holds the candidate of row 4 (bit 4) + 2 (bit 3) + (bit 2) over its 4-lane group's share
#pragma unroll
            for (int lvl = 0; lvl < 3; ++lvl) {
                const int o = 16 >> lvl, m = 4 >> lvl;                 // lane bit, candidates kept
                const bool up = lane & o;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (i < m) {
                        const float sv = up ? bv[i] : bv[i + m];
                        const int sb = up ? best[i] : best[i + m];
                        float kv = up ? bv[i + m] : bv[i];
                        int kb = up ? best[i + m] : best[i];
                        merge(kv, kb, __shfl_xor_sync(0xffffffffu, sv, o), __shfl_xor_sync(0xffffffffu, sb, o));
                        bv[i] = kv; best[i] = kb;
                    }
                }
            }
#pragma unroll
            for (int o = 2; o > 0; o >>= 1)
                merge(bv[0], best[0], __shfl_xor_sync(0xffffffffu, bv[0], o), __shfl_xor_sync(0xffffffffu, best[0], o));
            const int row_l = ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1);
            if ((lane & 3) == 0 && row0 + row_l < n) labels[row0 + row_l] = best[0];
        } else {
#pragma unroll
            for (int i = 0; i < ROWS; ++i) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1)
                    merge(bv[i], best[i], __shfl_xor_sync(0xffffffffu, bv[i], o), __shfl_xor_sync(0xffffffffu, best[i], o));
                if (lane == 0 && row0 + i < n) labels[row0 + i] = best[i];
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// Thread-per-row variants of the vector pass and of the column sums for narrow factors
// (r = 4 R4 <= 32): a thread reads its whole row with 16-byte loads (consecutive threads read
// consecutive rows, so a warp still covers one contiguous span) and keeps the row's share of s in
// registers.  Same outputs as k_rowvec / k_colsum.
// ------------------------------------------------------------------------------------------
template <int R4, bool MATERIALIZE>
__global__ void __launch_bounds__(256)
k_rowvec_small(float* __restrict__ U, float* __restrict__ ytilde, float* __restrict__ ybar,
               const Ctl* __restrict__ ctl, const float* __restrict__ p, int64_t n, double gamma,
               double* __restrict__ part, int ignore_stop)
{
    constexpr int R = 4 * R4;
    if (!ignore_stop && ctl->stopped) return;
    __shared__ float ssum[8][R];
    __shared__ double sred[32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float cf = ctl->c_f;
    const int dual = ctl->dual_pending;
    float pr[R], sacc[R];
#pragma unroll
    for (int j = 0; j < R; ++j) { pr[j] = p[j]; sacc[j] = 0.f; }
    double qq = 0.0, yq = 0.0;
    for (int64_t row = (int64_t)blockIdx.x * 256 + threadIdx.x; row < n; row += (int64_t)gridDim.x * 256) {
        float4* up = reinterpret_cast<float4*>(U + row * R);
        float u[R];
#pragma unroll
        for (int c = 0; c < R4; ++c) {
            const float4 w = up[c];
            u[4 * c] = cf * w.x; u[4 * c + 1] = cf * w.y; u[4 * c + 2] = cf * w.z; u[4 * c + 3] = cf * w.w;
        }
        float dot = 0.f;
#pragma unroll
        for (int j = 0; j < R; ++j) dot = fmaf(u[j], pr[j], dot);
        const float q = dot - 1.0f;
        float yt = ytilde[row];
        if (dual) { yt = (float)((double)yt + gamma * (double)q); ytilde[row] = yt; }
        const float yb = (float)((double)yt + gamma * (double)q);
        ybar[row] = yb;
        qq = fma((double)q, (double)q, qq);
        yq = fma((double)yt, (double)q, yq);
#pragma unroll
        for (int j = 0; j < R; ++j) sacc[j] = fmaf(u[j], yb, sacc[j]);
        if (MATERIALIZE) {
#pragma unroll
            for (int c = 0; c < R4; ++c) up[c] = make_float4(u[4 * c], u[4 * c + 1], u[4 * c + 2], u[4 * c + 3]);
        }
    }
    // block partial of s: lanes by butterfly, warps in warp order
#pragma unroll
    for (int j = 0; j < R; ++j) {
        const float v = warp_sum(sacc[j]);
        if (lane == 0) ssum[warp][j] = v;
    }
    qq = block_sum<256>(qq, sred);
    yq = block_sum<256>(yq, sred);
    double* out = part + (size_t)blockIdx.x * (R + 2);
    if (threadIdx.x < R) {
        double v = 0.0;
#pragma unroll
        for (int w = 0; w < 8; ++w) v += (double)ssum[w][threadIdx.x];
        out[threadIdx.x] = v;
    }
    if (threadIdx.x == 0) { out[R] = qq; out[R + 1] = yq; }
}

template <int R4>
__global__ void __launch_bounds__(256)
k_colsum_small(const float* __restrict__ U, const Ctl* __restrict__ ctl, int64_t n, double* __restrict__ part)
{
    constexpr int R = 4 * R4;
    __shared__ double ssum[8][R];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float cf = ctl->c_f;
    double acc[R];
#pragma unroll
    for (int j = 0; j < R; ++j) acc[j] = 0.0;
    for (int64_t row0 = (int64_t)blockIdx.x * 256 + threadIdx.x; row0 < n; row0 += (int64_t)gridDim.x * 256 * 8) {
        // eight rows per thread in FP32, then folded into the FP64 running sums
        float part32[R];
#pragma unroll
        for (int j = 0; j < R; ++j) part32[j] = 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int64_t row = row0 + (int64_t)k * gridDim.x * 256;
            if (row < n) {
                const float4* up = reinterpret_cast<const float4*>(U + row * R);
#pragma unroll
                for (int c = 0; c < R4; ++c) {
                    const float4 w = up[c];
                    part32[4 * c] += cf * w.x; part32[4 * c + 1] += cf * w.y;
                    part32[4 * c + 2] += cf * w.z; part32[4 * c + 3] += cf * w.w;
                }
            }
        }
#pragma unroll
        for (int j = 0; j < R; ++j) acc[j] += (double)part32[j];
    }
#pragma unroll
    for (int j = 0; j < R; ++j) {
        const double v = warp_sum(acc[j]);
        if (lane == 0) ssum[warp][j] = v;
    }
    __syncthreads();
    double* out = part + (size_t)blockIdx.x * (R + 2);
    if (threadIdx.x < R) {
        double v = 0.0;
#pragma unroll
        for (int w = 0; w < 8; ++w) v += ssum[w][threadIdx.x];
        out[threadIdx.x] = v;
    }
}

// ------------------------------------------------------------------------------------------
// Host-side launchers
// ------------------------------------------------------------------------------------------
static size_t rv_smem(int r) { return (size_t)RV_WARPS * r * sizeof(double); }

static void set_rv_attr(int r)
{
    static int done_r = -1;
    if (rv_smem(r) > 48 * 1024 && done_r < r) {
        cudaFuncSetAttribute(k_rowvec<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)rv_smem(r));
        cudaFuncSetAttribute(k_rowvec<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)rv_smem(r));
        cudaFuncSetAttribute(k_colsum, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)rv_smem(r));
        done_r = r;
    }
}

static bool small_r(int r) { return r % 4 == 0 && r >= 4 && r <= 32; }
static int small_grid(const Problem& pb)
{
    int64_t g = (pb.P.n + 255) / 256;
    if (g > pb.L.gv) g = pb.L.gv;
    return (int)(g < 1 ? 1 : g);
}

static bool wide_r(int r) { return r > 32 && r <= 1024 && r % 4 == 0; }
static int wide_nk(int r) { return r <= 128 ? 1 : r <= 256 ? 2 : r <= 512 ? 4 : 8; }
static int wide_grid(const Problem& pb)
{
    const int rows_per = RVW_WARPS * (8 / wide_nk(pb.P.r));
    int64_t g = (pb.P.n + rows_per - 1) / rows_per;
    const int cap = pb.L.gv < kSMs * 2 ? pb.L.gv : kSMs * 2;
    if (g > cap) g = cap;
    return (int)(g < 1 ? 1 : g);
}

template <bool MAT, int NK>
static void launch_rowvec_wide(const Problem& pb, int grid, int ignore_stop)
{
    const auto& P = pb.P;
    const size_t sm = sizeof(double) * RVW_WARPS * (size_t)P.r;
    static bool attr_set = false;
    if (!attr_set) {
        cudaFuncSetAttribute(k_rowvec_wide<MAT, NK>, cudaFuncAttributeMaxDynamicSharedMemorySize, 8 * 1024 * 8);
        attr_set = true;
    }
    k_rowvec_wide<MAT, NK><<<grid, RVW_WARPS * 32, sm, pb.stream>>>(
        pb.U, pb.ytilde(), pb.ybar(), pb.ctl(), pb.p(), P.n, P.r, pb.gamma, pb.part1v(), ignore_stop);
}

template <bool MAT>
static void launch_rowvec_small(const Problem& pb, int grid, int ignore_stop)
{
    const auto& P = pb.P;
#define RV_CASE(R4) case R4: k_rowvec_small<R4, MAT><<<grid, 256, 0, pb.stream>>>(pb.U, pb.ytilde(), pb.ybar(), pb.ctl(), pb.p(), P.n, pb.gamma, pb.part1v(), ignore_stop); break;
    switch (P.r / 4) { RV_CASE(1) RV_CASE(2) RV_CASE(3) RV_CASE(4) RV_CASE(5) RV_CASE(6) RV_CASE(7) RV_CASE(8) default: break; }
#undef RV_CASE
}

// Vector pass (optionally applying the pending multiplier to the U buffer); returns the number of
// per-block partial records it wrote.
static int launch_rowvec(const Problem& pb, bool materialize, int ignore_stop)
{
    const auto& P = pb.P;
    if (small_r(P.r)) {
        const int grid = small_grid(pb);
        if (materialize) launch_rowvec_small<true>(pb, grid, ignore_stop);
        else launch_rowvec_small<false>(pb, grid, ignore_stop);
        pb.count();
        return grid;
    }
    if (wide_r(P.r)) {
        const int grid = wide_grid(pb);
        const int nk = wide_nk(P.r);
#define RVW_CASE(NK) case NK: if (materialize) launch_rowvec_wide<true, NK>(pb, grid, ignore_stop); else launch_rowvec_wide<false, NK>(pb, grid, ignore_stop); break;
        switch (nk) { RVW_CASE(1) RVW_CASE(2) RVW_CASE(4) RVW_CASE(8) default: break; }
#undef RVW_CASE
        pb.count();
        return grid;
    }
    set_rv_attr(P.r);
    if (materialize)
        k_rowvec<true><<<pb.L.gv, RV_WARPS * 32, rv_smem(P.r), pb.stream>>>(
            pb.U, pb.ytilde(), pb.ybar(), pb.ctl(), pb.p(), P.n, P.r, pb.gamma, pb.part1v(), ignore_stop);
    else
        k_rowvec<false><<<pb.L.gv, RV_WARPS * 32, rv_smem(P.r), pb.stream>>>(
            pb.U, pb.ytilde(), pb.ybar(), pb.ctl(), pb.p(), P.n, P.r, pb.gamma, pb.part1v(), ignore_stop);
    pb.count();
    return pb.L.gv;
}

static void launch_fin1_g(const Problem& pb, int mode, int gv);

void launch_init_colsum(const Problem& pb)
{
    const auto& P = pb.P;
    int grid = pb.L.gv;
    if (small_r(P.r)) {
        grid = small_grid(pb);
#define CS_CASE(R4) case R4: k_colsum_small<R4><<<grid, 256, 0, pb.stream>>>(pb.U, pb.ctl(), P.n, pb.part1v()); break;
        switch (P.r / 4) { CS_CASE(1) CS_CASE(2) CS_CASE(3) CS_CASE(4) CS_CASE(5) CS_CASE(6) CS_CASE(7) CS_CASE(8) default: break; }
#undef CS_CASE
    } else if (wide_r(P.r)) {
        grid = pb.L.gv < kSMs * 4 ? pb.L.gv : kSMs * 4;
        k_colsum_vec<<<grid, 256, 0, pb.stream>>>(pb.U, pb.ctl(), P.n, P.r, pb.part1v());
    } else {
        set_rv_attr(P.r);
        k_colsum<<<grid, RV_WARPS * 32, rv_smem(P.r), pb.stream>>>(pb.U, pb.ctl(), P.n, P.r, pb.part1v());
    }
    k_fin_colsum<<<1, 256, 0, pb.stream>>>(pb.part1v(), grid, P.r, pb.p());
    pb.count(2);
}

void launch_vector_pass(const Problem& pb)
{
    launch_rowvec(pb, false, 0);
}

static void launch_fin1_g(const Problem& pb, int mode, int gv)
{
    const auto& P = pb.P;
    k_fin1<<<1, 1024, 0, pb.stream>>>(pb.ctl(), pb.part1v(), gv, pb.red1(), pb.L.nred1, P.r, P.n,
                                     P.alpha, pb.gamma, P.eps_c, P.T_min, pb.s(), pb.alpha_s(),
                                     pb.hist(), mode);
    pb.count();
}

void launch_fin1(const Problem& pb, int mode)
{
    launch_fin1_g(pb, mode, small_r(pb.P.r) ? small_grid(pb) : wide_r(pb.P.r) ? wide_grid(pb) : pb.L.gv);
}

void launch_fin2(const Problem& pb, int gx, int gy, int cols_per)
{
    const auto& P = pb.P;
    k_fin2<<<1, 256, 0, pb.stream>>>(pb.ctl(), pb.part2(), gx, gy, cols_per, P.r, P.K, P.eps_d, pb.p());
    pb.count();
}

void launch_generic_pass1(const Problem& pb, int ignore_stop)
{
    const auto& P = pb.P;
    const auto& L = pb.L;
    dim3 g1(L.g1x, L.g1y_d * L.g1y_r);
    k_pass1_generic<<<g1, 256, 0, pb.stream>>>(pb.X, pb.U, pb.ctl(), P.n, P.d, P.r, L.g1y_r, pb.part1(),
                                               ignore_stop);
    k_red1<<<L.nred1, 256, 0, pb.stream>>>(pb.part1(), L.g1x, (int64_t)P.d * P.r, pb.ctl(), pb.theta(),
                                            pb.red1(), ignore_stop, 0);
    pb.count(2);
}

void launch_red1(const Problem& pb, int g, int ignore_stop, int scale_cf)
{
    k_red1<<<pb.L.nred1, 256, 0, pb.stream>>>(pb.part1(), g, (int64_t)pb.P.d * pb.P.r, pb.ctl(), pb.theta(),
                                             pb.red1(), ignore_stop, scale_cf);
    pb.count(1);
}

void launch_generic_pass2_alpha(const Problem& pb, float alpha)
{
    const auto& P = pb.P;
    const auto& L = pb.L;
    dim3 g2(L.g2x, L.g2y);
    k_pass2_generic<<<g2, 256, 0, pb.stream>>>(pb.X, pb.theta(), pb.U, pb.ybar(), pb.p(), pb.alpha_s(),
                                               pb.ctl(), P.n, P.d, P.r, alpha, pb.part2());
    pb.count();
}

void launch_generic_pass2_kernel(const Problem& pb)
{
    launch_generic_pass2_alpha(pb, pb.P.alpha);
}

void launch_pass1_partials(const Problem& pb, const float* A, const float* B, int da, int rb, int tiles_b, dim3 grid)
{
    k_pass1_generic<<<grid, 256, 0, pb.stream>>>(A, B, pb.ctl(), pb.P.n, da, rb, tiles_b, pb.part1(), 1);
    pb.count();
}


void launch_tail(const Problem& pb)
{
    const int g = launch_rowvec(pb, true, 1);
    launch_fin1_g(pb, 1, g);
}

void launch_objective(const Problem& pb)
{
    // Called after the tail: no gate is pending and the multiplier is 1, so the vector pass has
    // no side effect on the dual.  The objective is also wanted after a stop, so the stop flag
    // is ignored.
    const int g = launch_rowvec(pb, false, 1);
    launch_generic_pass1(pb, 1);
    launch_fin1_g(pb, 2, g);
}

void launch_labels(const Problem& pb, int32_t* labels)
{
    const auto& P = pb.P;
    if (P.r % 4 == 0 && P.r <= 32) {
        int64_t blocks = (P.n + 511) / 512;
        if (blocks > kSMs * 8) blocks = kSMs * 8;
        k_labels_small4<<<(int)(blocks < 1 ? 1 : blocks), 256, 0, pb.stream>>>(pb.U, P.n, P.r / 4, labels);
        pb.count();
        return;
    }
    if (wide_r(P.r)) {
        const int nk = wide_nk(P.r);
        int64_t blocks = (P.n + 8 * (8 / nk) - 1) / (8 * (8 / nk));
        if (blocks > kSMs * 8) blocks = kSMs * 8;
        const int g = (int)(blocks < 1 ? 1 : blocks);
        switch (nk) {
        case 1: k_labels_wide<1><<<g, 256, 0, pb.stream>>>(pb.U, P.n, P.r, labels); break;
        case 2: k_labels_wide<2><<<g, 256, 0, pb.stream>>>(pb.U, P.n, P.r, labels); break;
        case 4: k_labels_wide<4><<<g, 256, 0, pb.stream>>>(pb.U, P.n, P.r, labels); break;
        default: k_labels_wide<8><<<g, 256, 0, pb.stream>>>(pb.U, P.n, P.r, labels); break;
        }
        pb.count();
        return;
    }
    int blocks = (int)((P.n + 255) / 256);
    if (P.r > 32) blocks = (int)((P.n + 7) / 8);
    if (blocks > kSMs * 16) blocks = kSMs * 16;
    if (blocks < 1) blocks = 1;
    k_labels<<<blocks, 256, 0, pb.stream>>>(pb.U, P.n, P.r, labels);
    pb.count();
}

}  // namespace gemnlr
