// FP32-FFMA family for skinny shapes (d a multiple of 32 up to 128, r in {8, 16}): both products
// are HBM-bound there and plain ALUs suffice, so the work is organised around streaming X-hat
// exactly twice per iteration.
//
//  * Persistent CTAs (one per SM), 8 consumer warps + 1 producer warp.  The producer streams row
//    tiles of X-hat through a ring of shared-memory stages with TMA tile loads (128-byte swizzle)
//    and, in the first product, the matching contiguous tile of U with a bulk copy; mbarriers
//    signal full / empty stages.  Every wait is bounded.
//  * First product (k_pass1_ffma): a warp owns a block of rows of the tile.  It first does the
//    row-local vector work of the iteration on those rows (u = c_f w, q = u.p - 1, gated dual
//    step, ybar, s += u ybar, sum q^2, sum ytilde q -- call sites 2, 3, 8-11 of Algorithm 2) and
//    writes u back into the stage, then accumulates its share of Theta = X-hat^T U in registers.
//    CTA partials (FP64) are reduced by k_red1_fused, whose last block also runs the scalars.
//  * Second product (k_pass2_ffma): thread tile of 2 rows x 4 columns against Theta held in
//    shared memory, epilogue of Eq. "entrywise-fusion" with FP64 statistics, in-place store of W;
//    the last CTA to finish reduces the partials in CTA order and runs the scalar step.
#include "nlr_common.cuh"
#include "device_utils.cuh"
#include "fin_logic.cuh"
#include "pipeline.cuh"
#include "ffma_family.cuh"
#include <cudaTypedefs.h>

namespace gemnlr {

bool make_tensor_map_2d(CUtensorMap* out, const float* base, int64_t rows, int cols, int box_rows,
                        int box_cols, bool atom32, int swizzle_bytes)
{
    static PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
    if (!encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres) !=
                cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn)
            return false;
        encode = (PFN_cuTensorMapEncodeTiled_v12000)fn;
    }
    cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t gstride[1] = {(cuuint64_t)cols * sizeof(float)};
    cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult rc = encode(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, (void*)base, gdim, gstride, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE,
                         swizzle_bytes == 1 ? CU_TENSOR_MAP_SWIZZLE_NONE
                         : (swizzle_bytes == 64 && box_cols * sizeof(float) == 64) ? CU_TENSOR_MAP_SWIZZLE_64B
                         : box_cols * sizeof(float) != 128 ? CU_TENSOR_MAP_SWIZZLE_NONE
                             : (atom32 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B),
                         CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS;
}

// 2D tensor map over a row-major fp16 matrix (rows x cols halves, row pitch pitch_halves), box of
// box_rows x box_cols; box_cols * 2 bytes must be 64 (64-byte swizzle) or 128 (128-byte swizzle).
bool make_tensor_map_2d_f16(CUtensorMap* out, const void* base, int64_t rows, int64_t cols, int64_t pitch_halves,
                            int box_rows, int box_cols)
{
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !fn)
        return false;
    auto encode = (PFN_cuTensorMapEncodeTiled_v12000)fn;
    cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t gstride[1] = {(cuuint64_t)pitch_halves * 2};
    cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    const CUtensorMapSwizzle sw = box_cols * 2 == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                : box_cols * 2 == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE;
    CUresult rc = encode(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS;
}

namespace ffma {

constexpr int NCW = 8;                    // consumer warps
constexpr int NTHREADS = (NCW + 1) * 32;  // + producer warp

// Byte offset of 16-byte chunk c (4 floats: columns 4c .. 4c+3) of tile row rl inside an X-hat
// stage: the stage holds D/32 boxes of TM rows x 128 bytes, each written with the 128-byte
// swizzle (chunk index XOR row mod 8).
template <int TM>
__device__ __forceinline__ uint32_t x_chunk_off(int rl, int c)
{
    return (uint32_t)((c >> 3) * (TM * 128) + rl * 128 + (((c & 7) ^ (rl & 7)) << 4));
}

// ------------------------------------------------------------------------------------------------
template <int D, int R, int TM, int NST>
__global__ void __launch_bounds__(NTHREADS, 1)
k_pass1_ffma(const __grid_constant__ CUtensorMap tmX, const float* __restrict__ U,
             float* __restrict__ ytilde, float* __restrict__ ybar, Ctl* __restrict__ ctl,
             const float* __restrict__ p, int64_t n, double gamma, double* __restrict__ part)
{
    constexpr int RW = TM / NCW;            // rows of a tile owned by one warp
    constexpr int LPR = 32 / RW;            // lanes per row in the vector phase
    constexpr int CPL = R / LPR;            // columns per lane in the vector phase
    constexpr int TK = R < 8 ? R : 8;       // Theta columns per lane
    constexpr int LK = R / TK;
    constexpr int NCHUNK = D / 4;
    constexpr int LJ = (NCHUNK < 32 / LK) ? NCHUNK : 32 / LK;
    constexpr int NCH = NCHUNK / LJ;        // 16-byte chunks of a row per lane
    constexpr int RC = 32 / (LJ * LK);      // rows processed per step by one warp
    constexpr int XB = TM * D * 4, UB = TM * R * 4, STAGE = XB + UB;
    static_assert(RW >= 1 && LPR >= 1 && LPR * RW == 32 && CPL % 4 == 0 && CPL * LPR == R, "vector phase mapping");
    static_assert(LJ * NCH == NCHUNK && RC >= 1 && RW % RC == 0 && TK % 4 == 0, "theta phase mapping");
    static_assert(XB % 1024 == 0 && UB % 1024 == 0 && D % 32 == 0, "stage alignment");
    static_assert(NCW * D * R * 4 <= NST * STAGE, "reduction scratch fits in the stage ring");

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

    float acc[NCH * 4][TK];
    float s_acc[CPL];
    double qq = 0.0, yq = 0.0;
#pragma unroll
    for (int a = 0; a < NCH * 4; ++a)
#pragma unroll
        for (int k = 0; k < TK; ++k) acc[a][k] = 0.f;
#pragma unroll
    for (int c = 0; c < CPL; ++c) s_acc[c] = 0.f;

    if (warp == NCW) {
        // ---------------- producer ----------------
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
        // ---------------- consumers ----------------
        const int v_row = lane / LPR, v_sub = lane % LPR;       // vector phase: row in the warp's block, column group
        const int lj = lane % LJ, lk = (lane / LJ) % LK, rc = lane / (LJ * LK);
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
            // ytilde of this lane's row, fetched before the wait so that its latency overlaps
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

            // ---- vector phase on the warp's own rows ----
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

            // ---- Theta phase: RC rows per step, lane tile (4 NCH) x TK ----
#pragma unroll 2
            for (int step = 0; step < RW / RC; ++step) {
                const int rl = warp * RW + step * RC + rc;
                float4 xv[NCH];
#pragma unroll
                for (int i = 0; i < NCH; ++i) xv[i] = lds128(xs + x_chunk_off<TM>(rl, lj + i * LJ));
                float uv[TK];
#pragma unroll
                for (int k4 = 0; k4 < TK / 4; ++k4) {
                    float4 w = lds128(us + (uint32_t)(rl * R + lk * TK + 4 * k4) * 4);
                    uv[4 * k4] = w.x; uv[4 * k4 + 1] = w.y; uv[4 * k4 + 2] = w.z; uv[4 * k4 + 3] = w.w;
                }
#pragma unroll
                for (int i = 0; i < NCH; ++i) {
                    const float xa[4] = {xv[i].x, xv[i].y, xv[i].z, xv[i].w};
#pragma unroll
                    for (int a = 0; a < 4; ++a)
#pragma unroll
                        for (int k = 0; k < TK; ++k) acc[i * 4 + a][k] = fmaf(xa[a], uv[k], acc[i * 4 + a][k]);
                }
            }
            // the stage was written through the generic proxy (u); order that before the next TMA fill
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_bar(s));
        }
    }
    __syncthreads();      // every load has landed and been consumed: the ring becomes scratch

    // ---- CTA partials: Theta (sum over row classes and warps), s, sum q^2, sum ytilde q ----
    float* red = reinterpret_cast<float*>(smem);       // [NCW][D * R]
    if (warp < NCW) {
        const int lj = lane % LJ, lk = (lane / LJ) % LK, rc = lane / (LJ * LK);
#pragma unroll
        for (int a = 0; a < NCH * 4; ++a)
#pragma unroll
            for (int k = 0; k < TK; ++k) {
                float v = acc[a][k];
#pragma unroll
                for (int o = LJ * LK; o < 32; o <<= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                if (rc == 0) {
                    const int j = 4 * (lj + (a >> 2) * LJ) + (a & 3);
                    red[(size_t)warp * (D * R) + j * R + lk * TK + k] = v;
                }
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

// Sums the g per-CTA records [d*r Theta | r s | sum q^2 | sum ytilde q] (FP64) entry by entry: a block
// takes 16 entries x 16 interleaved slices of the records (independent loads, combined in slice
// order, so the result does not depend on scheduling).  Theta is stored as FP32 with the block's
// share of ||Theta||_F^2; the r + 2 trailing sums go to a small FP64 array.  The last block to
// finish turns those into s, alpha s and the scalar step that finishes the previous iteration.
constexpr int RED1_EB = 16;
__global__ void __launch_bounds__(256)
k_red1_fused(const double* __restrict__ part, int g, int stride, int dr, int r, Ctl* __restrict__ ctl,
             float* __restrict__ theta, double* __restrict__ red, float* __restrict__ s,
             float* __restrict__ alpha_s, int64_t n, float alpha, double gamma, double eps_c, int T_min,
             gem_nlr_iter_info* __restrict__ hist, int mode, int ignore_stop, int combined)
{
    grid_dep_launch();
    grid_dep_wait();                        // the partial records of the first-product kernel before this one
    if (!ignore_stop && ctl->stopped) return;
    __shared__ double sl[16][RED1_EB];
    __shared__ double sred[32];
    __shared__ int is_last;
    double* extra = red + gridDim.x;           // [r + 2] behind the per-block ||Theta||^2 shares
    const int e_local = threadIdx.x & (RED1_EB - 1), slice = threadIdx.x >> 4;
    const int e = blockIdx.x * RED1_EB + e_local;
    double v = 0.0;
    if (e < stride) {
        const double* src = part + e;
#pragma unroll 4
        for (int b = slice; b < g; b += 16) v += __ldcg(src + (size_t)b * stride);
    }
    sl[slice][e_local] = v;
    __syncthreads();
    double t2 = 0.0;
    if (slice == 0 && e < stride) {
        double tot = sl[0][e_local];
#pragma unroll
        for (int k = 1; k < 16; ++k) tot += sl[k][e_local];
        if (e < dr) {
            if (mode != 1) theta[e] = (float)tot;          // the tail keeps Theta: its records carry no fresh product
            t2 = tot * tot;
        } else {
            extra[e - dr] = tot;
        }
    }
    t2 = block_sum<256>(t2, sred);
    if (threadIdx.x == 0) {
        red[blockIdx.x] = t2;
        __threadfence();
        const unsigned prev = atomicAdd(&ctl->counter[0], 1u);
        is_last = (prev == gridDim.x - 1) ? 1 : 0;
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    for (int j = threadIdx.x; j < r; j += blockDim.x) {
        const float sf = (float)__ldcg(extra + j);
        s[j] = sf;
        alpha_s[j] = alpha * sf;
    }
    double tt = 0.0;
    for (int b = threadIdx.x; b < (int)gridDim.x; b += blockDim.x) tt += __ldcg(red + b);
    tt = block_sum<256>(tt, sred);
    if (threadIdx.x == 0) {
        ctl->counter[0] = 0;
        fin1_scalars(ctl, __ldcg(extra + r), __ldcg(extra + r + 1), tt, n, gamma, eps_c, T_min, hist, mode, combined != 0);
    }
}

// ------------------------------------------------------------------------------------------------
template <int D, int R, int TM, int NST>
__global__ void __launch_bounds__(NTHREADS, 1)
k_pass2_ffma(const __grid_constant__ CUtensorMap tmX, const float* __restrict__ theta,
             float* __restrict__ U, const float* __restrict__ ybar, const float* __restrict__ p,
             const float* __restrict__ alpha_s, Ctl* __restrict__ ctl, int64_t n, float alpha, int K,
             double eps_d, double* __restrict__ part, float* __restrict__ p_out)
{
    constexpr int CG = R / 4;                 // column groups of 4
    constexpr int XB = TM * D * 4;
    constexpr int PS = 4 + R;                 // partial record: a, b, h, pad, column sums
    static_assert(TM * CG == 2 * NCW * 32, "2 rows x 4 columns per consumer thread");
    static_assert(XB % 1024 == 0 && D % 32 == 0 && R % 4 == 0, "stage alignment");
    static_assert(NCW * 32 * 4 * 8 <= NST * XB, "column-sum scratch fits in the stage ring");

    if (ctl->stopped) return;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t bars[2 * NST];
    __shared__ uint32_t abort_flag;
    __shared__ double sred[32];
    __shared__ int is_last;
    __shared__ double sc;
    __shared__ int sok;
    float* theta_s = reinterpret_cast<float*>(smem + (size_t)NST * XB);   // [D][R]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t th_base = smem_u32(theta_s);
    const uint32_t bar_base = smem_u32(bars);
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (NST + s); };
    if (threadIdx.x == 0) {
        for (int s = 0; s < NST; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), NCW); }
        abort_flag = 0;
        fence_barrier_init();
    }
    for (int e = threadIdx.x; e < D * R; e += NTHREADS) theta_s[e] = theta[e];
    __syncthreads();

    const int64_t n_tiles = (n + TM - 1) / TM;
    const float cf = ctl->c_f;
    const float two_alpha = 2.0f * alpha;
    double sa = 0.0, sb = 0.0, sh = 0.0;
    double csum[4] = {0.0, 0.0, 0.0, 0.0};

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
        const int rp = threadIdx.x / CG, cg = threadIdx.x % CG;
        const int r0 = 2 * rp;
        float pk[4], ask[4];
#pragma unroll
        for (int b = 0; b < 4; ++b) { pk[b] = p[4 * cg + b]; ask[b] = alpha_s[4 * cg + b]; }
        int it = 0;
        for (int64_t t = blockIdx.x; t < n_tiles; t += gridDim.x, ++it) {
            const int s = it % NST;
            const uint32_t xs = smem_base + (uint32_t)s * XB;
            const int64_t row0 = t * TM + r0;
            const bool v0 = row0 < n, v1 = row0 + 1 < n;
            float4* up0 = reinterpret_cast<float4*>(U + row0 * R + 4 * cg);
            float4* up1 = reinterpret_cast<float4*>(U + (row0 + 1) * R + 4 * cg);
            // old factor entries and ybar: issued before the wait so the loads overlap the FMA loop
            const float4 w0 = v0 ? __ldcs(up0) : make_float4(0.f, 0.f, 0.f, 0.f);
            const float4 w1 = v1 ? __ldcs(up1) : make_float4(0.f, 0.f, 0.f, 0.f);
            const float yb0 = v0 ? ybar[row0] : 0.f;
            const float yb1 = v1 ? ybar[row0 + 1] : 0.f;
            mbar_wait(full_bar(s), (it / NST) & 1, &abort_flag, ctl);
            const bool dead = abort_flag != 0;          // a wait ran out: the tile's data cannot be trusted, U is left as it is
            float acc[2][4];
#pragma unroll
            for (int b = 0; b < 4; ++b) { acc[0][b] = 0.f; acc[1][b] = 0.f; }
#pragma unroll 4
            for (int c = 0; c < D / 4; ++c) {
                const float4 x0 = lds128(xs + x_chunk_off<TM>(r0, c));
                const float4 x1 = lds128(xs + x_chunk_off<TM>(r0 + 1, c));
                const float xa0[4] = {x0.x, x0.y, x0.z, x0.w};
                const float xa1[4] = {x1.x, x1.y, x1.z, x1.w};
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    const float4 th = lds128(th_base + (uint32_t)((4 * c + jj) * R + 4 * cg) * 4);
                    acc[0][0] = fmaf(xa0[jj], th.x, acc[0][0]);
                    acc[0][1] = fmaf(xa0[jj], th.y, acc[0][1]);
                    acc[0][2] = fmaf(xa0[jj], th.z, acc[0][2]);
                    acc[0][3] = fmaf(xa0[jj], th.w, acc[0][3]);
                    acc[1][0] = fmaf(xa1[jj], th.x, acc[1][0]);
                    acc[1][1] = fmaf(xa1[jj], th.y, acc[1][1]);
                    acc[1][2] = fmaf(xa1[jj], th.z, acc[1][2]);
                    acc[1][3] = fmaf(xa1[jj], th.w, acc[1][3]);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_bar(s));

            // ---- epilogue: w = max{u + 2 alpha acc - alpha ybar_i p_j - alpha s_j, 0} ----
            const float wold[2][4] = {{w0.x, w0.y, w0.z, w0.w}, {w1.x, w1.y, w1.z, w1.w}};
            const float nay[2] = {-alpha * yb0, -alpha * yb1};
            float wn[2][4];
#pragma unroll
            for (int a = 0; a < 2; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    const float u = cf * wold[a][b];
                    float v = fmaf(two_alpha, acc[a][b], u);
                    v = fmaf(nay[a], pk[b], v);
                    v -= ask[b];
                    const float w = ((a == 0) ? v0 : v1) ? fmaxf(v, 0.f) : 0.f;
                    const double wd = (double)w, ud = (double)u;
                    sa = fma(wd, wd, sa);
                    sb = fma(ud, ud, sb);
                    sh = fma(wd, ud, sh);
                    csum[b] += wd;
                    wn[a][b] = w;
                }
            if (v0 && !dead) *up0 = make_float4(wn[0][0], wn[0][1], wn[0][2], wn[0][3]);
            if (v1 && !dead) *up1 = make_float4(wn[1][0], wn[1][1], wn[1][2], wn[1][3]);
        }
    }
    __syncthreads();

    // ---- CTA partial: a, b, h and the column sums of W ----
    sa = block_sum<NTHREADS>(sa, sred);
    sb = block_sum<NTHREADS>(sb, sred);
    sh = block_sum<NTHREADS>(sh, sred);
    double* scol = reinterpret_cast<double*>(smem);     // [NCW * 32][4]
    if (warp < NCW) {
#pragma unroll
        for (int b = 0; b < 4; ++b) scol[(size_t)threadIdx.x * 4 + b] = csum[b];
    }
    __syncthreads();
    double* out = part + (size_t)blockIdx.x * PS;
    if (threadIdx.x == 0) { out[0] = sa; out[1] = sb; out[2] = sh; out[3] = 0.0; }
    if (threadIdx.x < R) {
        const int cg = threadIdx.x / 4, b = threadIdx.x % 4;
        double v = 0.0;
        for (int rp = 0; rp < NCW * 32 / CG; ++rp) v += scol[(size_t)(rp * CG + cg) * 4 + b];
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

    // ---- last CTA: global sums in CTA order, scalar step, p = c * column sums ----
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
// Host side: shape table and launchers
// ------------------------------------------------------------------------------------------------
template <int D, int R, int TM1, int NST1, int TM2, int NST2>
struct Shape {
    static constexpr size_t smem1 = (size_t)NST1 * (TM1 * D * 4 + TM1 * R * 4) + 1024;
    static constexpr size_t smem2 = (size_t)NST2 * (TM2 * D * 4) + (size_t)D * R * 4 + 1024;
    static bool plan(const Problem& pb, FfmaPlan* pl)
    {
        if (!make_tensor_map_2d(&pl->tm1, pb.X, pb.P.n, D, TM1, 32)) return false;
        if (!make_tensor_map_2d(&pl->tm2, pb.X, pb.P.n, D, TM2, 32)) return false;
        const int64_t t1 = (pb.P.n + TM1 - 1) / TM1, t2 = (pb.P.n + TM2 - 1) / TM2;
        pl->g1 = (int)(t1 < kSMs ? t1 : kSMs);
        pl->g2 = (int)(t2 < kSMs ? t2 : kSMs);
        if (cudaFuncSetAttribute(k_pass1_ffma<D, R, TM1, NST1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem1) != cudaSuccess) return false;
        if (cudaFuncSetAttribute(k_pass2_ffma<D, R, TM2, NST2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem2) != cudaSuccess) return false;
        return true;
    }
    static void pass1(const Problem& pb, const FfmaPlan& pl)
    {
        k_pass1_ffma<D, R, TM1, NST1><<<pl.g1, NTHREADS, smem1, pb.stream>>>(
            pl.tm1, pb.U, pb.ytilde(), pb.ybar(), pb.ctl(), pb.p(), pb.P.n, pb.gamma, pb.part1());
    }
    static void pass2(const Problem& pb, const FfmaPlan& pl)
    {
        k_pass2_ffma<D, R, TM2, NST2><<<pl.g2, NTHREADS, smem2, pb.stream>>>(
            pl.tm2, pb.theta(), pb.U, pb.ybar(), pb.p(), pb.alpha_s(), pb.ctl(), pb.P.n, pb.P.alpha, pb.P.K,
            pb.P.eps_d, pb.part2(), pb.p());
    }
};

//                  D    R   TM1 NST1 TM2 NST2
using S_32_8   = Shape<32,  8,  256, 4, 256, 5>;
using S_32_16  = Shape<32,  16, 256, 4, 128, 6>;
using S_64_8   = Shape<64,  8,  128, 5, 256, 3>;
using S_64_16  = Shape<64,  16, 128, 4, 128, 5>;
using S_128_16 = Shape<128, 16, 64,  5, 128, 3>;

#define FFMA_DISPATCH(id, CALL)                 \
    switch (id) {                               \
        case 0: S_32_8::CALL; break;            \
        case 1: S_32_16::CALL; break;           \
        case 2: S_64_8::CALL; break;            \
        case 3: S_64_16::CALL; break;           \
        case 4: S_128_16::CALL; break;          \
        default: break;                         \
    }

}  // namespace ffma

bool ffma_plan(const Problem& pb, FfmaPlan* pl)
{
    const int d = pb.P.d, r = pb.P.r;
    int id = -1;
    if (d == 32 && r == 8) id = 0;
    else if (d == 32 && r == 16) id = 1;
    else if (d == 64 && r == 8) id = 2;
    else if (d == 64 && r == 16) id = 3;
    else if (d == 128 && r == 16) id = 4;
    if (id < 0 || pb.P.n < 1024 || pb.P.n > 2000000000ll) return false;
    pl->shape_id = id;
    bool ok = false;
    using namespace ffma;
    switch (id) {
        case 0: ok = S_32_8::plan(pb, pl); break;
        case 1: ok = S_32_16::plan(pb, pl); break;
        case 2: ok = S_64_8::plan(pb, pl); break;
        case 3: ok = S_64_16::plan(pb, pl); break;
        case 4: ok = S_128_16::plan(pb, pl); break;
    }
    return ok;
}

void red1_fused_launch(const Problem& pb, int g, int mode)
{
    const int dr = pb.P.d * pb.P.r;
    launch_pdl(ffma::k_red1_fused, dim3((dr + pb.P.r + 2 + ffma::RED1_EB - 1) / ffma::RED1_EB), dim3(256), 0, pb.stream,
               (const double*)pb.part1(), g, dr + pb.P.r + 2, dr, pb.P.r, pb.ctl(), pb.theta(), pb.red1(), pb.s(), pb.alpha_s(),
               pb.P.n, pb.P.alpha, pb.gamma, pb.P.eps_c, pb.P.T_min, pb.hist(), mode, 0, 0);
    pb.count(1);
}

void red1_combine_launch(const Problem& pb, const double* records, int world, int64_t n_global, int mode)
{
    const int dr = pb.P.d * pb.P.r;
    ffma::k_red1_fused<<<(dr + pb.P.r + 2 + ffma::RED1_EB - 1) / ffma::RED1_EB, 256, 0, pb.stream>>>(
        records, world, dr + pb.P.r + 2, dr, pb.P.r, pb.ctl(), pb.theta(), pb.red1(), pb.s(), pb.alpha_s(),
        n_global, pb.P.alpha, pb.gamma, pb.P.eps_c, pb.P.T_min, pb.hist(), mode, mode != 0, 1);
    pb.count(1);
}

void ffma_launch_first(const Problem& pb, const FfmaPlan& pl, int mode)
{
    using namespace ffma;
    FFMA_DISPATCH(pl.shape_id, pass1(pb, pl));
    pb.count(1);
    red1_fused_launch(pb, pl.g1, mode);
}

void ffma_launch_second(const Problem& pb, const FfmaPlan& pl)
{
    using namespace ffma;
    FFMA_DISPATCH(pl.shape_id, pass2(pb, pl));
    pb.count(1);
}

}  // namespace gemnlr
