// Tiled tensor-core kernels (tcgen05 + TMEM) for wide problems (d and r too large for the resident-Theta
// kernels: the embedding-sized shape d = 768, r = 1000).  Second product:
//   acc = X-hat Theta ;  W = [U + 2 alpha acc - alpha (ybar p^T + 1 s^T)]_+ in place ;  FP64 a, b, h ;
//   column sums of W                                               (Eq. "entrywise-fusion", Algorithm 2 call 4)
//
// FP32 accuracy from FP16 tensor cores: x 2^k = h1 + h2 with h1 = fp16(x 2^k), h2 = fp16(x 2^k - h1)
// (22 significant bits), product accumulated in FP32 as h1 h1' + h2 h1' + h1 h2' (three K = 16 MMAs).
// The scales are powers of two that cannot overflow: |x-hat_ij| <= ||X-hat||_2 = 1 (2^15) and
// |Theta_jk| <= ||X-hat||_2 ||U||_F = sqrt(K).  X-hat is static, so its images are built once at setup
// (k_ximg_build: row-major for this kernel, transposed for the first product) and arrive by TMA already
// in the K-major 64-byte-swizzle layout; nothing is split inside this kernel.
//
// Work item = (128-row tile, 256-column block).  The K loop streams d in chunks of 32 features: a
// stage holds the two X-hat image boxes (128 rows x 64 bytes) and the matching boxes of the Theta^T
// images (256 columns x 64 bytes, pre-swizzled in global memory, one bulk copy each).  With M = 128,
// N = 256 an MMA runs at the tensor pipe's full rate, and the accumulator (256 TMEM columns) is
// double-buffered, so the epilogue of one item overlaps the MMAs of the next.
//
// A CTA keeps one column block for the whole launch (CTA b: block b mod NCB, row tiles b / NCB, + lanes, ...;
// the grid is a multiple of NCB), so only that block's p, alpha s and running column sums live in shared memory
// and its Theta^T boxes stay hot in L2.
//
//   warp 0       producer (TMA / bulk copies, 3-stage ring; a fourth stage buys nothing)
//   warp 1       MMA issuer: per chunk 2 k-steps x 3 products; commits free the stage
//   warps 2-9    epilogue: warp = (TMEM lane quarter, column half); accumulators read in the 16x256b
//                fragment layout and swapped between neighbouring lanes so that a thread owns 4 consecutive
//                columns; the old entries of U are read from, and the new ones written into, the group's
//                panel in shared memory; statistics in FP32 over a thread's 16 entries of a group, then FP64;
//                column sums by warp shuffles, combined across the four quarters in fixed order
//   warp 10      U panel manager: panels of 128 rows x 32 columns (128-byte rows, 128-byte swizzle) by TMA into a
//                ring of four slots, one panel ahead per column half, and back to U by TMA from the same slot
// What sets the pace: everything that touches an SM's shared-memory array (TMA fills, the MMAs' operand fetches,
// the panels) shares about 128 bytes per clock; an item moves 24 x 120 KB of operands and 512 KB of panels, i.e.
// 26 thousand cycles against 18.6 thousand of tensor time, and that is the measured item period at d = 768.
// An earlier epilogue read and wrote U straight from global memory; its speed depended on the L1 capacity the
// shared-memory carve-out left (a 217 KB footprint was 8-12 % slower than a 157 KB one) and it set the pace at
// every d; through the panels the d = 256 shapes gain 9 % and d = 768 is unchanged.
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
constexpr int KC = 32;                        // features per chunk (64-byte fp16 rows)
constexpr int A_BOX = TILE_M * KC * 2;        // 8 KB
constexpr int B_BOX = NBLK * KC * 2;          // 16 KB
constexpr int STAGE = 2 * A_BOX + 2 * B_BOX;  // 48 KB: X-hat h1, h2, Theta^T h1, h2
constexpr int NS = 3;                        // see the note on the shared-memory carve-out below
constexpr int NEPI = 8;                       // epilogue warps
constexpr int NTHREADS = (3 + NEPI) * 32;     // + producer, MMA issuer, U panel manager
constexpr size_t SMEM_RING = (size_t)NS * STAGE;
constexpr int NPAN = 4;                       // U panel slots
constexpr int PAN_BYTES = TILE_M * 32 * 4;    // panel = 128 rows x 32 columns FP32 (128-byte rows, 128-byte swizzle): 16 KB
constexpr int W_PANEL = 2 + NEPI;             // warp index of the panel manager

// Theta (d x r, FP32 row-major) -> fp16 images h1, h2 of Theta^T 2^eT as K-major 64-byte-swizzled boxes:
// box (kb, cb) = features 32 kb .. 32 kb + 31 of columns 256 cb .. 256 cb + 255 (zero beyond r).
__global__ void k_theta_images64(const float* __restrict__ theta, int d, int r, int NCB, int eT, const Ctl* __restrict__ ctl,
                                 __half* __restrict__ img_h1, __half* __restrict__ img_h2)
{
    if (ctl->stopped) return;
    const float sT = ldexpf(1.0f, eT);
    const int64_t total = (int64_t)d * NCB * NBLK;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int j = (int)(e / (NCB * NBLK)), k = (int)(e % (NCB * NBLK));     // feature, column
        const float v = (k < r) ? theta[(size_t)j * r + k] * sT : 0.f;
        const __half h1 = __float2half_rn(v);
        const __half h2 = __float2half_rn(v - __half2float(h1));
        const int kb = j >> 5, jj = j & 31, c = jj >> 3, w = jj & 7;
        const int cb = k >> 8, kr = k & 255;
        const size_t off = ((size_t)(kb * NCB + cb) * NBLK + kr) * KC + (size_t)(((c ^ ((kr >> 1) & 3)) << 3) + w);
        img_h1[off] = h1;
        img_h2[off] = h2;
    }
}

// X-hat (n rows of dx features, FP32) -> its fp16 split images x 2^15 = h1 + h2 over d >= dx features (zero beyond
// dx): row-major (n x d), and transposed in the
// exact shared-memory form the first product consumes: for every stage of 32 data rows and block of fb
// features one contiguous box [feature][32 rows] with the 64-byte swizzle already applied (zero
// beyond n and d), so that a box arrives with one bulk copy.  One block per 32 x 32 tile; the
// transposition goes through shared memory.
__global__ void __launch_bounds__(256)
k_ximg_build(const float* __restrict__ X, int64_t n, int dx, int d, int64_t n_pad, int fb, __half* __restrict__ h1,
             __half* __restrict__ h2, __half* __restrict__ h1T, __half* __restrict__ h2T)
{
    __shared__ __half t1[32][33], t2[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;            // 32 x 8
    const int64_t row0 = (int64_t)blockIdx.x * 32;
    const int f0 = blockIdx.y * 32;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t row = row0 + ty + 8 * i;
        const int f = f0 + tx;
        const float v = (row < n && f < dx) ? X[row * dx + f] * 32768.0f : 0.f;      // features dx .. d - 1: zero padding
        const __half a = __float2half_rn(v);
        const __half b = __float2half_rn(v - __half2float(a));
        if (row < n && f < d) { h1[row * d + f] = a; h2[row * d + f] = b; }
        t1[ty + 8 * i][tx] = a;
        t2[ty + 8 * i][tx] = b;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int f = f0 + ty + 8 * i;
        const int64_t row = row0 + tx;
        if (row < n_pad) {                                 // features beyond d of the last block stay zero (memset)
            const int nnb = (d + fb - 1) / fb, nbk = f / fb, m = f - nbk * fb, kk = tx;     // kk = row inside the stage
            const size_t off = (((size_t)blockIdx.x * nnb + nbk) * fb + m) * 32 + (size_t)((((kk >> 3) ^ ((m >> 1) & 3)) << 3) + (kk & 7));
            if (f < d) { h1T[off] = t1[tx][ty + 8 * i]; h2T[off] = t2[tx][ty + 8 * i]; }
        }
    }
}

// The same images when X-hat itself may be given up (x_inplace == 2, d a multiple of 32): the row-major pair is
// written over X-hat, row by row (row i: d halves of h1 followed by d halves of h2 in the 4 d bytes of its FP32
// row, so each image has a row pitch of 2 d halves).  A block owns whole stages of 32 rows: it reads all of their
// FP32 entries into shared memory before it writes any of their bytes.
__global__ void __launch_bounds__(256)
k_ximg_build_inplace(float* X, int64_t n, int d, int64_t n_pad, int fb, __half* __restrict__ h1T, __half* __restrict__ h2T)
{
    extern __shared__ float xs[];                          // [32][d + 1]
    const int pitch = d + 1;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    __half* X16 = reinterpret_cast<__half*>(X);
    const int64_t n_stages = n_pad / 32;
    const int nnb = (d + fb - 1) / fb;
    for (int64_t st = blockIdx.x; st < n_stages; st += gridDim.x) {
        const int64_t row0 = st * 32;
        for (int idx = threadIdx.x; idx < 32 * d; idx += 256) {
            const int rr = idx / d, f = idx - rr * d;
            xs[rr * pitch + f] = (row0 + rr < n) ? X[(row0 + rr) * d + f] * 32768.0f : 0.f;
        }
        __syncthreads();
        for (int idx = threadIdx.x; idx < 32 * d; idx += 256) {
            const int rr = idx / d, f = idx - rr * d;
            if (row0 + rr < n) {
                const float v = xs[rr * pitch + f];
                const __half a = __float2half_rn(v);
                const __half b = __float2half_rn(v - __half2float(a));
                X16[(row0 + rr) * 2 * d + f] = a;
                X16[(row0 + rr) * 2 * d + d + f] = b;
            }
        }
        for (int f0 = 0; f0 < d; f0 += 32) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int f = f0 + ty + 8 * i;
                const float v = xs[tx * pitch + f];        // row tx of the stage, feature f
                const __half a = __float2half_rn(v);
                const __half b = __float2half_rn(v - __half2float(a));
                const int nbk = f / fb, m = f - nbk * fb, kk = tx;
                const size_t off = (((size_t)st * nnb + nbk) * fb + m) * 32 + (size_t)((((kk >> 3) ^ ((m >> 1) & 3)) << 3) + (kk & 7));
                h1T[off] = a;
                h2T[off] = b;
            }
        }
        __syncthreads();
    }
}

__global__ void __launch_bounds__(NTHREADS, 1)
k_pass2_tcg(const __grid_constant__ CUtensorMap tmX1, const __grid_constant__ CUtensorMap tmX2,
            const __grid_constant__ CUtensorMap tmU, const __half* __restrict__ img_h1, const __half* __restrict__ img_h2, float* __restrict__ U,
            const float* __restrict__ ybar, const float* __restrict__ p, const float* __restrict__ alpha_s,
            Ctl* __restrict__ ctl, int64_t n, int d, int r, int NCB, int eT, float alpha, int K, double eps_d,
            double* __restrict__ part, float* __restrict__ p_out)
{
    if (ctl->stopped) return;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t bars[2 * NS + 4 + 2 * NPAN];
    __shared__ uint32_t abort_flag;
    __shared__ uint32_t tmem_base_s;
    __shared__ double sred[32];
    __shared__ int is_last;
    __shared__ double sc;
    __shared__ int sok;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int KB = d / KC;
    const int cb = (int)(blockIdx.x % NCB);                              // this CTA's column block
    const int lane_id = (int)(blockIdx.x / NCB), lanes = (int)(gridDim.x / NCB);
    const int col0 = cb * NBLK;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t stage0 = smem_base;
    const uint32_t pan0 = stage0 + (uint32_t)SMEM_RING;                 // NPAN panel slots
    unsigned char* tail = smem + SMEM_RING + (size_t)NPAN * PAN_BYTES;
    float* sp = reinterpret_cast<float*>(tail);                         // [NBLK] p of the block
    float* sas = sp + NBLK;                                             // [NBLK] alpha s
    double* scol = reinterpret_cast<double*>(sas + NBLK);               // [NBLK] running column sums of W
    float* stmp = reinterpret_cast<float*>(scol + NBLK);                // [2][4][NBLK] per-quarter column sums of an item

    const uint32_t bar0 = smem_u32(bars);
    auto xfull = [&](int s) { return bar0 + 8u * s; };
    auto xfree = [&](int s) { return bar0 + 8u * (NS + s); };
    auto accfull = [&](int a) { return bar0 + 8u * (2 * NS + a); };
    auto accfree = [&](int a) { return bar0 + 8u * (2 * NS + 2 + a); };
    auto pfull = [&](int s) { return bar0 + 8u * (2 * NS + 4 + s); };            // panel landed
    auto pdone = [&](int s) { return bar0 + 8u * (2 * NS + 4 + NPAN + s); };     // its four warps have written W into it

    if (threadIdx.x == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(xfull(s), 1); mbar_init(xfree(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(accfull(a), 1); mbar_init(accfree(a), NEPI); }
        for (int s = 0; s < NPAN; ++s) { mbar_init(pfull(s), 1); mbar_init(pdone(s), 4); }
        abort_flag = 0;
        fence_barrier_init();
    }
    for (int j = threadIdx.x; j < NBLK; j += NTHREADS) {
        sp[j] = (col0 + j < r) ? p[col0 + j] : 0.f;
        sas[j] = (col0 + j < r) ? alpha_s[col0 + j] : 0.f;
        scol[j] = 0.0;
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_s), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;

    const int64_t n_tiles = (n + TILE_M - 1) / TILE_M;
    const float cf = ctl->c_f;
    // the accumulator holds (x-hat 2^15) (Theta 2^eT) sums: fold the scales into the 2 alpha factor
    const float two_alpha = 2.0f * alpha * ldexpf(1.0f, -15 - eT);
    double sa = 0.0, sb = 0.0, sh = 0.0;

    if (warp == 0) {
        // ------------------------------ producer ------------------------------
        if (lane == 0) {
            int64_t g = 0;
            for (int64_t t = lane_id; t < n_tiles && !abort_flag; t += lanes) {
                const int row0 = (int)(t * TILE_M);
                for (int kb = 0; kb < KB; ++kb, ++g) {
                    const int s = (int)(g % NS);
                    if (g >= NS) mbar_wait_backoff(xfree(s), (uint32_t)((g / NS) - 1) & 1, &abort_flag, ctl);
                    const uint32_t dst = stage0 + (uint32_t)s * STAGE;
                    const size_t boff = ((size_t)(kb * NCB + cb) * NBLK) * KC;
                    mbar_expect_tx(xfull(s), STAGE);
                    tma_load_2d(dst, &tmX1, kb * KC, row0, xfull(s));
                    tma_load_2d(dst + A_BOX, &tmX2, kb * KC, row0, xfull(s));
                    bulk_load_1d(dst + 2 * A_BOX, img_h1 + boff, B_BOX, xfull(s));
                    bulk_load_1d(dst + 2 * A_BOX + B_BOX, img_h2 + boff, B_BOX, xfull(s));
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        // Inside an item the wait for the next chunk is placed between the two k-steps of the current chunk,
        // so the tensor pipe has work queued while this thread polls.
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_f16(TILE_M, NBLK, 0, 0);
            const uint64_t da1_0 = umma_desc_k_sw64(stage0), da2_0 = umma_desc_k_sw64(stage0 + A_BOX);
            const uint64_t db1_0 = umma_desc_k_sw64(stage0 + 2 * A_BOX), db2_0 = umma_desc_k_sw64(stage0 + 2 * A_BOX + B_BOX);
            // stage slot and the parity of its current phase, accumulator index and its phase: kept incrementally
            // in 32-bit registers (this thread's instruction stream is on the critical path)
            int s = 0;
            uint32_t ph = 0;
            int i = 0;
            for (int64_t t = lane_id; t < n_tiles; t += lanes, ++i) {
                const int a = i & 1;
                // item boundary: the previous accumulator is already handed over; wait for a free one and for
                // the first chunk
                if (i >= 2) mbar_wait_spin(accfree(a), (uint32_t)((i >> 1) - 1) & 1, &abort_flag, ctl);
                mbar_wait_spin(xfull(s), ph, &abort_flag, ctl);
                const uint32_t tacc = tmem_base + (uint32_t)(a * NBLK);
                for (int kb = 0; kb < KB; ++kb) {
                    tc_fence_after();
                    // descriptors of stage 0 plus s * STAGE / 16 in the address field (16-byte units)
                    const uint64_t doff = (uint64_t)(uint32_t)((STAGE >> 4) * s);
                    const uint64_t da1 = da1_0 + doff, da2 = da2_0 + doff, db1 = db1_0 + doff, db2 = db2_0 + doff;
                    // a k-step (16 features = 32 bytes inside the 64-byte swizzled row) advances the start address by 2
                    umma_f16_x3(tacc, da1, da2, db1, db2, idesc, kb ? 1u : 0u);
                    int sn = s + 1;
                    uint32_t phn = ph;
                    if (sn == NS) { sn = 0; phn ^= 1u; }
                    if (kb + 1 < KB) mbar_wait_spin(xfull(sn), phn, &abort_flag, ctl);
                    umma_f16_x3(tacc, da1 + 2, da2 + 2, db1 + 2, db2 + 2, idesc, 1u);
                    umma_commit(xfree(s));
                    s = sn; ph = phn;
                }
                umma_commit(accfull(a));
            }
        }
    } else if (warp == W_PANEL) {
        // ------------------------------ U panel manager ------------------------------
        // Panels (128 rows x 32 columns of U) in the order the epilogue consumes them: item, pair of 16-column
        // groups, column half.  A slot is loaded NPAN panels ahead, rewritten in place by the four warps of its
        // half and stored from the same slot; it is loaded again once that store has read it.
        if (lane == 0) {
            const int64_t my_items = (n_tiles > lane_id) ? (n_tiles - lane_id + lanes - 1) / lanes : 0;
            const int64_t total = my_items * 8;
            auto px = [&](int64_t pi) { return col0 + (int)(pi & 1) * 128 + (int)((pi >> 1) & 3) * 32; };
            auto py = [&](int64_t pi) { return (int)((lane_id + (pi >> 3) * lanes) * TILE_M); };
            auto load = [&](int64_t pi) {
                const int s = (int)(pi % NPAN);
                mbar_expect_tx(pfull(s), PAN_BYTES);
                tma_load_2d(pan0 + (uint32_t)s * PAN_BYTES, &tmU, px(pi), py(pi), pfull(s));
            };
            for (int64_t pi = 0; pi < NPAN && pi < total; ++pi) load(pi);
            for (int64_t pi = 0; pi < total; ++pi) {
                const int s = (int)(pi % NPAN);
                mbar_wait_backoff(pdone(s), (uint32_t)(pi / NPAN) & 1, &abort_flag, ctl);
                if (abort_flag) break;                 // after a time-out nothing more is stored
                if (px(pi) < r) {
                    tma_store_2d(&tmU, px(pi), py(pi), pan0 + (uint32_t)s * PAN_BYTES);
                    bulk_commit();
                    bulk_wait_read<0>();
                }
                if (pi + NPAN < total) load(pi + NPAN);
            }
            bulk_wait<0>();
        }
    } else {
        // ------------------------------ epilogue (warps 2..9) ------------------------------
        // Warp = (TMEM lane quarter q, column half).  Accumulators are read in the 16x256b fragment layout:
        // a thread holds rows q*32 + g + {0, 8, 16, 24} (g = lane / 4) and, per 16-column group, the column
        // pairs 8 b + 2 tq, + 1 (tq = lane % 4, b = 0, 1).  Neighbouring lanes (tq ^ 1) swap half of their
        // fragment, so that a thread owns four consecutive columns of each of its rows: columns cbase ..
        // cbase + 3 of the group with cbase = 0, 8, 4, 12 for tq = 0, 1, 2, 3.  The old entries of U come from
        // the group's panel in shared memory and the new ones go back into it: one 16-byte access per row
        // and direction, the eight row groups of a warp covering 512 contiguous bytes (no bank conflicts).
        const int q = warp & 3;
        const int half = (warp - 2) >> 2;
        const int g4 = lane >> 2, tq = lane & 3;
        const int et = (warp - 2) * 32 + lane;            // 0..255 among the epilogue threads
        const bool odd = tq & 1;
        const int cbase = 4 * (tq >> 1) + 8 * (tq & 1);
        // this thread's 16-byte chunk of panel row q*32 + g4 (+ 8 x: 1 KB further, same swizzle phase g4) for the
        // even and the odd group of a panel: chunk index (0..7 along the 128-byte row) XOR row mod 8
        const uint32_t row_off = (uint32_t)((q * 32 + g4) * 128);
        const uint32_t ch_even = (uint32_t)((((cbase >> 2)) ^ g4) << 4), ch_odd = (uint32_t)(((4 + (cbase >> 2)) ^ g4) << 4);
        int i = 0;
        for (int64_t t = lane_id; t < n_tiles; t += lanes, ++i) {
            const int a = i & 1;
            bool valid[4];
            float nay[4];
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const int64_t row = t * TILE_M + q * 32 + g4 + 8 * x;
                valid[x] = row < n;
                nay[x] = valid[x] ? -alpha * ybar[row] : 0.f;
            }
            float* my_tmp = stmp + (size_t)(a * 4 + q) * NBLK + half * 128;
            mbar_wait_relaxed(accfull(a), (uint32_t)(i >> 1) & 1, &abort_flag, ctl);
            tc_fence_after();
#pragma unroll 1
            for (int jj = 0; jj < 8; ++jj) {
                const int lc = half * 128 + jj * 16 + cbase;                 // this thread's four columns inside the block
                const int c = col0 + lc;
                // acc[x2][...]: x2 = 0: rows g4, g4 + 8; x2 = 1: rows g4 + 16, g4 + 24
                float acc[2][8];
                const uint32_t tcol = (uint32_t)(a * NBLK + half * 128 + jj * 16);
                tmem_ld_16x256b_x2(tmem_base + ((uint32_t)(q * 32) << 16) + tcol, acc[0]);
                tmem_ld_16x256b_x2(tmem_base + ((uint32_t)(q * 32 + 16) << 16) + tcol, acc[1]);
                const uint32_t pidx = ((uint32_t)i * 4u + (uint32_t)(jj >> 1)) * 2u + (uint32_t)half;   // this CTA's panel ordinal
                const int slot = (int)(pidx % NPAN);
                const uint32_t pan = pan0 + (uint32_t)slot * PAN_BYTES + row_off + ((jj & 1) ? ch_odd : ch_even);
                const float4 p4 = *reinterpret_cast<const float4*>(sp + lc);
                const float4 s4 = *reinterpret_cast<const float4*>(sas + lc);
                const bool cok = c < r;
                if (!(jj & 1)) mbar_wait_relaxed(pfull(slot), (pidx / NPAN) & 1u, &abort_flag, ctl);
                float4 wold[4];
#pragma unroll
                for (int x = 0; x < 4; ++x) wold[x] = lds128(pan + (uint32_t)x * 1024u);
                tmem_ld_wait();
                float cs[4] = {0.f, 0.f, 0.f, 0.f};
                float fa = 0.f, fb = 0.f, fh = 0.f;     // FP32 over the thread's 16 entries of the group, then FP64
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    // row g4 + 8 x: registers 4 b + 2 (x & 1) + {0, 1} of load x >> 1 hold columns 8 b + 2 tq + {0, 1}
                    const float b0x = acc[x >> 1][2 * (x & 1)], b0y = acc[x >> 1][2 * (x & 1) + 1];
                    const float b1x = acc[x >> 1][4 + 2 * (x & 1)], b1y = acc[x >> 1][4 + 2 * (x & 1) + 1];
                    const float rx = __shfl_xor_sync(0xffffffffu, odd ? b0x : b1x, 1);
                    const float ry = __shfl_xor_sync(0xffffffffu, odd ? b0y : b1y, 1);
                    const float av[4] = {odd ? rx : b0x, odd ? ry : b0y, odd ? b1x : rx, odd ? b1y : ry};
                    const float uw[4] = {wold[x].x, wold[x].y, wold[x].z, wold[x].w};
                    const float pv[4] = {p4.x, p4.y, p4.z, p4.w}, sv[4] = {s4.x, s4.y, s4.z, s4.w};
                    const bool live = valid[x] && cok;
                    float wv[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float u = live ? cf * uw[e] : 0.f;
                        float v = fmaf(two_alpha, av[e], u);
                        v = fmaf(nay[x], pv[e], v);
                        v -= sv[e];
                        wv[e] = live ? fmaxf(v, 0.f) : 0.f;
                        fa = fmaf(wv[e], wv[e], fa); fb = fmaf(u, u, fb); fh = fmaf(wv[e], u, fh);
                        cs[e] += wv[e];
                    }
                    sts128(pan + (uint32_t)x * 1024u, make_float4(wv[0], wv[1], wv[2], wv[3]));
                }
                // the panel's new contents are visible to the TMA store the manager issues after the four arrivals
                if (jj & 1) {
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(pdone(slot));
                }
                sa += (double)fa; sb += (double)fb; sh += (double)fh;
                // column sums over the 32 rows of the quarter: the 8 row groups g4 of the warp
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float v = cs[e];
                    v += __shfl_xor_sync(0xffffffffu, v, 4);
                    v += __shfl_xor_sync(0xffffffffu, v, 8);
                    v += __shfl_xor_sync(0xffffffffu, v, 16);
                    if (lane < 4) my_tmp[jj * 16 + cbase + e] = v;
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
                scol[et] += v;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, 512);

    // ---- CTA partial: a, b, h and the column sums of W ----
    const int PS = 4 + NBLK;
    sa = block_sum<NTHREADS>(sa, sred);
    sb = block_sum<NTHREADS>(sb, sred);
    sh = block_sum<NTHREADS>(sh, sred);
    double* out = part + (size_t)blockIdx.x * PS;
    if (threadIdx.x == 0) { out[0] = sa; out[1] = sb; out[2] = sh; out[3] = 0.0; }
    for (int j = threadIdx.x; j < NBLK; j += NTHREADS) out[4 + j] = scol[j];
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
        // column j belongs to the CTAs of block j / NBLK: fixed order over their row lanes
        const int cj = j / NBLK, k = j % NBLK;
        double v = 0.0;
        for (int l = 0; l < lanes; ++l) v += __ldcg(part + (size_t)(l * NCB + cj) * PS + 4 + k);
        p_out[j] = (float)(sc * v);
    }
}


// ================================================================================================
// First product for the same wide problems:  Theta = X-hat^T U  as Theta^T tiles, u = c_f w.
//
// Work item (one CTA each, all resident at once) = (128 columns of U, up to 256 features, one of
// NSPLIT contiguous row ranges).  The contraction runs over the data rows, the slow (MN-major)
// operand orientation of the tensor core, so both operands are presented K-major instead: the X-hat
// side comes from the transposed fp16 images built at setup (one contiguous, pre-swizzled 16 KB box per
// stage and 256-feature block, bulk-copied straight into the image stage); the U side is transposed on the fly: TMA brings
// the 32 x 128 FP32 slice of the stage, a team of four warps (thread = column) scales by c_f and a power
// of two, splits u 2^k = h1 + h2 in fp16 and writes one 16-byte chunk per (column, 8 rows).  The MMA
// issuer runs 2 k-steps (K = 16) x 3 products per stage with M = 128, N = 256 into one of two TMEM
// accumulators, which is handed to the epilogue every FLUSH1 stages (8192 rows) and folded, rescaled, into the FP64
// partial of this row range (layout [feature][column] like the generic first product, so the same
// reduction kernel follows).  The row-local vector work cannot be fused here (a CTA sees 128 of the r
// columns): it runs as the separate vector pass before this kernel.
// ================================================================================================
constexpr int TR1 = 32;                        // data rows per stage (2 k-steps of 16)
constexpr int NT1 = 2;                         // teams of four warps on alternate stages
constexpr int NIM1 = 3, NRAW1 = 4;             // image stages, raw U stages
// Ring sizes and the two alternating teams.  A wait on an mbarrier names a phase by its parity only, so a waiter
// must never be two phases behind the barrier it polls.  NRAW1 is a multiple of NT1: a raw slot always belongs to
// the same team, which therefore sees each of its phases (with three slots the teams took turns on a slot, and a
// team could find the barrier still in the other team's phase, whose parity reads as "done": on a late TMA
// load it then converted a stale slice -- one 32-row stage of a few 32-column groups wrong, about once in
// twenty-five launches at n = 2 x 10^6 with 147 CTAs).  The image slots may rotate through both teams (NIM1 >=
// NT1 is enough there): a team that has seen the MMAs of stage g - 2 finish knows that those of stage g - 6
// have, so the barrier of its slot is at most one phase away from the one it names.
constexpr int URAW1 = TR1 * 128 * 4;           // raw U slice: 32 rows x 128 columns FP32 = 16 KB
constexpr int UIMG1 = 128 * 64;                // fp16 image of the U operand: 128 columns x 32 data rows
constexpr int XIMG1 = 256 * 64;                // fp16 image of the X-hat operand: 256 features x 32 data rows
constexpr int IMG1 = 2 * UIMG1 + 2 * XIMG1;    // U h1, U h2, X h1, X h2: 48 KB
constexpr int FLUSH1 = 256;                    // stages per accumulation period (8192 rows)
// The tensor core's FP32 accumulation rounds with a bias, so the error of a period grows linearly with its length:
// against an FP64 Theta at n = 2 x 10^6, d = 768, r = 1000 the largest deviation is 4.0e-5 of max |Theta| with 256
// stages per period and 1.5e-4 with 1024 (rms 8e-6 and 3.2e-5); U after the step is unchanged (2.9e-7 either way).
// Longer periods save fold traffic and time (first phase 10.5 ms at 128, 10.2 at 256, 10.0 at 512, 9.9 at 1024);
// 256 keeps Theta at the accuracy of a plain FP32 accumulation over that many rows.
constexpr int NTH1 = 16 * 32;
// Warp roles of the first product.  A warp runs on scheduler (warp index mod 4) and the thread that issues the
// MMAs executes a serial instruction stream whose speed sets the stage rate, so scheduler 1 hosts only light
// roles: the issuer (warp 1), one epilogue warp (5; the TMEM lane quarter of a warp is its index mod 4), the
// two producers (9, 13).  The eight team warps are 0, 2, 3, 8, 10, 11, 12, 14 (15 idles).
constexpr int W1_ISSUER = 1, W1_EPI0 = 4, W1_UPROD = 9, W1_XPROD = 13;
__device__ __forceinline__ bool is_team_warp1(int w) { return (w & 3) != 1 && (w >> 2) != 1 && w != 15; }
__device__ __forceinline__ int team_warp_index1(int w)         // 0 .. 7 over the team warps in increasing order
{
    const int q = w >> 2, res = w & 3;
    return (q == 0 ? 0 : q - 1) * 3 + (res == 0 ? 0 : res - 1);
}

__global__ void __launch_bounds__(NTH1, 1)
k_pass1_tcg(const __grid_constant__ CUtensorMap tmU, const __half* __restrict__ xT1,
            const __half* __restrict__ xT2, Ctl* __restrict__ ctl, int64_t n, int d, int r, int K,
            int NMT, int NNB, int NSPLIT, int fb, double* __restrict__ part)
{
    if (ctl->stopped) return;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t bars[2 * NIM1 + 2 * NRAW1 + 4];
    __shared__ uint32_t abort_flag;
    __shared__ uint32_t tmem_base_s;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int mt = blockIdx.x % NMT, nb = (blockIdx.x / NMT) % NNB, sp = blockIdx.x / (NMT * NNB);
    const int c0 = mt * 128;                               // first column of U of this item
    const int f0 = nb * fb;                                // fb = features per block of the transposed images: 256, or d < 256
    const int Nb = (d - f0 < fb) ? d - f0 : fb;            // features of this item (multiple of 32)

    const uint32_t img0 = smem_u32(smem);
    const uint32_t raw0 = img0 + (uint32_t)NIM1 * IMG1;
    const uint32_t bar0 = smem_u32(bars);
    auto imgfull = [&](int l) { return bar0 + 8u * l; };
    auto imgfree = [&](int l) { return bar0 + 8u * (NIM1 + l); };
    auto ufull = [&](int s) { return bar0 + 8u * (2 * NIM1 + s); };
    auto ufree = [&](int s) { return bar0 + 8u * (2 * NIM1 + NRAW1 + s); };
    auto accfull = [&](int a) { return bar0 + 8u * (2 * NIM1 + 2 * NRAW1 + a); };
    auto accfree = [&](int a) { return bar0 + 8u * (2 * NIM1 + 2 * NRAW1 + 2 + a); };
    if (threadIdx.x == 0) {
        for (int l = 0; l < NIM1; ++l) { mbar_init(imgfull(l), 4 + 1); mbar_init(imgfree(l), 1); }   // team warps + X-hat boxes
        for (int s = 0; s < NRAW1; ++s) { mbar_init(ufull(s), 1); mbar_init(ufree(s), 4); }
        for (int a = 0; a < 2; ++a) { mbar_init(accfull(a), 1); mbar_init(accfree(a), 4); }
        abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == W1_ISSUER) tmem_alloc(smem_u32(&tmem_base_s), 512);
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
    const float cf = ctl->c_f;
    // power-of-two operand scales: x-hat 2^15 (in the images), u 2^eU with |u| 2^eU <= 2^14
    int eU;
    {
        int e;
        frexpf(sqrtf((float)K), &e);                       // |u_ij| <= ||U||_F = sqrt(K) <= 2^e
        eU = 14 - e;
    }
    const float sU = ldexpf(1.0f, eU);
    const double unscale = ldexp(1.0, -15 - eU);

    if (warp == W1_UPROD) {
        // ------------------------------ producer ------------------------------
        if (lane == 0) {
            for (int g = 0; g < my_stages && !abort_flag; ++g) {
                const int s = g % NRAW1;
                const int row0 = (int)((g_lo + g) * TR1);
                if (g >= NRAW1) mbar_wait_backoff(ufree(s), ((g / NRAW1) - 1) & 1, &abort_flag, ctl);
                mbar_expect_tx(ufull(s), URAW1);
                tma_load_2d(raw0 + (uint32_t)s * URAW1, &tmU, c0, row0, ufull(s));
            }
        }
    } else if (warp == W1_XPROD) {
        // ------------------------------ X-hat image producer ------------------------------
        // Its own thread: the image ring is released by the MMAs, the raw U ring by the teams; one thread
        // serving both would let the U loads run only one stage ahead.
        if (lane == 0) {
            for (int g = 0; g < my_stages && !abort_flag; ++g) {
                const int l = g % NIM1;
                if (g >= NIM1) mbar_wait_backoff(imgfree(l), ((g / NIM1) - 1) & 1, &abort_flag, ctl);
                const uint32_t im = img0 + (uint32_t)l * IMG1;
                const size_t xoff = ((size_t)(g_lo + g) * NNB + nb) * ((size_t)fb * 32);   // this stage's box of the feature block
                const uint32_t xbytes = (uint32_t)fb * 64;
                mbar_expect_tx(imgfull(l), 2 * xbytes);
                bulk_load_1d(im + 2 * UIMG1, xT1 + xoff, xbytes, imgfull(l));
                bulk_load_1d(im + 2 * UIMG1 + XIMG1, xT2 + xoff, xbytes, imgfull(l));
            }
        }
    } else if (warp == W1_ISSUER) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_f16(128, Nb, 0, 0);
            if (my_stages > 0) mbar_wait_spin(imgfull(0), 0, &abort_flag, ctl);
            int l = 0, lph = 0, a = 0, in_period = 0, period = 0;
            // descriptors of image stage 0; the address field counts 16-byte units, so stage l adds l * IMG1 / 16
            const uint64_t da1_0 = umma_desc_k_sw64(img0), da2_0 = umma_desc_k_sw64(img0 + UIMG1);
            const uint64_t db1_0 = umma_desc_k_sw64(img0 + 2 * UIMG1), db2_0 = umma_desc_k_sw64(img0 + 2 * UIMG1 + XIMG1);
            for (int g = 0; g < my_stages; ++g) {
                if (in_period == 0 && period >= 2) mbar_wait_spin(accfree(a), ((period >> 1) - 1) & 1, &abort_flag, ctl);
                tc_fence_after();
                const uint32_t tacc = tmem_base + (uint32_t)(a * 256);
                // K-major images; a k-step of 16 data rows (32 bytes inside the 64-byte swizzled row) advances
                // the start address by 2
                const uint64_t doff = (uint64_t)(IMG1 >> 4) * (uint64_t)l;
                const uint64_t da1 = da1_0 + doff, da2 = da2_0 + doff, db1 = db1_0 + doff, db2 = db2_0 + doff;
                umma_f16_x3(tacc, da1, da2, db1, db2, idesc, in_period ? 1u : 0u);
                int ln = l + 1, lphn = lph;
                if (ln == NIM1) { ln = 0; lphn ^= 1; }
                if (g + 1 < my_stages) mbar_wait_spin(imgfull(ln), (uint32_t)lphn, &abort_flag, ctl);
                umma_f16_x3(tacc, da1 + 2, da2 + 2, db1 + 2, db2 + 2, idesc, 1u);
                umma_commit(imgfree(l));
                if (in_period == FLUSH1 - 1 || g == my_stages - 1) umma_commit(accfull(a));
                l = ln; lph = lphn;
                if (++in_period == FLUSH1) { in_period = 0; ++period; a ^= 1; }
            }
        }
    } else if (is_team_warp1(warp)) {
        // ------------------------------ U teams: FP32 slice -> K-major fp16 images ------------------------------
        const int vw = team_warp_index1(warp), team = vw >> 2, tw = vw & 3;
        const int tt = tw * 32 + lane;                     // column of the slice
        for (int g = team; g < my_stages; g += NT1) {
            const int s = g % NRAW1, l = g % NIM1;
            mbar_wait_backoff(ufull(s), (g / NRAW1) & 1, &abort_flag, ctl);
            const uint32_t rs = raw0 + (uint32_t)s * URAW1;
            float uv[4][8];
#pragma unroll
            for (int kg = 0; kg < 4; ++kg)
#pragma unroll
                for (int k = 0; k < 8; ++k) uv[kg][k] = lds32f(rs + (uint32_t)(((8 * kg + k) * 128 + tt) * 4));
            if (g >= NIM1) mbar_wait_backoff(imgfree(l), ((g / NIM1) - 1) & 1, &abort_flag, ctl);
            const uint32_t im = img0 + (uint32_t)l * IMG1;
#pragma unroll
            for (int kg = 0; kg < 4; ++kg) {
                float v[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) v[k] = (cf * uv[kg][k]) * sU;      // u = c_f w rounded to FP32, then scaled
                uint4 h1, h2;
                split_h8(v, h1, h2);
                const uint32_t io = kimg_off(tt, kg);
                sts128u(im + io, h1);
                sts128u(im + UIMG1 + io, h2);
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(imgfull(l));
                mbar_arrive(ufree(s));
            }
        }
    } else if (warp >= W1_EPI0 && warp < W1_EPI0 + 4) {
        // ------------------------------ epilogue: FP64 fold of the accumulator (warps 4-7) ------------------------------
        // thread = column j of U (TMEM lane); entry (feature f, column j) of this row range's partial
        const int q4 = warp & 3;
        const int j = c0 + q4 * 32 + lane;
        double* const out = part + (size_t)sp * ((size_t)d * r);
        for (int period = 0; period < n_periods; ++period) {
            const int a = period & 1;
            mbar_wait_relaxed(accfull(a), (period >> 1) & 1, &abort_flag, ctl);
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
                    for (int k = 0; k < 16; ++k) o[(size_t)k * r] = prev[k] + unscale * (double)v[k];
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(accfree(a));
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == W1_ISSUER) tmem_dealloc(tmem_base, 512);
}

}  // namespace tcg

bool tcg_plan(const Problem& pb, TcgPlan* pl, float* img_storage)
{
    const int d = pb.P.d, r = pb.P.r;
    if (!pb.has_ximg() || d % tcg::KC != 0 || r % 4 != 0 || pb.P.n < 4096 || pb.P.n > 2000000000ll) return false;
    const int NCB = (r + tcg::NBLK - 1) / tcg::NBLK;
    const int RP = NCB * tcg::NBLK;
    if (RP > 2048) return false;
    pl->NCB = NCB;
    {
        int e;
        frexpf(sqrtf((float)pb.P.K), &e);                  // |Theta_jk| <= ||X-hat||_2 ||U||_F = sqrt(K) <= 2^e
        pl->eT = 14 - e;
    }
    pl->smem2 = tcg::SMEM_RING + (size_t)tcg::NPAN * tcg::PAN_BYTES + (size_t)tcg::NBLK * (4 + 4 + 8) + (size_t)2 * 4 * tcg::NBLK * 4 + 1024;
    if (!make_tensor_map_2d(&pl->tmU, pb.U, pb.P.n, r, tcg::TILE_M, 32, false, 128)) return false;     // U panels: 128-byte rows, 128-byte swizzle
    if (pl->smem2 > 227 * 1024 - 1024) return false;
    pl->img_h1 = img_storage;
    pl->img_h2 = reinterpret_cast<uint16_t*>(img_storage) + (size_t)d * RP;
    if (!make_tensor_map_2d_f16(&pl->tmX1, pb.ximg(0), pb.P.n, d, pb.ximg_pitch(), tcg::TILE_M, tcg::KC)) return false;
    if (!make_tensor_map_2d_f16(&pl->tmX2, pb.ximg(1), pb.P.n, d, pb.ximg_pitch(), tcg::TILE_M, tcg::KC)) return false;
    // one column block per CTA: (SMs / NCB) row lanes x NCB blocks
    const int64_t tiles = (pb.P.n + tcg::TILE_M - 1) / tcg::TILE_M;
    const int64_t lanes = tiles < kSMs / NCB ? tiles : kSMs / NCB;
    pl->g2 = (int)lanes * NCB;
    if (cudaFuncSetAttribute(tcg::k_pass2_tcg, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl->smem2) != cudaSuccess)
        return false;
    return true;
}

void tcg_prepare(const Problem& pb)
{
    cudaMemsetAsync(pb.ximgT(0), 0, sizeof(uint16_t) * 2 * pb.ximgT_halves(), pb.stream);
    if (pb.L.img_inplace) {
        const size_t sm = sizeof(float) * 32 * (size_t)(pb.P.d + 1);
        cudaFuncSetAttribute(tcg::k_ximg_build_inplace, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
        const int64_t stages = pb.L.n_pad / 32;
        tcg::k_ximg_build_inplace<<<(int)(stages < kSMs ? stages : kSMs), 256, sm, pb.stream>>>(
            pb.X, pb.P.n, pb.P.d, pb.L.n_pad, pb.L.fb, reinterpret_cast<__half*>(pb.ximgT(0)), reinterpret_cast<__half*>(pb.ximgT(1)));
        pb.count(1);
        return;
    }
    const dim3 grid((unsigned)((pb.L.n_pad + 31) / 32), (unsigned)((pb.P.d + 31) / 32));
    tcg::k_ximg_build<<<grid, 256, 0, pb.stream>>>(pb.X, pb.P.n, pb.dx, pb.P.d, pb.L.n_pad, pb.L.fb,
                                                   reinterpret_cast<__half*>(pb.ximg(0)), reinterpret_cast<__half*>(pb.ximg(1)),
                                                   reinterpret_cast<__half*>(pb.ximgT(0)), reinterpret_cast<__half*>(pb.ximgT(1)));
    pb.count(1);
}

bool tcg1_plan(const Problem& pb, Tcg1Plan* pl)
{
    const int d = pb.P.d, r = pb.P.r;
    // 256-feature blocks only (d >= 256): narrower blocks with more row ranges are not enabled
    if (!pb.has_ximg() || pb.L.fb != 256 || d % 32 != 0 || r % 4 != 0 || pb.P.n < 4096 || pb.P.n > 2000000000ll) return false;
    pl->NMT = (r + 127) / 128;
    pl->NNB = (d + pb.L.fb - 1) / pb.L.fb;
    const int tiles = pl->NMT * pl->NNB;
    if (tiles > kSMs) return false;
    pl->NSPLIT = tiled_first_row_ranges(pb.P.n, d, r);              // the partial area is sized with the same rule
    if (pl->NSPLIT < 1 || sizeof(double) * (size_t)pl->NSPLIT * d * r > pb.L.part1_bytes) return false;
    pl->grid = tiles * pl->NSPLIT;
    pl->smem = (size_t)tcg::NIM1 * tcg::IMG1 + (size_t)tcg::NRAW1 * tcg::URAW1 + 1024;
    if (!make_tensor_map_2d(&pl->tmU, pb.U, pb.P.n, r, tcg::TR1, 128, false, 1)) return false;     // plain FP32 rows
    if (cudaFuncSetAttribute(tcg::k_pass1_tcg, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl->smem) != cudaSuccess)
        return false;
    return true;
}

void tcg_launch_first(const Problem& pb, const Tcg1Plan& pl)
{
    tcg::k_pass1_tcg<<<pl.grid, tcg::NTH1, pl.smem, pb.stream>>>(pl.tmU, reinterpret_cast<const __half*>(pb.ximgT(0)),
                                                                 reinterpret_cast<const __half*>(pb.ximgT(1)), pb.ctl(), pb.P.n, pb.P.d, pb.P.r,
                                                                 pb.P.K, pl.NMT, pl.NNB, pl.NSPLIT, pb.L.fb, pb.part1());
    pb.count(1);
    launch_red1(pb, pl.NSPLIT, 0, 0);
}

void tcg_launch_second(const Problem& pb, const TcgPlan& pl)
{
    const int d = pb.P.d, r = pb.P.r;
    __half* i1 = reinterpret_cast<__half*>(pl.img_h1);
    __half* i2 = reinterpret_cast<__half*>(pl.img_h2);
    tcg::k_theta_images64<<<kSMs * 4, 256, 0, pb.stream>>>(pb.theta(), d, r, pl.NCB, pl.eT, pb.ctl(), i1, i2);
    tcg::k_pass2_tcg<<<pl.g2, tcg::NTHREADS, pl.smem2, pb.stream>>>(
        pl.tmX1, pl.tmX2, pl.tmU, i1, i2, pb.U, pb.ybar(), pb.p(), pb.alpha_s(), pb.ctl(), pb.P.n, d, r, pl.NCB, pl.eT,
        pb.P.alpha, pb.P.K, pb.P.eps_d, pb.part2(), pb.p());
    pb.count(2);
}

}  // namespace gemnlr
