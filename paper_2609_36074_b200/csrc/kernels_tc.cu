// 3xTF32 tensor-core family (tcgen05 + TMEM): the fused second product of the iteration,
//   acc = X-hat Theta ;  W = [U + 2 alpha acc - alpha (ybar p^T + 1 s^T)]_+ in place ;  FP64 a, b, h ;
//   column sums of W,
// for shapes where FP32 FFMA cannot keep up with HBM (d >= 64 with r >= 16).
//
// FP32 accuracy from TF32 tensor cores: each operand is split as x = hi + lo with hi exactly
// representable in TF32, and the product is accumulated as hi*hi' + lo*hi' + hi*lo' (three MMAs
// into the same TMEM accumulator); the dropped lo*lo' term is below 2^-22 relative.
//
// One persistent CTA per SM, 22 warps:
//   warp 0      producer: TMA loads of X-hat boxes (128 rows x 32 features, 128-byte swizzle = the
//               K-major UMMA operand layout) and of U panels (128 rows x 32 columns); the pre-split
//               Theta^T images are brought in once per CTA.
//   warps 18-21 split: lo image (x - trunc(x)) of each box in a second buffer; the raw box is the hi
//               operand as it is (kind::tf32 ignores the low 13 mantissa bits).
//   warp 1      MMA issuer: per box 4 k-steps x 3 tcgen05.mma (M = 128 rows, N = padded r);
//               tcgen05.commit frees the stage and publishes the accumulator (two TMEM buffers).
//   warps 2-17  epilogue, four groups taking the panels of a tile round-robin: thread = row;
//               tcgen05.ld of 16 columns at a time, entrywise update
//               against the U panel in shared memory, FP64 statistics, W written back into the
//               panel and stored with a TMA tile store; column sums by a transposed second sweep.
// The last CTA reduces the per-CTA partials in CTA order and runs the scalar step.
// Every mbarrier wait is bounded; on expiry the kernel flags GEM_NLR_E_TIMEOUT, stops waiting,
// runs to its end and frees its TMEM.
#include "nlr_common.cuh"
#include "device_utils.cuh"
#include "fin_logic.cuh"
#include "pipeline.cuh"
#include "tc_common.cuh"
#include "tc_family.cuh"

namespace gemnlr {
namespace tc {

constexpr int TILE_M = 128;
constexpr int BOX_BYTES = TILE_M * 128;       // 128 rows x 32 floats
constexpr int NGROUPS = 4;               // epilogue warp groups; group g owns panels pn = g (mod 4)
constexpr int NTHREADS = (2 + 4 * NGROUPS + 4 + 1) * 32;   // X producer, MMA, 16 epilogue, 4 split, U-panel producer warps
constexpr int GROUP_THREADS = 128;
constexpr int MAX_RING = 8;

// Theta (d x r, FP32 row-major) -> two images of Theta^T in the K-major 128-byte-swizzled UMMA
// layout: box b (features 32b..32b+31) holds NP rows (columns of Theta, zero beyond r) of 128 bytes.
__global__ void k_theta_images(const float* __restrict__ theta, int d, int r, int NP, const Ctl* __restrict__ ctl,
                               float* __restrict__ img_hi, float* __restrict__ img_lo)
{
    if (ctl->stopped) return;
    const int NB = d / 32;
    const int total = NB * 32 * NP;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < total; e += gridDim.x * blockDim.x) {
        const int j = e / NP, k = e % NP;             // feature, column
        const float v = (k < r) ? theta[(size_t)j * r + k] : 0.f;
        const float hi = tf32_hi(v);
        const int b = j >> 5, jj = j & 31, c = jj >> 2, w = jj & 3;
        const size_t off = (size_t)b * NP * 32 + (size_t)k * 32 + (((c ^ (k & 7)) << 2) + w);
        img_hi[off] = hi;
        img_lo[off] = v - hi;
    }
}

// FP16 variant of the images for the two-term fp16 split: Theta^T 2^eT = h1 + h2, boxes of NP rows x 64 bytes
// (32 features) with the 64-byte swizzle.
__global__ void k_theta_images_h(const float* __restrict__ theta, int d, int r, int NP, int eT, const Ctl* __restrict__ ctl,
                                 __half* __restrict__ img_h1, __half* __restrict__ img_h2)
{
    if (ctl->stopped) return;
    const float sT = ldexpf(1.0f, eT);
    const int NB = d / 32;
    const int total = NB * 32 * NP;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < total; e += gridDim.x * blockDim.x) {
        const int j = e / NP, k = e % NP;             // feature, column
        const float v = (k < r) ? theta[(size_t)j * r + k] * sT : 0.f;
        const __half h1 = __float2half_rn(v);
        const __half h2 = __float2half_rn(v - __half2float(h1));
        const int b = j >> 5, jj = j & 31, c = jj >> 3, w = jj & 7;
        const size_t off = (size_t)b * NP * 32 + (size_t)k * 32 + (((c ^ ((k >> 1) & 3)) << 3) + w);
        img_h1[off] = h1;
        img_h2[off] = h2;
    }
}

// F16 = false: 3-product TF32 split, X-hat boxes split inside the kernel (warps 18-21).
// F16 = true:  3-product FP16 split on the static fp16 images of X-hat (tmX = image h1, tmX2 = image h2: boxes
//              of 128 rows x 32 features = 64-byte rows, 64-byte swizzle) and fp16 Theta^T images; K = 16 MMAs,
//              nothing is split inside the kernel and the accumulator carries the scale 2^(15 + eT).
template <bool F16>
__global__ void __launch_bounds__(NTHREADS, 1)
k_pass2_tc(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmX2,
           const __grid_constant__ CUtensorMap tmU, int eT,
           const float* __restrict__ U, const float* __restrict__ img_hi, const float* __restrict__ img_lo,
           const float* __restrict__ ybar, const float* __restrict__ p, const float* __restrict__ alpha_s,
           Ctl* __restrict__ ctl, int64_t n, int d, int r, int NP, int PW, int NSB, int NLO, int NUP, float alpha, int K,
           double eps_d, double* __restrict__ part, float* __restrict__ p_out)
{
    if (ctl->stopped) return;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t bars[6 * MAX_RING + 5];
    __shared__ uint32_t abort_flag;
    __shared__ uint32_t tmem_base_s;
    __shared__ double sred[32];
    __shared__ int is_last;
    __shared__ double sc;
    __shared__ int sok;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int NB = d / 32;                         // boxes (k blocks) per tile
    const int NPAN = (r + PW - 1) / PW;            // PW-column panels of U per tile (PW = 16 or 32)
    const int ACC_COLS = (NPAN * PW + 31) / 32 * 32;   // TMEM columns per accumulator buffer
    const int PAN_BYTES = TILE_M * PW * 4;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < 2 * ACC_COLS) tmem_cols <<= 1;
    const uint32_t th_bytes = (uint32_t)NB * NP * (F16 ? 64 : 128);

    const uint32_t smem_base = smem_u32(smem);
    const uint32_t stage0 = smem_base;                                   // NSB boxes: raw, then hi in place
    const uint32_t lo0 = stage0 + (uint32_t)NSB * BOX_BYTES;             // NLO boxes: lo parts
    const uint32_t th_hi_s = lo0 + (uint32_t)NLO * BOX_BYTES;
    const uint32_t th_lo_s = th_hi_s + th_bytes;
    const uint32_t upan0 = th_lo_s + th_bytes;                           // NUP panels
    float* sp = reinterpret_cast<float*>(smem + (size_t)(NSB + NLO) * BOX_BYTES + (size_t)NUP * PAN_BYTES +
                                         2 * (size_t)th_bytes);          // p, then alpha*s
    float* sas = sp + ACC_COLS;

    const uint32_t bar0 = smem_u32(bars);
    auto xfull = [&](int s) { return bar0 + 8u * s; };
    auto xsplit = [&](int s) { return bar0 + 8u * (MAX_RING + s); };
    auto xfree = [&](int s) { return bar0 + 8u * (2 * MAX_RING + s); };
    auto ufull = [&](int s) { return bar0 + 8u * (3 * MAX_RING + s); };
    auto ufree = [&](int s) { return bar0 + 8u * (4 * MAX_RING + s); };
    auto lofree = [&](int s) { return bar0 + 8u * (5 * MAX_RING + s); };
    auto accfull = [&](int a) { return bar0 + 8u * (6 * MAX_RING + a); };
    auto accfree = [&](int a) { return bar0 + 8u * (6 * MAX_RING + 2 + a); };
    const uint32_t thfull = bar0 + 8u * (6 * MAX_RING + 4);

    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_RING; ++s) {
            mbar_init(xfull(s), 1); mbar_init(xsplit(s), 4); mbar_init(xfree(s), 1);
            mbar_init(ufull(s), 1); mbar_init(ufree(s), 1); mbar_init(lofree(s), 1);
        }
        for (int a = 0; a < 2; ++a) { mbar_init(accfull(a), 1); mbar_init(accfree(a), 4 * NGROUPS); }
        mbar_init(thfull, 1);
        abort_flag = 0;
        fence_barrier_init();
    }
    for (int j = threadIdx.x; j < ACC_COLS; j += NTHREADS) {
        sp[j] = (j < r) ? p[j] : 0.f;
        sas[j] = (j < r) ? alpha_s[j] : 0.f;
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_s), tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;

    const int64_t n_tiles = (n + TILE_M - 1) / TILE_M;
    const float cf = ctl->c_f;
    // F16: the accumulator holds (x-hat 2^15)(Theta 2^eT) sums; the scales go into the 2 alpha factor
    const float two_alpha = F16 ? 2.0f * alpha * ldexpf(1.0f, -15 - eT) : 2.0f * alpha;
    double sa = 0.0, sb = 0.0, sh = 0.0;
    double csum[2][2];                   // epilogue thread: running sums of its column (after the transpose-reduce) per
    csum[0][0] = csum[0][1] = csum[1][0] = csum[1][1] = 0.0;   // (panel of the group, 16-column half); over this quarter's rows

    if (warp == 0) {
        // ------------------------------ producer ------------------------------
        if (lane == 0) {
            mbar_expect_tx(thfull, 2 * th_bytes);
            bulk_load_1d(th_hi_s, img_hi, th_bytes, thfull);
            bulk_load_1d(th_lo_s, img_lo, th_bytes, thfull);
            int i = 0;
            for (int64_t t = blockIdx.x; t < n_tiles && !abort_flag; t += gridDim.x, ++i) {
                const int row0 = (int)(t * TILE_M);
                for (int b = 0; b < NB; ++b) {
                    const int g = i * NB + b, s = g % NSB;
                    if (g >= NSB) mbar_wait(xfree(s), ((g / NSB) - 1) & 1, &abort_flag, ctl);
                    mbar_expect_tx(xfull(s), BOX_BYTES);
                    if (F16) {      // image boxes h1 | h2, 8 KB each
                        tma_load_2d(stage0 + (uint32_t)s * BOX_BYTES, &tmX, b * 32, row0, xfull(s));
                        tma_load_2d(stage0 + (uint32_t)s * BOX_BYTES + BOX_BYTES / 2, &tmX2, b * 32, row0, xfull(s));
                    } else {
                        tma_load_2d(stage0 + (uint32_t)s * BOX_BYTES, &tmX, b * 32, row0, xfull(s));
                    }
                }
            }
        }
    } else if (warp == 2 + 4 * NGROUPS + 4) {
        // ------------------------------ U-panel producer ------------------------------
        // Its own thread, so that waiting for a free panel slot (the epilogue of the previous tile) never
        // holds back the X-hat loads of the next tile.  The U rows of the tile after next (one contiguous
        // block) are asked into L2 ahead of time: a slot is refilled only once its group has stored the
        // previous panel, and the refill should then not pay DRAM latency.
        if (lane == 0) {
            int i = 0;
            for (int64_t t = blockIdx.x; t < n_tiles && !abort_flag; t += gridDim.x, ++i) {
                const int row0 = (int)(t * TILE_M);
                {
                    const int64_t tn = t + gridDim.x;
                    if (tn < n_tiles) {
                        const int64_t r0 = tn * TILE_M, r1 = (r0 + TILE_M < n) ? r0 + TILE_M : n;
                        const char* src = reinterpret_cast<const char*>(U + r0 * (int64_t)r);
                        const int64_t bytes = (r1 - r0) * (int64_t)r * 4;        // multiple of 16: r is a multiple of 4
                        for (int64_t o = 0; o < bytes; o += 16384)
                            bulk_prefetch_l2(src + o, (uint32_t)(bytes - o < 16384 ? bytes - o : 16384));
                    }
                }
                for (int pn = 0; pn < NPAN; ++pn) {
                    // slot and phase of the panel inside its epilogue group's own part of the ring (see the epilogue)
                    const int eg = pn % NGROUPS, depth = NUP / NGROUPS;
                    const int cnt = i * ((NPAN - eg + NGROUPS - 1) / NGROUPS) + pn / NGROUPS;
                    const int sl = eg + NGROUPS * (cnt % depth);
                    if (cnt >= depth) mbar_wait(ufree(sl), ((cnt / depth) - 1) & 1, &abort_flag, ctl);
                    mbar_expect_tx(ufull(sl), PAN_BYTES);
                    tma_load_2d(upan0 + (uint32_t)sl * PAN_BYTES, &tmU, pn * PW, row0, ufull(sl));
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            const uint32_t idesc = F16 ? umma_idesc_f16(TILE_M, NP, 0, 0) : umma_idesc_tf32(TILE_M, NP, 0, 0);
            mbar_wait_spin(thfull, 0, &abort_flag, ctl);
            // Inside a tile the wait for the next box sits in the middle of the current box's k-steps, so the
            // tensor pipe has MMAs queued while this thread polls.  F16: the boxes come ready from TMA (xfull);
            // TF32: from the split warps (xsplit).  Ring positions and phase parities are kept incrementally in
            // 32-bit registers and the barrier is polled without suspension: this thread's instruction stream
            // shares a scheduler with four epilogue warps and sets the rate at which MMAs reach the tensor pipe.
            int s = 0, l = 0;
            uint32_t sph = 0;                    // parity of the current fill of box slot s
            int i = 0;
            for (int64_t t = blockIdx.x; t < n_tiles; t += gridDim.x, ++i) {
                const int a = i & 1;
                // tile boundary: the accumulator hand-over of the previous tile is already committed, so the
                // epilogue runs while this thread waits for a free accumulator and the first box
                if (i >= 2) mbar_wait_spin(accfree(a), ((i >> 1) - 1) & 1, &abort_flag, ctl);
                mbar_wait_spin(F16 ? xfull(s) : xsplit(s), sph, &abort_flag, ctl);
                const uint32_t tacc = tmem_base + (uint32_t)(a * ACC_COLS);
                for (int b = 0; b < NB; ++b) {
                    int sn = s + 1;
                    uint32_t sphn = sph;
                    if (sn == NSB) { sn = 0; sphn ^= 1u; }
                    tc_fence_after();
                    if (F16) {
                        const uint32_t a_h1 = stage0 + (uint32_t)s * BOX_BYTES, a_h2 = a_h1 + BOX_BYTES / 2;
                        const uint32_t b_h1 = th_hi_s + (uint32_t)b * NP * 64, b_h2 = th_lo_s + (uint32_t)b * NP * 64;
                        const uint64_t da1 = umma_desc_k_sw64(a_h1), da2 = umma_desc_k_sw64(a_h2);
                        const uint64_t db1 = umma_desc_k_sw64(b_h1), db2 = umma_desc_k_sw64(b_h2);
                        umma_f16_x3(tacc, da1, da2, db1, db2, idesc, b ? 1u : 0u);
                        if (b + 1 < NB) mbar_wait_spin(xfull(sn), sphn, &abort_flag, ctl);
                        umma_f16_x3(tacc, da1 + 2, da2 + 2, db1 + 2, db2 + 2, idesc, 1u);
                        umma_commit(xfree(s));
                    } else {
                        const uint32_t a_hi = stage0 + (uint32_t)s * BOX_BYTES, a_lo = lo0 + (uint32_t)l * BOX_BYTES;
                        const uint32_t b_hi = th_hi_s + (uint32_t)b * NP * 128, b_lo = th_lo_s + (uint32_t)b * NP * 128;
                        // descriptors once per box; a k-step (8 features = 32 bytes inside the 128-byte
                        // swizzled row) advances the start-address field by 2
                        const uint64_t da_hi = umma_desc_sw128(a_hi, 16, 1024), da_lo = umma_desc_sw128(a_lo, 16, 1024);
                        const uint64_t db_hi = umma_desc_sw128(b_hi, 16, 1024), db_lo = umma_desc_sw128(b_lo, 16, 1024);
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {
                            if (ks == 2 && b + 1 < NB) mbar_wait_spin(xsplit(sn), sphn, &abort_flag, ctl);
                            umma_tf32_x3(tacc, da_hi + 2 * ks, da_lo + 2 * ks, db_hi + 2 * ks, db_lo + 2 * ks, idesc,
                                         (b | ks) ? 1u : 0u);
                        }
                        umma_commit(xfree(s));
                        umma_commit(lofree(l));
                        if (++l == NLO) l = 0;
                    }
                    s = sn; sph = sphn;
                }
                umma_commit(accfull(a));
            }
        }
    } else if (warp >= 2 + 4 * NGROUPS && warp < 2 + 4 * NGROUPS + 4) {
        // ------------------------------ split: box -> hi (in place), lo ------------------------------
        const int st = threadIdx.x - (2 + 4 * NGROUPS) * 32;   // 0..127
        int i = 0;
        for (int64_t t = blockIdx.x; !F16 && t < n_tiles; t += gridDim.x, ++i) {
            for (int b = 0; b < NB; ++b) {
                const int g = i * NB + b, s = g % NSB, l = g % NLO;
                mbar_wait(xfull(s), (g / NSB) & 1, &abort_flag, ctl);
                if (g >= NLO) mbar_wait(lofree(l), ((g / NLO) - 1) & 1, &abort_flag, ctl);
                const uint32_t hi_a = stage0 + (uint32_t)s * BOX_BYTES, lo_a = lo0 + (uint32_t)l * BOX_BYTES;
                float4 xin[BOX_BYTES / 16 / 128];
#pragma unroll
                for (int k = 0; k < BOX_BYTES / 16 / 128; ++k) xin[k] = lds128(hi_a + (uint32_t)(k * 128 + st) * 16);
#pragma unroll
                for (int k = 0; k < BOX_BYTES / 16 / 128; ++k) {
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
        // ------------------------------ epilogue (warps 2..17) ------------------------------
        // Four groups of four warps (one warp per TMEM lane quarter).  Group g processes the panels
        // pn = g, g + 4, ... of every tile, so the panels of a tile are in flight concurrently and
        // their latency chains (panel wait, TMEM load, FP64 chains, store hand-off) overlap.
        // Thread = one row of the tile, all PW columns of the panel, 16 at a time.
        // Panel layout: PW = 32: 128-byte rows, 128-byte swizzle; PW = 16: plain 64-byte rows.
        const int q = warp & 3;                           // TMEM lane quarter of this warp
        const int grp = (warp - 2) >> 2;                  // epilogue group
        const int rl = q * 32 + lane;                     // row of the tile owned by this thread
        const int gt = (q * 32 + lane);                   // 0..127 inside the group
        int i = 0;
        for (int64_t t = blockIdx.x; t < n_tiles; t += gridDim.x, ++i) {
            const int a = i & 1;
            const int64_t row = t * TILE_M + rl;
            const bool valid = row < n;
            const float nay = valid ? -alpha * ybar[row] : 0.f;
            mbar_wait(accfull(a), (i >> 1) & 1, &abort_flag, ctl);
            tc_fence_after();
#pragma unroll 1
            for (int pn = grp; pn < NPAN; pn += NGROUPS) {
                // The ring of NUP slots is split among the groups: group grp owns slots grp, grp + NGROUPS, ... and
                // uses them in turn for its own panels (cnt = this group's panel count so far).  A slot therefore
                // always belongs to the same group, which sees every phase of its barrier; a wait names a phase
                // by its parity only, and a group that met a barrier still in another group's phase would read
                // that parity as "landed".
                const int depth = NUP / NGROUPS;
                const int cnt = i * ((NPAN - grp + NGROUPS - 1) / NGROUPS) + pn / NGROUPS;
                const int sl = grp + NGROUPS * (cnt % depth);
                const uint32_t pan = upan0 + (uint32_t)sl * PAN_BYTES;
                mbar_wait(ufull(sl), (cnt / depth) & 1, &abort_flag, ctl);
#pragma unroll 1
                for (int hf = 0; hf < PW / 16; ++hf) {
                    if (pn * PW + hf * 16 >= r) break;       // columns beyond r: nothing to compute, TMA clips the store
                    float acc[16], wn[16];
                    tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(a * ACC_COLS + pn * PW + hf * 16), acc);
                    // Statistics of these 16 entries in FP32 (w >= 0, u >= 0: no cancellation), folded into the
                    // FP64 running sums once per group: the FP32 -> FP64 conversion unit is the scarce resource.
                    float a32 = 0.f, b32 = 0.f, h32 = 0.f;
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        const int c = hf * 4 + cc;
                        const int col0 = pn * PW + 4 * c;
                        if (col0 >= r) {                     // r is a multiple of 4: the whole quad is beyond r
                            wn[4 * cc] = wn[4 * cc + 1] = wn[4 * cc + 2] = wn[4 * cc + 3] = 0.f;
                            continue;
                        }
                        const uint32_t addr = (PW == 32) ? pan + (uint32_t)rl * 128 + (uint32_t)((c ^ (rl & 7)) << 4)
                                                         : pan + (uint32_t)rl * 64 + (uint32_t)(c << 4);
                        const float4 w4 = lds128(addr);
                        const float4 p4 = *reinterpret_cast<const float4*>(sp + col0);
                        const float4 s4 = *reinterpret_cast<const float4*>(sas + col0);
                        const float wold[4] = {w4.x, w4.y, w4.z, w4.w};
                        const float pj[4] = {p4.x, p4.y, p4.z, p4.w};
                        const float sj[4] = {s4.x, s4.y, s4.z, s4.w};
                        const bool live = valid && (col0 < r);           // r is a multiple of 4
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float u = live ? cf * wold[e] : 0.f;
                            float v = fmaf(two_alpha, acc[4 * cc + e], u);
                            v = fmaf(nay, pj[e], v);
                            v -= sj[e];
                            const float w = live ? fmaxf(v, 0.f) : 0.f;
                            a32 = fmaf(w, w, a32);
                            b32 = fmaf(u, u, b32);
                            h32 = fmaf(w, u, h32);
                            wn[4 * cc + e] = w;
                        }
                        sts128(addr, make_float4(wn[4 * cc], wn[4 * cc + 1], wn[4 * cc + 2], wn[4 * cc + 3]));
                    }
                    sa += (double)a32;
                    sb += (double)b32;
                    sh += (double)h32;
                    // column sums over this warp's 32 rows (transpose-reduce), FP64 across tiles
                    const float cs = colsum16(wn, lane);
                    csum[(pn / NGROUPS) & 1][hf & 1] += (double)cs;
                }
                fence_proxy_async();
                named_bar_sync(1 + grp, GROUP_THREADS);
                if (gt == 0 && !abort_flag) {                // after a time-out the panel cannot be trusted: U is left as it is
                    tma_store_2d(&tmU, pn * PW, (int)(t * TILE_M), pan);
                    bulk_commit();
                }
                // the slot goes back to the producer as soon as the store has read it (every thread of the group
                // passed the barrier above after its last access)
                if (gt == 0) {
                    bulk_wait_read<0>();
                    mbar_arrive(ufree(sl));
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(accfree(a));
        }
        if (gt == 0) bulk_wait<0>();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, tmem_cols);

    // ---- CTA partial: a, b, h and the column sums of W ----
    const int PS = 4 + r;
    sa = block_sum<NTHREADS>(sa, sred);
    sb = block_sum<NTHREADS>(sb, sred);
    sh = block_sum<NTHREADS>(sh, sred);
    double* scol = reinterpret_cast<double*>(smem);        // [4 lane quarters][ACC_COLS]
    if (warp >= 2 && warp < 2 + 4 * NGROUPS && (lane & 1) == 0) {
        const int grp = (warp - 2) >> 2, q = warp & 3;
        const int ccol = ((lane >> 4) & 1) * 8 + ((lane >> 3) & 1) * 4 + ((lane >> 2) & 1) * 2 + ((lane >> 1) & 1);
        for (int pn = grp; pn < NPAN; pn += NGROUPS)
            for (int hf = 0; hf < PW / 16; ++hf)
                scol[(size_t)q * ACC_COLS + pn * PW + hf * 16 + ccol] = csum[(pn / NGROUPS) & 1][hf & 1];
    }
    __syncthreads();
    double* out = part + (size_t)blockIdx.x * PS;
    if (threadIdx.x == 0) { out[0] = sa; out[1] = sb; out[2] = sh; out[3] = 0.0; }
    for (int j = threadIdx.x; j < r; j += NTHREADS)
        out[4 + j] = ((scol[j] + scol[(size_t)ACC_COLS + j]) + scol[(size_t)2 * ACC_COLS + j]) + scol[(size_t)3 * ACC_COLS + j];
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

}  // namespace tc

bool tc_plan(const Problem& pb, TcPlan* pl, float* img_storage)
{
    const int d = pb.P.d, r = pb.P.r;
    if (d % 32 != 0 || r % 4 != 0 || r < 8 || r > 256 || pb.P.n < 1024 || pb.P.n > 2000000000ll) return false;
    const int NB = d / 32;
    const int NP = (r + 15) / 16 * 16;
    const int PW = (r <= 16) ? 16 : 32;
    const int NPAN = (r + PW - 1) / PW;
    if (NPAN > 8) return false;
    const int ACC_COLS = (NPAN * PW + 31) / 32 * 32;
    const size_t pan_bytes = (size_t)tc::TILE_M * PW * 4;
    // fp16 split on the static images of X-hat when the workspace holds them, else the TF32 split
    const bool f16 = pb.has_ximg();
    if (!f16 && d != pb.dx) return false;                     // the TF32 variant reads X-hat itself: no feature padding
    const size_t th = (size_t)NB * NP * (f16 ? 64 : 128);
    const size_t fixed = 2 * th + (size_t)2 * ACC_COLS * 4 + 1024;
    const size_t limit = 227 * 1024 - 2048;
    // Ring sizes under the 227 KB limit.  The U panel ring comes first (a group's slot is refilled only
    // after its store, so more slots let the next tile's panels load during this tile's epilogue); then the
    // lo boxes of the TF32 split (split -> MMA -> free round trip); the X-hat box ring takes what is left.
    int NSB = 0, NUP = 0, NLO = 0;
    if (f16) {
        for (int nup = 8; nup >= 4 && !NSB; nup -= 4)              // a multiple of the four epilogue groups
            for (int nsb = 6; nsb >= (nup == 4 ? 3 : 4); --nsb)
                if (fixed + (size_t)nsb * tc::BOX_BYTES + (size_t)nup * pan_bytes <= limit) { NSB = nsb; NUP = nup; break; }
    } else {
        for (int nup = 4; nup >= 4 && !NSB; nup -= 4)
            for (int nlo = 3; nlo >= 2 && !NSB; --nlo)
                for (int nsb = tc::MAX_RING; nsb >= (nlo == 3 ? 4 : 2); --nsb)
                    if (fixed + (size_t)(nsb + nlo) * tc::BOX_BYTES + (size_t)nup * pan_bytes <= limit) {
                        NSB = nsb; NUP = nup; NLO = nlo; break;
                    }
    }
    if (!NSB) return false;
    pl->f16 = f16;
    {
        int e;
        frexpf(sqrtf((float)pb.P.K), &e);                  // |Theta_jk| <= ||X-hat||_2 ||U||_F = sqrt(K) <= 2^e
        pl->eT = 14 - e;
    }
    pl->NP = NP; pl->PW = PW; pl->NSB = NSB; pl->NLO = NLO; pl->NUP = NUP;
    pl->smem2 = fixed + (size_t)(NSB + NLO) * tc::BOX_BYTES + (size_t)NUP * pan_bytes;
    pl->img_hi = img_storage;
    pl->img_lo = f16 ? reinterpret_cast<float*>(reinterpret_cast<uint16_t*>(img_storage) + (size_t)NB * 32 * NP)
                     : img_storage + (size_t)NB * 32 * NP;
    if (f16) {
        if (!make_tensor_map_2d_f16(&pl->tmX, pb.ximg(0), pb.P.n, d, pb.ximg_pitch(), tc::TILE_M, 32)) return false;
        if (!make_tensor_map_2d_f16(&pl->tmX2, pb.ximg(1), pb.P.n, d, pb.ximg_pitch(), tc::TILE_M, 32)) return false;
    } else {
        if (!make_tensor_map_2d(&pl->tmX, pb.X, pb.P.n, d, tc::TILE_M, 32)) return false;
        pl->tmX2 = pl->tmX;
    }
    if (!make_tensor_map_2d(&pl->tmU, pb.U, pb.P.n, r, tc::TILE_M, PW)) return false;
    const int64_t tiles = (pb.P.n + tc::TILE_M - 1) / tc::TILE_M;
    pl->g2 = (int)(tiles < kSMs ? tiles : kSMs);
    if (cudaFuncSetAttribute(tc::k_pass2_tc<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl->smem2) != cudaSuccess ||
        cudaFuncSetAttribute(tc::k_pass2_tc<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl->smem2) != cudaSuccess)
        return false;
    return true;
}

void tc_launch_second(const Problem& pb, const TcPlan& pl)
{
    const int d = pb.P.d, r = pb.P.r;
    const int total = d * pl.NP;
    if (pl.f16) {
        tc::k_theta_images_h<<<(total + 255) / 256, 256, 0, pb.stream>>>(pb.theta(), d, r, pl.NP, pl.eT, pb.ctl(),
                                                                         reinterpret_cast<__half*>(pl.img_hi),
                                                                         reinterpret_cast<__half*>(pl.img_lo));
        tc::k_pass2_tc<true><<<pl.g2, tc::NTHREADS, pl.smem2, pb.stream>>>(
            pl.tmX, pl.tmX2, pl.tmU, pl.eT, pb.U, pl.img_hi, pl.img_lo, pb.ybar(), pb.p(), pb.alpha_s(), pb.ctl(), pb.P.n, d,
            r, pl.NP, pl.PW, pl.NSB, pl.NLO, pl.NUP, pb.P.alpha, pb.P.K, pb.P.eps_d, pb.part2(), pb.p());
    } else {
        tc::k_theta_images<<<(total + 255) / 256, 256, 0, pb.stream>>>(pb.theta(), d, r, pl.NP, pb.ctl(), pl.img_hi, pl.img_lo);
        tc::k_pass2_tc<false><<<pl.g2, tc::NTHREADS, pl.smem2, pb.stream>>>(
            pl.tmX, pl.tmX2, pl.tmU, 0, pb.U, pl.img_hi, pl.img_lo, pb.ybar(), pb.p(), pb.alpha_s(), pb.ctl(), pb.P.n, d, r,
            pl.NP, pl.PW, pl.NSB, pl.NLO, pl.NUP, pb.P.alpha, pb.P.K, pb.P.eps_d, pb.part2(), pb.p());
    }
    pb.count(2);
}

}  // namespace gemnlr
