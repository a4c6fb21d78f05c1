// C ABI of the NLR iteration library: argument checks, workspace layout, the host control loop.
// Every arithmetic step of the method runs in the kernels; this file only orders launches and
// reads back the small control block.
#include "nlr_common.cuh"
#include "ffma_family.cuh"
#include "tc_family.cuh"
#include <math.h>
#include <stdio.h>
#include <string.h>
#include <new>

namespace gemnlr {

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
static int clampi(int64_t v, int64_t lo, int64_t hi) { return (int)(v < lo ? lo : (v > hi ? hi : v)); }

static bool valid_params(const gem_nlr_params& P)
{
    if (P.n < 1 || P.d < 1 || P.K < 1 || P.r < P.K) return false;
    if (P.r > 7168 || P.d > 2816) return false;       // shared-memory accumulators of the vector / setup passes
    if (!(P.alpha > 0.f) || !(P.beta > 0.f)) return false;
    if (P.T < 0 || P.T_min < 0 || P.eps_d < 0.0 || P.eps_c < 0.0) return false;
    if (P.precision < -1 || P.precision > 3) return false;
    if (P.x_inplace < 0 || P.x_inplace > 2) return false;
    return true;
}

Layout make_layout(const gem_nlr_params& P)
{
    Layout L;
    memset(&L, 0, sizeof(L));
    const int64_t n = P.n;
    const int d = P.d, r = P.r;
    L.g1y_d = (int)ceil_div(d, G_DT);
    L.g1y_r = (int)ceil_div(r, G_RT);
    const int tiles1 = L.g1y_d * L.g1y_r;
    L.g1x = clampi(ceil_div(kSMs * 4, tiles1), 1, ceil_div(n, G_TM));
    L.gv = clampi(ceil_div(n, 4), 1, kSMs * 8);
    L.g2y = (int)ceil_div(r, G2_RT);
    L.g2x = clampi(ceil_div(kSMs * 4, L.g2y), 1, ceil_div(n, G2_TM));
    L.gs = clampi(ceil_div(n, 8), 1, kSMs * 4);
    // tcgen05 shapes: X-hat is static, so its two-term fp16 split is built once (below).  Those kernels see the
    // feature count rounded up to a multiple of 32 (zero features in the images), so Theta, its partial records
    // and the reduction are sized for dp x r.
    const bool tc_images = (P.precision == -1 || P.precision == 1) && r >= 32 && n >= 4096;
    int dp = tc_images ? (d + 31) / 32 * 32 : d;
    // Wide factors (r > 128) have no resident-Theta first product; the tiled one works on 256-feature blocks.  For
    // 128 < d < 256 (the paper's d = 200 with r = 150 .. 300) the images are padded to 256 features: at most twice
    // the tensor-core work, against a first product on the FFMA fallback otherwise.
    // The same padding serves r <= 128 when d r is beyond what the resident-Theta first product takes (d r <= 16384): the
    // pair of tiled kernels then replaces a first product on the FFMA fallback.
    // Wide factors with fewer features (64 <= d <= 128) are padded as well: up to four times the tensor-core work and
    // image bytes of the first product, which is still several times faster than the fallback (d = 128, r = 300:
    // 11.6 ms on the FFMA kernels).
    if (tc_images && dp < 256 && ((r > 128 && dp >= 64) || (dp > 128 && (size_t)dp * r > 16384))) dp = 256;
    L.dp = dp;
    L.has_img = tc_images ? 1 : 0;
    // x_inplace == 2: X-hat itself may be given up after setup.  Where both products read only the fp16 images (the
    // shapes below: the resident-Theta pair and the tiled pair) the row-major image pair takes X-hat's place, which
    // has exactly its size when d needs no padding.  The rule is deliberately narrower than the kernels' own shape
    // tests; gem_nlr_create checks it against the kernels actually chosen.
    const bool pair_small = d % 32 == 0 && d >= 32 && d <= 256 && r % 4 == 0 && r <= 128 && (size_t)d * r <= 16384;
    const bool pair_tiled = d % 32 == 0 && d >= 256 && d <= 1536 && r % 4 == 0 && r > 256 && r <= 1536 &&
                            ((r + 127) / 128) * ((d + 255) / 256) <= kSMs;
    L.img_inplace = (P.x_inplace == 2 && tc_images && (pair_small || pair_tiled)) ? 1 : 0;
    L.nred1 = (int)ceil_div((int64_t)dp * r, 64);

    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    L.ctl = take(1024);
    L.p = take(sizeof(float) * r);
    L.s = take(sizeof(float) * r);
    L.alpha_s = take(sizeof(float) * r);
    L.theta = take(sizeof(float) * (size_t)dp * r);
    // Theta^T operand images: the resident-Theta kernels keep 2 x dp x pad16(r) floats (TF32 split) or halves; the tiled
    // kernel 2 x dp x pad256(r) halves, also for r <= 256 when the resident form does not fit in shared memory
    {
        const size_t d32 = (size_t)((dp + 31) / 32 * 32);
        size_t cols = r > 256 ? (size_t)((r + 255) / 256 * 256) : (size_t)((r + 15) / 16 * 16);
        if (tc_images && cols < 128) cols = 128;
        L.thimg = take(sizeof(float) * 2 * d32 * cols);
    }
    L.ytilde = take(sizeof(float) * (size_t)n);
    L.ybar = take(sizeof(float) * (size_t)n);
    // partial areas are sized for the largest user among the kernel families
    int p1_records = L.g1x;
    if (tc_images && p1_records < 8) p1_records = 8;
    if (tc_images && dp >= 256 && tiled_first_row_ranges(n, dp, r) > p1_records)
        p1_records = tiled_first_row_ranges(n, dp, r);           // the tiled tcgen05 first product: one record per row range
    size_t p1 = sizeof(double) * (size_t)p1_records * dp * r;
    size_t p1_fast = ((size_t)dp * r <= 16384) ? sizeof(double) * (size_t)kSMs * 2 * ((size_t)dp * r + r + 4) : 0;
    if (r <= d && p1 < sizeof(double) * 8 * (size_t)d * d) p1 = sizeof(double) * 8 * (size_t)d * d;   // X-hat^T X-hat of the data-informed start: up to 8 row chunks
    L.part1_bytes = p1 > p1_fast ? p1 : p1_fast;
    L.part1 = take(L.part1_bytes);
    L.part1v = take(sizeof(double) * (size_t)L.gv * (r + 2));
    size_t p2 = sizeof(double) * (size_t)L.g2x * L.g2y * (3 + G2_RT);
    size_t p2_fast = sizeof(double) * (size_t)kSMs * 4 * (4 + (size_t)r);
    const size_t p2_tiled = sizeof(double) * (size_t)kSMs * (4 + 256);      // tiled tcgen05 second product: one 256-column block per CTA
    if (p2_fast < p2_tiled) p2_fast = p2_tiled;
    L.part2 = take(p2 > p2_fast ? p2 : p2_fast);
    // generic family: nred1 block shares; fused reduction: one share per 16 entries of a record + r + 2 sums
    L.red1 = take(sizeof(double) * ((size_t)L.nred1 + ((size_t)dp * r + r + 2 + 15) / 16 + r + 2 + 8));
    L.setup = take(sizeof(double) * (3 * (size_t)d + 4 + (size_t)L.gs * d));
    L.init = take(r <= d ? sizeof(double) * ((size_t)d * d + 2 * (size_t)d * r + (size_t)r * r) : 0);
    L.hist = take(P.history ? sizeof(gem_nlr_iter_info) * (size_t)(P.T > 0 ? P.T : 1) : 0);
    L.xhat = take(P.x_inplace ? 0 : sizeof(float) * (size_t)n * d);
    // tcgen05 shapes: X-hat is static, so its two-term fp16 split is built once, row-major (second product)
    // and transposed in blocks of fb features x 32 rows (first product): about 2 x 2 x n x d halves.
    L.n_pad = (n + 63) / 64 * 64;
    L.fb = dp >= 256 ? 256 : dp;
    L.ximg = take(tc_images && !L.img_inplace ? sizeof(uint16_t) * 2 * (size_t)n * dp : 0);
    L.ximgT = take(tc_images ? sizeof(uint16_t) * 2 * (size_t)(L.n_pad / 32) * ((dp + L.fb - 1) / L.fb) * L.fb * 32 : 0);
    L.total = off;
    return L;
}

}  // namespace gemnlr

using namespace gemnlr;

struct gem_nlr {
    Problem pb;
    Problem pbp;           // the view of pb for the fp16-image tensor-core kernels: P.d = L.dp
    float* X_in;
    bool normalized;
    bool loaded;           // p = U^T 1 is on the device for the current U
    double a;
    int32_t t_host;        // iterations completed as of the last read-back
    int32_t sticky_error;
    Ctl* host_ctl;         // pinned read-back record
    double* host_scratch;  // pinned
    const char* path;
    bool use_ffma;         // first (and, unless use_tc, second) product by the FFMA family
    bool use_mma;          // with use_ffma: the warp-level TF32 tensor-core kernels of that family
    bool use_tc;           // second product by the tcgen05 family
    bool use_tc1;          // first product by the tcgen05 family
    bool use_tcg;          // second product by the tiled tcgen05 kernel (wide d, r)
    FfmaPlan ffma;
    TcPlan tc;
    Tc1Plan tc1;
    TcgPlan tcg;
    Tcg1Plan tcg1;
    bool use_tcg1;         // first product by the tiled tcgen05 kernel (vector pass separate)
    bool x_consumed;       // x_inplace == 2 in effect: after setup the X buffer holds the row-major fp16 images, not X-hat
    ShardInfo shard;       // row-sharded run: rank, world, callbacks (world <= 1: single GPU)
    char err[256];
    int64_t launches;      // kernels launched by this handle
    int pi_iters;          // power iterations taken by the last setup
    // optional per-phase timing: events recorded around the two passes of every iteration
    bool profile;
    cudaEvent_t* ev;       // 3 per iteration: start, after the first-product phase, after the second product
    int ev_cap, ev_used;
    double prof_ms[3];     // accumulated: first-product phase, second-product kernel, (unused)
    int64_t prof_iters;
};

static int cuda_fail(gem_nlr_t* h, cudaError_t e, const char* where)
{
    snprintf(h->err, sizeof(h->err), "%s: %s", where, cudaGetErrorString(e));
    h->sticky_error = GEM_NLR_E_CUDA;
    return GEM_NLR_E_CUDA;
}

#define CK(h, call)                                                   \
    do {                                                              \
        cudaError_t e__ = (call);                                     \
        if (e__ != cudaSuccess) return cuda_fail((h), e__, #call);    \
    } while (0)

static int reset_ctl(gem_nlr_t* h, int32_t t)
{
    Ctl c;
    memset(&c, 0, sizeof(c));
    c.c_f = 1.0f;
    c.t = t;
    c.hist_cap = h->pb.P.history ? (h->pb.P.T > 0 ? h->pb.P.T : 1) : 0;
    c.shard_world = h->shard.world;
    *h->host_ctl = c;
    CK(h, cudaMemcpyAsync(h->pb.ctl(), h->host_ctl, sizeof(Ctl), cudaMemcpyHostToDevice, h->pb.stream));
    CK(h, cudaStreamSynchronize(h->pb.stream));   // host_ctl is reused for read-backs
    h->t_host = t;
    h->loaded = false;
    return GEM_NLR_OK;
}

static int read_ctl(gem_nlr_t* h)
{
    CK(h, cudaMemcpyAsync(h->host_ctl, h->pb.ctl(), sizeof(Ctl), cudaMemcpyDeviceToHost, h->pb.stream));
    CK(h, cudaStreamSynchronize(h->pb.stream));
    CK(h, cudaGetLastError());
    h->t_host = h->host_ctl->t;
    return GEM_NLR_OK;
}

static int ensure_loaded(gem_nlr_t* h)
{
    if (!h->loaded) {
        launch_init_colsum(h->pb);
        if (h->pb.shard) {
            const int rc = shard_exchange_second(h->pb, 1);
            if (rc) return rc;
        }
        h->loaded = true;
    }
    return GEM_NLR_OK;
}

// One iteration = vector pass + first product (+ reductions), then the fused second product
// and its scalar reduction.  With profiling on, events bracket the two phases.
static int launch_iteration(gem_nlr_t* h)
{
    const bool sharded = h->pb.shard != nullptr;
    int xrc = GEM_NLR_OK;
    const bool prof = h->profile && h->ev_used + 3 <= h->ev_cap;
    cudaEvent_t* e = prof ? h->ev + h->ev_used : nullptr;
    if (prof) cudaEventRecord(e[0], h->pb.stream);
    if (h->use_tc1) {
        tc1_launch_first(h->pbp, h->tc1);
        red1_fused_launch(h->pbp, h->tc1.grid, 0);
    } else if (h->use_ffma) {
        if (h->use_mma) mma_launch_first(h->pb, h->ffma, 0);
        else ffma_launch_first(h->pb, h->ffma, 0);
    } else {
        launch_vector_pass(h->pb);
        if (h->use_tcg1) tcg_launch_first(h->pbp, h->tcg1);
        else launch_generic_pass1(h->pb, 0);
        launch_fin1(h->pb, 0);
    }
    // row-sharded: the kernels above parked this rank's sums; combine all ranks' and take the scalar step
    if (sharded) xrc = shard_exchange_first((h->use_tc1 || h->use_tcg1 || h->use_tc || h->use_tcg) ? h->pbp : h->pb, 0);
    if (xrc) return xrc;
    if (prof) cudaEventRecord(e[1], h->pb.stream);
    if (h->use_tc || h->use_ffma || h->use_tcg) {
        if (h->use_tcg) tcg_launch_second(h->pbp, h->tcg);
        else if (h->use_tc) tc_launch_second(h->pbp, h->tc);
        else if (h->use_mma) mma_launch_second(h->pb, h->ffma);
        else ffma_launch_second(h->pb, h->ffma);
        if (sharded) xrc = shard_exchange_second(h->pb, 0);
        if (prof) { cudaEventRecord(e[2], h->pb.stream); h->ev_used += 3; }
        return xrc;
    }
    launch_generic_pass2_kernel(h->pb);
    if (prof) { cudaEventRecord(e[2], h->pb.stream); h->ev_used += 3; }
    launch_fin2(h->pb, h->pb.L.g2x, h->pb.L.g2y, G2_RT);
    if (sharded) xrc = shard_exchange_second(h->pb, 0);
    return xrc;
}

// Finishes the last iteration (dual step, rho, stop test) and writes the pending multiplier into U.
static int launch_tail_any(gem_nlr_t* h)
{
    launch_tail(h->pb);
    if (h->pb.shard) return shard_exchange_first(h->pb, 1);
    return GEM_NLR_OK;
}

static void drain_profile(gem_nlr_t* h)
{
    for (int i = 0; i + 2 < h->ev_used; i += 3) {
        float a = 0.f, b = 0.f;
        if (cudaEventElapsedTime(&a, h->ev[i], h->ev[i + 1]) == cudaSuccess &&
            cudaEventElapsedTime(&b, h->ev[i + 1], h->ev[i + 2]) == cudaSuccess) {
            h->prof_ms[0] += a;
            h->prof_ms[1] += b;
            h->prof_iters += 1;
        }
    }
    h->ev_used = 0;
}

static int clear_stop(gem_nlr_t* h)
{
    // a previous "converged" stop does not forbid further iterations; errors are sticky
    CK(h, cudaMemsetAsync(&h->pb.ctl()->stopped, 0, 2 * sizeof(int32_t), h->pb.stream));
    return GEM_NLR_OK;
}

extern "C" {

size_t gem_nlr_workspace_bytes(const gem_nlr_params* params)
{
    if (!params || !valid_params(*params)) return 0;
    return make_layout(*params).total;
}

size_t gem_nlr_paper_storage_bytes(const gem_nlr_params* params)
{
    if (!params || !valid_params(*params)) return 0;
    const size_t n = (size_t)params->n, d = (size_t)params->d, r = (size_t)params->r;
    const size_t n_tile = ((n + 127) / 128) * ((r + 63) / 64);
    return 4 * (n * d + n * r + d * r + 4 * n + 2 * r) + 24 * (n_tile + 1);
}

int gem_nlr_create(gem_nlr_t** out, const gem_nlr_params* params, float* X_dev, float* U_dev,
                   void* workspace_dev, size_t workspace_bytes, void* cuda_stream)
{
    if (!out) return GEM_NLR_E_INVALID;
    *out = nullptr;
    if (!params || !X_dev || !U_dev || !workspace_dev) return GEM_NLR_E_INVALID;
    if (!valid_params(*params)) return GEM_NLR_E_INVALID;
    if (((uintptr_t)X_dev & 15) || ((uintptr_t)U_dev & 15) || ((uintptr_t)workspace_dev & 255))
        return GEM_NLR_E_INVALID;
    Layout L = make_layout(*params);
    if (workspace_bytes < L.total) return GEM_NLR_E_WORKSPACE;
    gem_nlr_t* h = new (std::nothrow) gem_nlr_t;
    if (!h) return GEM_NLR_E_INVALID;
    memset(h, 0, sizeof(*h));
    h->pb.P = *params;
    h->pb.L = L;
    h->pb.ws = (char*)workspace_dev;
    h->pb.U = U_dev;
    h->X_in = X_dev;
    h->pb.X = params->x_inplace ? X_dev : (float*)((char*)workspace_dev + L.xhat);
    h->pb.stream = (cudaStream_t)cuda_stream;
    h->pb.gamma = (double)params->beta / (double)params->n;
    h->pb.gamma_f = (float)h->pb.gamma;
    h->path = "generic";
    h->err[0] = 0;
    h->pb.launches = &h->launches;
    h->pb.dx = params->d;
    h->pbp = h->pb;
    h->pbp.P.d = L.dp;
    // Kernel families by shape.  precision 3: the warp-level TF32 (mma.sync, 3-product split) kernels
    // where instantiated, else generic; precision -1 prefers them to the FFMA kernels for d >= 64.
    // precision 2: generic only.  precision 0: FFMA family where a shape is
    // instantiated, else generic.  precision 1: tensor cores wherever they are available.  precision -1:
    // FFMA for the skinny shapes (r <= 16: there the FP32 pipes keep up and the tensor-core path would
    // issue one MMA triple per 8 rows for 16 useful columns), tensor cores for r >= 32, else generic.
    const bool want_ffma = params->precision != 2;
    const bool want_mma = params->precision == 3 || params->precision == -1;
    const bool want_tc = params->precision == 1 || (params->precision == -1 && params->r >= 32);
    // the wide-factor mma.sync shapes (r > 16) are slower than the tcgen05 pair: explicit request only
    if (want_mma && (params->precision == 3 || params->r <= 16) && mma_plan(h->pb, &h->ffma)) {
        h->use_ffma = h->use_mma = true;
        h->path = "mma.tf32x3";
    } else if (want_ffma && params->precision != 3 && ffma_plan(h->pb, &h->ffma)) {
        h->use_ffma = true;
        h->path = "ffma";
    }
    if (want_tc && !(params->precision == -1 && h->use_ffma)) {
        float* img = reinterpret_cast<float*>((char*)workspace_dev + L.thimg);
        if (tc_plan(h->pbp, &h->tc, img)) {
            h->use_tc = true;
            h->path = h->use_ffma ? (h->tc.f16 ? "ffma+f16x3" : "ffma+tf32x3") : (h->tc.f16 ? "generic+f16x3" : "generic+tf32x3");
            if (tc1_plan(h->pbp, &h->tc1)) {
                h->use_tc1 = true;
                // first product on the fp16 split; second on the fp16 split when the static images of X-hat
                // are in the workspace, else on the TF32 split
                h->path = h->tc.f16 ? "f16x3" : "f16x3+tf32x3";
            }
        }
        else if (tcg_plan(h->pbp, &h->tcg, img)) {
            h->use_tcg = true;
            h->path = "generic+f16x3.tiled";
            if (tcg1_plan(h->pbp, &h->tcg1)) {
                h->use_tcg1 = true;
                h->path = "f16x3.tiled";
            }
        }
    }
    if (L.img_inplace) {
        const bool both = (h->use_tc1 && h->use_tc && h->tc.f16) || (h->use_tcg1 && h->use_tcg);
        if (both) {
            h->x_consumed = true;
        } else {
            // the kernels chosen for this shape still read X-hat: keep it, build no images, iterate on the
            // general-shape kernels (correct for every shape; the layout holds no room for separate images)
            h->use_tc = h->use_tc1 = h->use_tcg = h->use_tcg1 = false;
            h->pb.L.has_img = h->pbp.L.has_img = 0;
            h->pb.L.img_inplace = h->pbp.L.img_inplace = 0;
            h->path = h->use_mma ? "mma.tf32x3" : h->use_ffma ? "ffma" : "generic";
        }
    }
    if (cudaMallocHost((void**)&h->host_ctl, sizeof(Ctl)) != cudaSuccess ||
        cudaMallocHost((void**)&h->host_scratch, 64) != cudaSuccess) {
        if (h->host_ctl) cudaFreeHost(h->host_ctl);
        delete h;
        return GEM_NLR_E_CUDA;
    }
    int rc = reset_ctl(h, 0);
    if (rc == GEM_NLR_OK &&
        cudaMemsetAsync(h->pb.ytilde(), 0, sizeof(float) * (size_t)params->n, h->pb.stream) != cudaSuccess)
        rc = GEM_NLR_E_CUDA;
    // the padding rows of Theta (features d .. dp - 1) are written only by the image kernels' own reduction
    if (rc == GEM_NLR_OK &&
        cudaMemsetAsync(h->pb.theta(), 0, sizeof(float) * (size_t)L.dp * params->r, h->pb.stream) != cudaSuccess)
        rc = GEM_NLR_E_CUDA;
    if (rc != GEM_NLR_OK) {
        cudaFreeHost(h->host_ctl);
        cudaFreeHost(h->host_scratch);
        delete h;
        return rc;
    }
    *out = h;
    return GEM_NLR_OK;
}

int gem_nlr_spectral_norm(gem_nlr_t* h, double* a_out)
{
    if (!h) return GEM_NLR_E_INVALID;
    if (h->sticky_error) return h->sticky_error;
    if (h->normalized) return GEM_NLR_E_INVALID;     // X_dev already holds X-hat
    double a = 0.0;
    int rc = run_spectral_norm(h->pb, h->X_in, h->pb.X, &a, h->host_scratch);
    if (rc != GEM_NLR_OK) {
        if (rc == GEM_NLR_E_CUDA) return cuda_fail(h, cudaGetLastError(), "spectral_norm");
        return rc;
    }
    CK(h, cudaStreamSynchronize(h->pb.stream));
    h->a = a;
    h->normalized = true;
    if (h->pb.has_ximg() && (h->use_tcg || h->use_tc)) {  // static fp16 images of X-hat for the tensor-core kernels
        tcg_prepare(h->pbp);
        CK(h, cudaStreamSynchronize(h->pb.stream));
    }
    if (a_out) *a_out = a;
    return GEM_NLR_OK;
}

int gem_nlr_set_normalized(gem_nlr_t* h, double a)
{
    if (!h) return GEM_NLR_E_INVALID;
    if (!h->pb.P.x_inplace) return GEM_NLR_E_INVALID;  // X-hat must be in the caller's buffer
    h->a = a;
    h->normalized = true;
    if (h->pb.has_ximg() && (h->use_tcg || h->use_tc)) {
        tcg_prepare(h->pbp);
        CK(h, cudaStreamSynchronize(h->pb.stream));
    }
    return GEM_NLR_OK;
}

static int result_code(gem_nlr_t* h, bool capped)
{
    const Ctl& c = *h->host_ctl;
    if (c.status < 0) { h->sticky_error = c.status; return c.status; }
    if (c.last.stop) return GEM_NLR_CONVERGED;
    return capped ? GEM_NLR_ITER_CAP : GEM_NLR_OK;
}

size_t gem_nlr_shard_exchange_bytes(const gem_nlr_params* params, int32_t world)
{
    if (!params || !valid_params(*params) || world < 1) return 0;
    const Layout L = make_layout(*params);
    return sizeof(double) * shard_record_doubles(*params, L.dp) * (size_t)(world + 1);
}

int gem_nlr_shard_attach(gem_nlr_t* h, int32_t rank, int32_t world, int64_t n_global, gem_nlr_gather_fn gather,
                         gem_nlr_host_sum_fn host_sum, void* ctx, void* exchange_dev, size_t exchange_bytes)
{
    if (!h || world < 1 || rank < 0 || rank >= world || n_global < h->pb.P.n || !gather || !host_sum || !exchange_dev)
        return GEM_NLR_E_INVALID;
    if (((uintptr_t)exchange_dev & 255) || h->normalized || h->t_host != 0) return GEM_NLR_E_INVALID;
    if (exchange_bytes < gem_nlr_shard_exchange_bytes(&h->pb.P, world)) return GEM_NLR_E_WORKSPACE;
    h->shard.rank = rank;
    h->shard.world = world;
    h->shard.n_global = n_global;
    h->shard.gather = gather;
    h->shard.host_sum = host_sum;
    h->shard.ctx = ctx;
    h->shard.xbuf = reinterpret_cast<double*>(exchange_dev);
    h->shard.xcount = shard_record_doubles(h->pb.P, h->pb.L.dp);
    // the penalty weight and rho refer to all rows
    h->pb.gamma = (double)h->pb.P.beta / (double)n_global;
    h->pb.gamma_f = (float)h->pb.gamma;
    h->pbp.gamma = h->pb.gamma;
    h->pbp.gamma_f = h->pb.gamma_f;
    if (world == 1) {                                         // one rank: nothing to exchange, the single-GPU path as it is
        h->shard.world = 0;
        return GEM_NLR_OK;
    }
    h->pb.shard = &h->shard;
    h->pbp.shard = &h->shard;
    return reset_ctl(h, 0);                                   // the control block now says "sharded"
}

int gem_nlr_init_range(gem_nlr_t* h)
{
    if (!h) return GEM_NLR_E_INVALID;
    if (h->sticky_error) return h->sticky_error;
    if (!h->normalized) return GEM_NLR_E_NOT_READY;
    if (h->pb.shard) return GEM_NLR_E_INVALID;                // single-GPU call
    if (h->x_consumed) return GEM_NLR_E_INVALID;              // X-hat itself was given up (x_inplace == 2)
    if (h->pb.P.r > h->pb.P.d) return GEM_NLR_E_INVALID;      // the sample X-hat X-hat^T Z has rank <= d
    int rc = reset_ctl(h, 0);                                 // multiplier 1, no gate pending, not stopped
    if (rc) return rc;
    if (!launch_range_init(h->pb)) return GEM_NLR_E_WORKSPACE;
    launch_tail(h->pb);                                       // U0 = c [Q]_+ written out
    rc = read_ctl(h);
    if (rc) return rc;
    const int status = h->host_ctl->status;
    // the starting factor is in place: y = 0, iteration counter 0, no record of an iteration
    CK(h, cudaMemsetAsync(h->pb.ytilde(), 0, sizeof(float) * (size_t)h->pb.P.n, h->pb.stream));
    rc = reset_ctl(h, 0);
    if (rc) return rc;
    return status < 0 ? status : GEM_NLR_OK;
}

int gem_nlr_step(gem_nlr_t* h, gem_nlr_iter_info* info)
{
    if (!h) return GEM_NLR_E_INVALID;
    if (h->sticky_error) return h->sticky_error;
    if (!h->normalized) return GEM_NLR_E_NOT_READY;
    int rc = clear_stop(h);
    if (rc) return rc;
    rc = ensure_loaded(h);
    if (rc == GEM_NLR_OK) rc = launch_iteration(h);
    if (rc == GEM_NLR_OK) rc = launch_tail_any(h);
    if (rc) return rc;
    rc = read_ctl(h);
    if (rc) return rc;
    if (info) *info = h->host_ctl->last;
    return result_code(h, false);
}

int gem_nlr_run(gem_nlr_t* h, gem_nlr_iter_info* last, int32_t* iters_done)
{
    if (!h) return GEM_NLR_E_INVALID;
    if (h->sticky_error) return h->sticky_error;
    if (!h->normalized) return GEM_NLR_E_NOT_READY;
    int rc = clear_stop(h);
    if (rc) return rc;
    rc = ensure_loaded(h);
    if (rc) return rc;
    const int32_t T = h->pb.P.T, T_min = h->pb.P.T_min;
    const int32_t t0 = h->t_host;
    int since_check = 0;
    for (int32_t t = t0; t < T; ++t) {
        rc = launch_iteration(h);
        if (rc) return rc;
        ++since_check;
        // The stop test of iteration t is evaluated by the first kernels of iteration t + 1, so a
        // flag seen here is at most one iteration old; kernels launched after a stop return at once.
        if (t + 1 >= T_min && since_check >= 16 && t + 1 < T) {
            rc = read_ctl(h);
            if (rc) return rc;
            if (h->profile) drain_profile(h);
            since_check = 0;
            if (h->host_ctl->stopped) break;
        }
    }
    rc = launch_tail_any(h);
    if (rc) return rc;
    rc = read_ctl(h);
    if (rc) return rc;
    if (h->profile) drain_profile(h);
    if (last) *last = h->host_ctl->last;
    if (iters_done) *iters_done = h->host_ctl->t;
    return result_code(h, true);
}

int gem_nlr_labels(gem_nlr_t* h, int32_t* labels_dev)
{
    if (!h || !labels_dev) return GEM_NLR_E_INVALID;
    launch_labels(h->pb, labels_dev);
    CK(h, cudaGetLastError());
    return GEM_NLR_OK;
}

size_t gem_nlr_labels_spectral_scratch_bytes(const gem_nlr_params* params)
{
    if (!params || !valid_params(*params)) return 0;
    return readout_scratch_bytes(*params);
}

int gem_nlr_labels_spectral(gem_nlr_t* h, int32_t* labels_dev, void* scratch_dev, size_t scratch_bytes,
                            int32_t max_iter, int32_t* passes_out)
{
    if (!h || !labels_dev || !scratch_dev || max_iter < 1) return GEM_NLR_E_INVALID;
    if (((uintptr_t)scratch_dev & 255) != 0) return GEM_NLR_E_INVALID;
    if (scratch_bytes < readout_scratch_bytes(h->pb.P)) return GEM_NLR_E_WORKSPACE;
    if (h->pb.P.r > 2048) return GEM_NLR_E_INVALID;          // one-CTA eigen-decomposition of the r x r Gram matrix
    if (h->pb.shard) return GEM_NLR_E_INVALID;               // single-GPU call
    int rc = run_spectral_labels(h->pb, labels_dev, (char*)scratch_dev, max_iter, passes_out,
                                 reinterpret_cast<unsigned long long*>(h->host_scratch));
    if (rc == GEM_NLR_E_CUDA) return cuda_fail(h, cudaGetLastError(), "labels_spectral");
    return rc;
}

int gem_nlr_objective(gem_nlr_t* h, double* fhat_out)
{
    if (!h || !fhat_out) return GEM_NLR_E_INVALID;
    if (!h->normalized) return GEM_NLR_E_NOT_READY;
    if (h->x_consumed) return GEM_NLR_E_INVALID;              // the stand-alone evaluation reads X-hat itself
    int rc = ensure_loaded(h);
    if (rc) return rc;
    launch_objective(h->pb);
    if (h->pb.shard) {
        rc = shard_exchange_first(h->pb, 2);
        if (rc) return rc;
    }
    rc = read_ctl(h);
    if (rc) return rc;
    *fhat_out = h->host_ctl->f_final;
    return GEM_NLR_OK;
}

int gem_nlr_get_state(gem_nlr_t* h, float* ytilde_dev, int32_t* t_out)
{
    if (!h) return GEM_NLR_E_INVALID;
    if (ytilde_dev)
        CK(h, cudaMemcpyAsync(ytilde_dev, h->pb.ytilde(), sizeof(float) * (size_t)h->pb.P.n,
                              cudaMemcpyDeviceToDevice, h->pb.stream));
    CK(h, cudaStreamSynchronize(h->pb.stream));
    if (t_out) *t_out = h->t_host;
    return GEM_NLR_OK;
}

int gem_nlr_set_state(gem_nlr_t* h, const float* ytilde_dev, int32_t t)
{
    if (!h || t < 0) return GEM_NLR_E_INVALID;
    if (ytilde_dev)
        CK(h, cudaMemcpyAsync(h->pb.ytilde(), ytilde_dev, sizeof(float) * (size_t)h->pb.P.n,
                              cudaMemcpyDeviceToDevice, h->pb.stream));
    else
        CK(h, cudaMemsetAsync(h->pb.ytilde(), 0, sizeof(float) * (size_t)h->pb.P.n, h->pb.stream));
    h->sticky_error = 0;
    return reset_ctl(h, t);
}

int gem_nlr_history(gem_nlr_t* h, gem_nlr_iter_info* records_host, int32_t max_records)
{
    if (!h || !records_host || max_records < 0) return GEM_NLR_E_INVALID;
    if (!h->pb.P.history) return GEM_NLR_E_INVALID;
    int rc = read_ctl(h);
    if (rc) return rc;
    int n = h->host_ctl->hist_len < max_records ? h->host_ctl->hist_len : max_records;
    if (n > 0) CK(h, cudaMemcpy(records_host, h->pb.hist(), sizeof(gem_nlr_iter_info) * (size_t)n,
                                cudaMemcpyDeviceToHost));
    return n;
}

int gem_nlr_buffer(gem_nlr_t* h, int32_t which, void** ptr_dev)
{
    if (!h || !ptr_dev) return GEM_NLR_E_INVALID;
    switch (which) {
        case 0: *ptr_dev = h->pb.theta(); break;
        case 1: *ptr_dev = h->pb.p(); break;
        case 2: *ptr_dev = h->pb.s(); break;
        case 3: *ptr_dev = h->pb.ytilde(); break;
        case 4: *ptr_dev = h->pb.ybar(); break;
        case 5:
            if (h->x_consumed && h->normalized) return GEM_NLR_E_INVALID;
            *ptr_dev = h->pb.X;
            break;
        default: return GEM_NLR_E_INVALID;
    }
    return GEM_NLR_OK;
}

const char* gem_nlr_path(gem_nlr_t* h) { return h ? h->path : ""; }

const char* gem_nlr_last_error(gem_nlr_t* h) { return h ? h->err : ""; }

int gem_nlr_destroy(gem_nlr_t* h)
{
    if (!h) return GEM_NLR_E_INVALID;
    cudaStreamSynchronize(h->pb.stream);
    if (h->host_ctl) cudaFreeHost(h->host_ctl);
    if (h->host_scratch) cudaFreeHost(h->host_scratch);
    if (h->ev) {
        for (int i = 0; i < h->ev_cap; ++i) cudaEventDestroy(h->ev[i]);
        delete[] h->ev;
    }
    delete h;
    return GEM_NLR_OK;
}

int gem_nlr_profile(gem_nlr_t* h, int32_t enable)
{
    if (!h) return GEM_NLR_E_INVALID;
    if (enable && !h->ev) {
        h->ev_cap = 3 * 1024;
        h->ev = new (std::nothrow) cudaEvent_t[h->ev_cap];
        if (!h->ev) return GEM_NLR_E_INVALID;
        for (int i = 0; i < h->ev_cap; ++i) CK(h, cudaEventCreate(&h->ev[i]));
    }
    h->profile = enable != 0;
    h->ev_used = 0;
    h->prof_ms[0] = h->prof_ms[1] = h->prof_ms[2] = 0.0;
    h->prof_iters = 0;
    return GEM_NLR_OK;
}

int gem_nlr_profile_read(gem_nlr_t* h, double* ms_first_phase, double* ms_second_product,
                         int64_t* iterations)
{
    if (!h) return GEM_NLR_E_INVALID;
    if (ms_first_phase) *ms_first_phase = h->prof_ms[0];
    if (ms_second_product) *ms_second_product = h->prof_ms[1];
    if (iterations) *iterations = h->prof_iters;
    return GEM_NLR_OK;
}

int64_t gem_nlr_launch_count(gem_nlr_t* h) { return h ? h->launches : 0; }

int gem_nlr_selftest_wait_timeout(gem_nlr_t* h, uint32_t max_polls, int64_t* cycles_out)
{
    if (!h || max_polls < 1 || max_polls > (1u << 20)) return GEM_NLR_E_INVALID;
    if (h->sticky_error) return h->sticky_error;
    // two counters at the end of the (otherwise unused between iterations) setup scratch
    long long* cyc = reinterpret_cast<long long*>(h->pb.setup());
    CK(h, cudaMemsetAsync(cyc, 0, 2 * sizeof(long long), h->pb.stream));
    launch_selftest_wait(h->pb, max_polls, cyc);
    long long host_cyc[2] = {0, 0};
    CK(h, cudaMemcpyAsync(host_cyc, cyc, sizeof(host_cyc), cudaMemcpyDeviceToHost, h->pb.stream));
    int rc = read_ctl(h);
    if (rc) return rc;
    if (cycles_out) { cycles_out[0] = host_cyc[0]; cycles_out[1] = host_cyc[1]; }
    return result_code(h, false);
}

size_t gem_nlr_host_job_device_bytes(const gem_nlr_params* params)
{
    if (!params || !valid_params(*params)) return 0;
    gem_nlr_params P = *params;
    P.x_inplace = 2;                                          // the device copy of X belongs to the job
    const size_t n = (size_t)P.n;
    return align_up(4 * n * P.d, 256) + align_up(4 * n * P.r, 256) + align_up(4 * n, 256) +
           make_layout(P).total;
}

int gem_nlr_run_host(const gem_nlr_params* params, const float* X_host, float* U_host,
                     int32_t* labels_host, void* device_buffer_dev, size_t device_bytes,
                     void* cuda_stream, double* a_out, gem_nlr_iter_info* last, int32_t* iters_done)
{
    return gem_nlr_run_host_timed(params, X_host, U_host, labels_host, device_buffer_dev, device_bytes, cuda_stream,
                                  a_out, last, iters_done, nullptr);
}

int gem_nlr_run_host_timed(const gem_nlr_params* params, const float* X_host, float* U_host,
                           int32_t* labels_host, void* device_buffer_dev, size_t device_bytes,
                           void* cuda_stream, double* a_out, gem_nlr_iter_info* last, int32_t* iters_done,
                           double* phase_ms_out)
{
    if (!params || !X_host || !U_host || !device_buffer_dev) return GEM_NLR_E_INVALID;
    if (!valid_params(*params) || ((uintptr_t)device_buffer_dev & 255)) return GEM_NLR_E_INVALID;
    if (device_bytes < gem_nlr_host_job_device_bytes(params)) return GEM_NLR_E_WORKSPACE;
    gem_nlr_params P = *params;
    P.x_inplace = 2;                                          // the device copy of X belongs to the job
    const size_t n = (size_t)P.n;
    char* base = (char*)device_buffer_dev;
    float* Xd = (float*)base;
    float* Ud = (float*)(base + align_up(4 * n * P.d, 256));
    int32_t* Ld = (int32_t*)((char*)Ud + align_up(4 * n * P.r, 256));
    char* ws = (char*)Ld + align_up(4 * n, 256);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // X goes first on the caller's stream; the starting factor follows on a side stream once X has arrived, so that
    // its transfer overlaps the setup (mean, power iteration, normalization, images), which needs X only.
    cudaStream_t side = nullptr;
    cudaEvent_t x_there = nullptr, u_there = nullptr;
    cudaEvent_t tev[4] = {nullptr, nullptr, nullptr, nullptr};   // job start, setup done, iterations done, copies done
    if (phase_ms_out) {
        for (int i = 0; i < 5; ++i) phase_ms_out[i] = 0.0;
        for (int i = 0; i < 4; ++i)
            if (cudaEventCreate(&tev[i]) != cudaSuccess) {
                for (int k = 0; k < i; ++k) cudaEventDestroy(tev[k]);
                return GEM_NLR_E_CUDA;
            }
    }
    auto release_tev = [&]() { for (int i = 0; i < 4; ++i) if (tev[i]) cudaEventDestroy(tev[i]); };
    if (cudaStreamCreateWithFlags(&side, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&x_there, phase_ms_out ? cudaEventDefault : cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&u_there, cudaEventDisableTiming) != cudaSuccess) {
        if (side) cudaStreamDestroy(side);
        if (x_there) cudaEventDestroy(x_there);
        release_tev();
        return GEM_NLR_E_CUDA;
    }
    auto release = [&]() { cudaStreamDestroy(side); cudaEventDestroy(x_there); cudaEventDestroy(u_there); release_tev(); };
    if (tev[0]) cudaEventRecord(tev[0], st);
    if (cudaMemcpyAsync(Xd, X_host, 4 * n * P.d, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaEventRecord(x_there, st) != cudaSuccess ||
        cudaStreamWaitEvent(side, x_there, 0) != cudaSuccess ||
        cudaMemcpyAsync(Ud, U_host, 4 * n * P.r, cudaMemcpyHostToDevice, side) != cudaSuccess ||
        cudaEventRecord(u_there, side) != cudaSuccess) {
        cudaStreamSynchronize(side);
        release();
        return GEM_NLR_E_CUDA;
    }
    gem_nlr_t* h = nullptr;
    int rc = gem_nlr_create(&h, &P, Xd, Ud, ws, make_layout(P).total, cuda_stream);
    if (rc < 0) { cudaStreamSynchronize(side); release(); return rc; }
    rc = gem_nlr_spectral_norm(h, a_out);
    if (tev[1]) cudaEventRecord(tev[1], st);
    // nothing before this point touches U; the iterations wait for it on the caller's stream
    if (cudaStreamWaitEvent(st, u_there, 0) != cudaSuccess) rc = GEM_NLR_E_CUDA;
    int run_rc = rc;
    if (rc >= 0) run_rc = gem_nlr_run(h, last, iters_done);
    if (tev[2]) cudaEventRecord(tev[2], st);
    if (run_rc >= 0 || run_rc == GEM_NLR_E_BREAKDOWN) {
        if (labels_host) {
            gem_nlr_labels(h, Ld);
            if (cudaMemcpyAsync(labels_host, Ld, 4 * n, cudaMemcpyDeviceToHost, st) != cudaSuccess)
                run_rc = GEM_NLR_E_CUDA;
        }
        if (cudaMemcpyAsync(U_host, Ud, 4 * n * P.r, cudaMemcpyDeviceToHost, st) != cudaSuccess)
            run_rc = GEM_NLR_E_CUDA;
        if (tev[3]) cudaEventRecord(tev[3], st);
        if (cudaStreamSynchronize(st) != cudaSuccess) run_rc = GEM_NLR_E_CUDA;
        if (phase_ms_out && run_rc >= 0) {
            float ms = 0.f;
            if (cudaEventElapsedTime(&ms, tev[0], x_there) == cudaSuccess) phase_ms_out[0] = ms;
            if (cudaEventElapsedTime(&ms, x_there, tev[1]) == cudaSuccess) phase_ms_out[1] = ms;
            if (cudaEventElapsedTime(&ms, tev[1], tev[2]) == cudaSuccess) phase_ms_out[2] = ms;
            if (cudaEventElapsedTime(&ms, tev[2], tev[3]) == cudaSuccess) phase_ms_out[3] = ms;
            if (cudaEventElapsedTime(&ms, tev[0], tev[3]) == cudaSuccess) phase_ms_out[4] = ms;
        }
    }
    gem_nlr_destroy(h);
    cudaStreamSynchronize(side);
    release();
    return run_rc;
}

}  // extern "C"
