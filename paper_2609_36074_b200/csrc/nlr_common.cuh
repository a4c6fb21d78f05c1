// Shared declarations of the NLR iteration library: the device-resident control block,
// the workspace layout and the launch entry points of each kernel family.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>
#include "../../include/gem_nlr.h"

namespace gemnlr {

// Device-resident control block.  The gate, the pending multiplier and the stop flag never
// leave the GPU between iterations; every iteration kernel reads them from here.
struct Ctl {
    float   c_f;            // pending multiplier: logical U = c_f * (contents of the U buffer)
    int32_t t;              // iterations completed
    int32_t dual_pending;   // gate of the last completed iteration fired, ytilde not yet updated
    int32_t tail_pending;   // rho / stop test of the last completed iteration not yet evaluated
    int32_t stopped;        // stop test fired or an error was raised: iteration kernels return at once
    int32_t status;         // GEM_NLR_OK / GEM_NLR_CONVERGED / negative error
    int32_t hist_cap;       // capacity of the history array (0: none)
    int32_t hist_len;       // records written
    double  fhat_cur;       // objective at the iterate the iteration in flight started from
    double  theta2;         // ||Theta||_F^2 of the latest Theta
    double  qq, yq;         // sum q_i^2, sum ytilde_i q_i of the latest vector pass
    double  f_final;        // objective at the current iterate when the stop test fired
    gem_nlr_iter_info last; // latest iteration (rho/stop filled in when its tail has run)
    uint32_t counter[4];    // arrival counters for last-block reductions (always left at zero)
    // Row-sharded runs (several GPUs, each with a block of rows): with shard_world > 1 the scalar steps inside the
    // iteration kernels only park their local sums here (and in the Theta, s, p buffers); the sums of all ranks
    // are combined, in rank order, by the exchange kernels, which then take the scalar step on every rank alike.
    int32_t shard_world;    // 0 or 1: not sharded
    int32_t pad_;
    double  sa, sb, sh;     // parked local a, b, h
};

struct Layout {
    size_t ctl, p, s, alpha_s, theta, thimg, ytilde, ybar, part1, part1v, part2, red1, setup, hist, xhat, total;
    size_t init;             // FP64 scratch of the data-informed start: M, C, T, G (0 bytes when r > d)
    size_t part1_bytes;      // size of the split-K partial area
    size_t ximg, ximgT;      // fp16 split images of X-hat (row-major and transposed), wide tensor-core shapes only (else 0 bytes)
    int has_img;             // the fp16 images of X-hat exist (tensor-core shapes)
    int img_inplace;         // x_inplace == 2 and both products read images only: the row-major image pair is built over
                             // X-hat in the caller's X buffer (row i: d halves of h1, then d halves of h2) and ximg is 0 bytes
    int dp;                  // d rounded up to a multiple of 32 when the fp16 images exist, else d: feature count of the image kernels
    int64_t n_pad;           // n rounded up to 64: the transposed images cover n_pad / 32 stages of 32 rows
    int fb;                  // features per block of the transposed images: 256, or d when d < 256
    int g1x, g1y_d, g1y_r;   // generic pass-1 grid: row chunks, d tiles, r tiles
    int gv;                  // vector kernel CTAs
    int g2x, g2y;            // generic pass-2 grid: row-tile CTAs, column tiles
    int gs;                  // setup kernels' CTAs
    int nred1;               // CTAs of the Theta reduction
};

constexpr int kSMs = 148;
constexpr int G_TM = 64, G_DT = 64, G_RT = 64;       // generic pass-1 tile
constexpr int G2_TM = 64, G2_RT = 64, G2_DT = 32;    // generic pass-2 tile

// Row ranges of the tiled tcgen05 first product (one resident CTA per 128 columns of U, 256-feature block and row
// range): as many as fill the SMs, while every range keeps at least eight 32-row stages and the FP64 partial
// records (one dp x r record per range) stay within 64 MB.
inline int tiled_first_row_ranges(int64_t n, int dp, int r)
{
    const int tiles = ((r + 127) / 128) * ((dp + 255) / 256);
    if (tiles > kSMs) return 0;
    int64_t s = kSMs / tiles;
    const int64_t rec = (int64_t)sizeof(double) * dp * r;
    const int64_t cap = ((int64_t)64 << 20) / rec;
    const int64_t by_rows = (n + 31) / 32 / 8;
    if (s > cap) s = cap;
    if (s > by_rows) s = by_rows;
    return s < 1 ? 1 : (int)s;
}

Layout make_layout(const gem_nlr_params& P);

// Host-side description of a row-sharded run (owned by the handle).
struct ShardInfo {
    int rank, world;
    int64_t n_global;                       // rows over all ranks: gamma = beta / n_global, rho = ||q|| / sqrt(n_global)
    gem_nlr_gather_fn gather;               // all-gather of equal-sized device records, in rank order, on a stream
    gem_nlr_host_sum_fn host_sum;           // in-place sum of a host FP64 vector over the ranks, in rank order
    void* ctx;
    double* xbuf;                           // device exchange area: [count] send, then [world][count] receive
    size_t xcount;                          // doubles per record the area was sized for
};

struct Problem {
    const ShardInfo* shard;                 // null: single GPU
    gem_nlr_params P;
    int dx;          // features per row of X as stored (row pitch).  P.d equals dx except in the view the
                     // fp16-image tensor-core kernels get, where P.d is dx rounded up to a multiple of 32:
                     // those kernels read X-hat only through its images, whose padding features are zero,
                     // so Theta gains zero rows and nothing else changes
    float* X;        // X-hat once normalized
    float* U;
    char*  ws;
    Layout L;
    cudaStream_t stream;
    float gamma_f;   // beta / n
    double gamma;
    int64_t* launches;       // host counter of kernel launches (owned by the handle)
    void count(int k = 1) const { if (launches) *launches += k; }
    Ctl* ctl() const { return reinterpret_cast<Ctl*>(ws + L.ctl); }
    float* p() const { return reinterpret_cast<float*>(ws + L.p); }
    float* s() const { return reinterpret_cast<float*>(ws + L.s); }
    float* alpha_s() const { return reinterpret_cast<float*>(ws + L.alpha_s); }
    float* theta() const { return reinterpret_cast<float*>(ws + L.theta); }
    // fp16 split images of X-hat (wide tensor-core shapes): h1 then h2, row-major n x d; transposed d x n_pad
    uint16_t* ximg(int which) const
    {
        if (L.img_inplace) return reinterpret_cast<uint16_t*>(X) + (size_t)which * P.d;
        return reinterpret_cast<uint16_t*>(ws + L.ximg) + (size_t)which * P.n * P.d;
    }
    int64_t ximg_pitch() const { return L.img_inplace ? 2 * (int64_t)P.d : (int64_t)P.d; }   // halves between rows of an image
    // transposed images: [n_pad / 32 stages][ceil(d / fb) blocks][fb features][32 rows] halves each
    size_t ximgT_halves() const { return (size_t)(L.n_pad / 32) * ((P.d + L.fb - 1) / L.fb) * L.fb * 32; }
    uint16_t* ximgT(int which) const { return reinterpret_cast<uint16_t*>(ws + L.ximgT) + (size_t)which * ximgT_halves(); }
    bool has_ximg() const { return L.has_img != 0; }
    float* ytilde() const { return reinterpret_cast<float*>(ws + L.ytilde); }
    float* ybar() const { return reinterpret_cast<float*>(ws + L.ybar); }
    double* part1() const { return reinterpret_cast<double*>(ws + L.part1); }
    double* part1v() const { return reinterpret_cast<double*>(ws + L.part1v); }
    double* part2() const { return reinterpret_cast<double*>(ws + L.part2); }
    double* red1() const { return reinterpret_cast<double*>(ws + L.red1); }
    double* setup() const { return reinterpret_cast<double*>(ws + L.setup); }
    double* init() const { return reinterpret_cast<double*>(ws + L.init); }
    gem_nlr_iter_info* hist() const { return reinterpret_cast<gem_nlr_iter_info*>(ws + L.hist); }
};

// ---- generic family (any n, d, r) -------------------------------------------------------
// One iteration = vector pass, Theta partials, Theta reduction + scalars, fused second product,
// statistics reduction + scalars.  tail: finish the last iteration (dual step, rho, stop) and
// apply the pending multiplier to the U buffer.
void launch_init_colsum(const Problem& pb);                 // p = U^T 1 for a freshly loaded U
void launch_vector_pass(const Problem& pb);
void launch_generic_pass1(const Problem& pb, int ignore_stop);
void launch_fin1(const Problem& pb, int mode);
void launch_generic_pass2_kernel(const Problem& pb);
void launch_generic_pass2_alpha(const Problem& pb, float alpha);    // the same kernel with a given step size
// FP64 split-K partials of A^T (c_f B) into part1 (A: n x da, B: n x rb, both row-major with their own width as
// pitch; grid = (row chunks, da tiles x rb tiles)); ignores the stop flag.
void launch_pass1_partials(const Problem& pb, const float* A, const float* B, int da, int rb, int tiles_b, dim3 grid);
// Data-informed starting factor (kernels_init.cu).
bool launch_range_init(const Problem& pb);
void launch_red_f64(const Problem& pb, const double* part, int g, int64_t count, double* out);
// Spectral label read-out for r >= K (kernels_readout.cu): leading K left singular vectors + K-means.
size_t readout_scratch_bytes(const gem_nlr_params& P);
int run_spectral_labels(const Problem& pb, int32_t* labels, char* scratch, int max_iter, int32_t* passes_out,
                        unsigned long long* pinned_host /* >= 16 bytes */);
// Reduction of g FP64 partials of Theta (layout [d][r] each) into Theta and the ||Theta||^2 shares.
void launch_red1(const Problem& pb, int g, int ignore_stop, int scale_cf);   // the fused second product alone
void launch_fin2(const Problem& pb, int gx, int gy, int cols_per);
void launch_tail(const Problem& pb);
void launch_objective(const Problem& pb);                   // fills ctl->f_final for the current (U, y)
void launch_labels(const Problem& pb, int32_t* labels);

// ---- row-sharded runs (kernels_shard.cu): exchange of the small replicated quantities ----------
// After the first phase (local Theta, s, sum q^2, sum ytilde q parked): gather, combine in rank order, scalar step
// with the mode of the deferred call (0 iteration, 1 tail, 2 objective).  Returns a GEM_NLR_* code.
int shard_exchange_first(const Problem& pb, int mode);
// After the second product (local a, b, h parked, local column sums in p): gather, combine, multiplier, gate, p.
// colsum_only: just p = sum of the ranks' column sums (a freshly loaded factor).
int shard_exchange_second(const Problem& pb, int colsum_only);
size_t shard_record_doubles(const gem_nlr_params& P, int dp);

// ---- self-test of the bounded waits (selftest.cu) ------------------------------------------
void launch_selftest_wait(const Problem& pb, uint32_t max_polls, long long* cycles_dev /* 2 entries */);

// ---- setup (Section 3) -------------------------------------------------------------------
// Returns a negative GEM_NLR_E_* or 0; writes a to *a_out.  Synchronizes the stream.
int run_spectral_norm(const Problem& pb, const float* X_in, float* Xhat_out, double* a_out,
                      double* host_scratch /* pinned, >= 4 doubles */);

}  // namespace gemnlr
