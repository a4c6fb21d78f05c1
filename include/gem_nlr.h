/*
 * gem_nlr.h -- C ABI of the B200 (sm_100a) library for the spectrally normalized
 * nonnegative low-rank (NLR) K-means iteration ("GEM iteration").
 *
 * The library runs Algorithm 1 of the paper (restated call by call in its
 * Algorithm 2) on one GPU:
 *
 *   setup      X_c = X - 1 xbar^T,  a = ||X_c||_2,  X-hat = X_c / a        (Section 3)
 *   iteration  Theta = X-hat^T U;  ybar = y/sqrt(n) + (beta/n) q;  s = U^T ybar;
 *              W = [U + 2 alpha X-hat Theta - alpha (ybar p^T + 1 s^T)]_+   (Eq. "gpu-positive-update")
 *              a = ||W||_F^2, b = ||U||_F^2, h = <W, U> in FP64            (Eq. "fused-statistics")
 *              c = FP32(sqrt(K)/sqrt(a));  U <- c W;
 *              delta-hat = sqrt(max{c^2 a + b - 2 c h, 0} / K)             (Eq. "movement-estimate")
 *              p = U^T 1;  q = U p - 1;  dual step if gated;  rho = ||q||_2 / sqrt(n); stop test.
 *
 * Conventions
 *  - All matrices are row-major FP32.  X is n x d, U is n x r (r >= K), Theta is d x r.
 *  - Every pointer named *_dev is DEVICE memory owned by the caller; it must stay valid
 *    until gem_nlr_destroy.  Pointers named *_host are host memory.  The handle itself
 *    owns only host memory (a pinned read-back record); it never calls a device allocator.
 *  - U_dev is the single n x r factor buffer.  It is updated in place.  Between the
 *    kernels of an iteration it holds the unnormalized W together with a pending FP32
 *    multiplier kept on the device; whenever a call of this header returns, U_dev holds the
 *    normalized factor (the multiplier has been applied), except after a normalization
 *    breakdown, where it holds W as the paper's loop leaves it.
 *  - Work is enqueued on the CUDA stream given at creation (a cudaStream_t passed as
 *    void*; NULL is the legacy default stream).  Calls that return host-visible numbers
 *    synchronize that stream before returning.  One handle = one stream; a handle is not
 *    thread-safe.
 *  - Return values: >= 0 success (GEM_NLR_OK, GEM_NLR_CONVERGED, GEM_NLR_ITER_CAP),
 *    < 0 error.  No exception crosses this boundary and no kernel traps.
 */
#ifndef GEM_NLR_H
#define GEM_NLR_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GEM_NLR_OK            0   /* call succeeded; iteration neither stopped nor capped        */
#define GEM_NLR_CONVERGED     1   /* the stopping test of Algorithm 1 fired                      */
#define GEM_NLR_ITER_CAP      2   /* gem_nlr_run reached T iterations                            */
#define GEM_NLR_E_INVALID    -1   /* bad argument, NULL or misaligned pointer                    */
#define GEM_NLR_E_CUDA       -2   /* a CUDA call failed; see gem_nlr_last_error                  */
#define GEM_NLR_E_WORKSPACE  -3   /* workspace smaller than gem_nlr_workspace_bytes              */
#define GEM_NLR_E_BREAKDOWN  -4   /* sqrt(a) <= 1e-20: W vanished (Algorithm 1, breakdown line)   */
#define GEM_NLR_E_NONFINITE  -5   /* a, b or h is not finite                                     */
#define GEM_NLR_E_NOT_READY  -6   /* iteration requested before X was normalized                 */
#define GEM_NLR_E_TIMEOUT    -7   /* a bounded device-side wait (copy pipeline) ran out; the     */
                                  /* kernel ran to its end without the data it waited for (most  */
                                  /* kernels stop storing into U_dev then), so U_dev and the     */
                                  /* dual are undefined afterwards: reload them                  */
                                  /* (gem_nlr_set_state) before iterating again                  */
#define GEM_NLR_E_TOO_LARGE  -8   /* size beyond the fixed capacity of a *_static entry point    */

typedef struct gem_nlr gem_nlr_t;   /* opaque handle */

/* Problem statement of Algorithm 1 plus the controls the paper leaves open. */
typedef struct {
    int64_t  n;             /* rows of X (data points)                                           */
    int32_t  d;             /* columns of X (features)                                           */
    int32_t  K;             /* number of clusters: radius ||U||_F^2 = K and divisor of delta-hat */
    int32_t  r;             /* columns of U, r >= K                                              */
    float    alpha;         /* primal step size                                                  */
    float    beta;          /* penalty on h = g/sqrt(n); the stored penalty is beta/n            */
    int32_t  T;             /* iteration cap                                                     */
    int32_t  T_min;         /* no stop before this many iterations                               */
    double   eps_d;         /* dual gate:  max{c^2 a + b - 2 c h, 0} < eps_d^2 K                 */
    double   eps_c;         /* stop: gate and delta-hat < eps_c and rho < eps_c                  */
    int32_t  center;        /* 1: subtract the column mean before the spectral norm (paper)      */
    int32_t  x_inplace;     /* 1: X_dev is overwritten by X-hat; 0: X-hat lives in the workspace; */
                            /* 2: X_dev may be given up: as 1, and where both products read only  */
                            /* the fp16 operand images the row-major image pair is built over     */
                            /* X-hat after setup (same bytes), so the workspace holds only the    */
                            /* transposed pair; gem_nlr_objective, gem_nlr_init_range and buffer 5 */
                            /* then return GEM_NLR_E_INVALID (they read X-hat itself)             */
    int32_t  pi_max_iters;  /* power-iteration cap for ||X_c||_2 (<=0: 100)                      */
    double   pi_tol;        /* stop when |sigma_k - sigma_{k-1}| <= pi_tol * sigma_k (<=0: 1e-7) */
    uint64_t pi_seed;       /* seed of the starting vector                                       */
    int32_t  precision;     /* contraction arithmetic, always FP32-accurate with FP32           */
                            /* accumulation: 0 FP32 FFMA; 1 tcgen05 tensor cores (3-product      */
                            /* TF32 split, or 3-product FP16 split x 2^k = h1 + h2 with          */
                            /* overflow-free power-of-two scales, which needs U in Omega:        */
                            /* ||U||_F^2 = K); 2 the generic FFMA kernels whatever the shape     */
                            /* (cross-checks); 3 3xTF32 warp-level MMA; -1 let the library       */
                            /* choose by shape                                                   */
    int32_t  history;       /* 1: keep one gem_nlr_iter_info per iteration in the workspace      */
} gem_nlr_params;

/* What one iteration of Algorithm 1 produced (all FP64 as on the paper's host side). */
typedef struct {
    int32_t t;              /* index of the iteration (0-based)                                  */
    int32_t dual_applied;   /* 1 if the dual-ascent gate fired                                   */
    int32_t stop;           /* 1 if the stopping test fired at this iteration                    */
    int32_t status;         /* GEM_NLR_OK or a negative GEM_NLR_E_* raised by this iteration     */
    double  a, b, h;        /* ||W||_F^2, ||U_prev||_F^2, <W, U_prev>                            */
    double  c;              /* FP64 value of the FP32 multiplier sqrt(K)/sqrt(a)                 */
    double  delta_hat;      /* relative primal movement estimate                                 */
    double  rho;            /* ||q||_2 / sqrt(n) for the new iterate                             */
    double  fhat;           /* objective f-hat_y(U) at the iterate this iteration started from   */
} gem_nlr_iter_info;

/* Bytes of caller-provided device workspace needed for these parameters (0 if invalid).
 * Includes the y/sqrt(n) and ybar vectors, Theta, p, s, the reduction partials, the
 * optional history, when x_inplace == 0 a copy of X and, for the tensor-core shapes
 * (precision -1 or 1, r >= 32, n >= 4096), the static fp16 split images of X-hat, row-major
 * and transposed (8 n d' bytes, d' = d rounded up to a multiple of 32: the image kernels see
 * zero features beyond d, so any d is accepted; d' = 256 for wide factors, r > 128 with
 * 64 <= d < 256, and for 128 < d < 256 with d' r > 16384, whose kernels work on 256-feature
 * blocks), and one FP64 partial record of d' r entries per row range of the first product
 * (up to 64 MB).                                                                               */
size_t gem_nlr_workspace_bytes(const gem_nlr_params *params);

/* Device bytes the paper's own buffer table would use for the same problem:
 * 4 (nd + nr + dr + 4n + 2r) + 24 (ceil(n/128) ceil(r/64) + 1)   (Eq. "gpu-storage").          */
size_t gem_nlr_paper_storage_bytes(const gem_nlr_params *params);

/* Create a solver.  X_dev: n x d data (16-byte aligned).  U_dev: n x r starting factor in the
 * feasible set (nonnegative, ||U||_F^2 = K), 16-byte aligned.  workspace_dev: 256-byte aligned,
 * at least gem_nlr_workspace_bytes.  The dual variable starts at zero.  Nothing is launched.   */
int gem_nlr_create(gem_nlr_t **out, const gem_nlr_params *params, float *X_dev, float *U_dev,
                   void *workspace_dev, size_t workspace_bytes, void *cuda_stream);

/* Setup of Section 3: column mean (if center), a = ||X_c||_2, then X-hat = X_c / a written over
 * X_dev (x_inplace) or into the workspace.  a comes from applying X_c^T X_c implicitly to unit
 * vectors (one streaming pass over X per application, the power-iteration kernel pair) combined
 * by a Lanczos recurrence on the host: the estimate is the largest Ritz value, never above the
 * true norm; it stops when the estimate moves by less than pi_tol (relative) twice in a row or
 * after pi_max_iters passes.  *a_out receives a.  Synchronizes.                                */
int gem_nlr_spectral_norm(gem_nlr_t *h, double *a_out);

/* Declare that X_dev already holds X-hat (normalized elsewhere); a is recorded only.           */
int gem_nlr_set_normalized(gem_nlr_t *h, double a);

/* Data-informed starting factor (appendix "Additional Computation Details", paragraph "Initialization"):
 *     V = X-hat X-hat^T Z,  V = Q R,  U0 = Proj_Omega(Q) = sqrt(K) [Q]_+ / ||[Q]_+||_F,
 * the orthonormalization done as Cholesky QR in feature space (M = X-hat^T Z, C = X-hat^T X-hat,
 * M^T C M = R^T R, Q = X-hat (M R^{-1})).  On entry U_dev holds the sample matrix Z (n x r, the caller's
 * random draw, e.g. i.i.d. N(0,1); finite entries); on return it holds U0, the dual is zero and the
 * iteration counter is 0.  X must have been normalized.  The large products run on the general-shape FFMA
 * kernels with FP64 accumulation of the split-K partials; the r x r factorization and the solve are FP64.
 * Needs r <= d (the sample has rank at most d) -- GEM_NLR_E_INVALID otherwise -- and a sample that is not
 * too ill-conditioned for Cholesky QR: a non-positive pivot returns GEM_NLR_E_BREAKDOWN (U_dev then still
 * holds Z, and the handle stays usable: write another Z, or a starting factor of your own, and go on).
 * Synchronizes.                                                                                     */
int gem_nlr_init_range(gem_nlr_t *h);

/* Exactly one iteration of Algorithm 1 from the current (U, y).  On return U_dev holds the new
 * normalized U and *info (may be NULL) the iteration's numbers.  Returns GEM_NLR_OK,
 * GEM_NLR_CONVERGED if the stop test fired, or an error.  Synchronizes.                        */
int gem_nlr_step(gem_nlr_t *h, gem_nlr_iter_info *info);

/* Iterate until the stop test fires or T iterations have been taken in total.  No host round
 * trip per iteration: the gate, the multiplier and the stop flag stay on the device.
 * *last (may be NULL) describes the final iteration, *iters_done the total count.
 * Returns GEM_NLR_CONVERGED, GEM_NLR_ITER_CAP or an error.  Synchronizes once at the end.      */
int gem_nlr_run(gem_nlr_t *h, gem_nlr_iter_info *last, int32_t *iters_done);

/* label_i = smallest j with U_ij = max_j U_ij (an all-zero row gets 0).  labels_dev: n int32.
 * Enqueued on the handle's stream; does not synchronize.
 * This row argmax is this library's read-out, not the paper's (its appendix on rounding takes the top-K
 * left singular vectors of U and runs K-means on the embedded rows).  It names clusters only for
 * r == K: at an exact solution U U^T is block diagonal with U >= 0, so rows of different clusters have
 * disjoint supports and each of the K clusters owns exactly one of the K columns.  For r > K a cluster
 * may own several columns, and the argmax then splits it: the labels are still the row argmax, but they
 * are column indices, not cluster indices.                                                       */
int gem_nlr_labels(gem_nlr_t *h, int32_t *labels_dev);

/* The paper's own read-out (appendix "Additional Computation Details", paragraph "Recover cluster labels
 * from U matrix"), for any r >= K: the leading K left singular vectors of U as a spectral embedding, then
 * K-means on its rows.  The singular vectors come from the r x r Gram matrix (U^T U = Q S^2 Q^T,
 * P_K = U Q_K S_K^{-1}; FP64, Jacobi).  The paper fixes neither the seeding nor the stopping rule of its
 * K-means; here both are deterministic: farthest-point seeding (first centre = the row of largest norm, each
 * further centre the row farthest from its nearest centre, lowest row index on ties), then Lloyd passes
 * (nearest centre, lowest centre index on ties; a centre without rows stays) until no label changes or
 * max_iter passes.  Label k is the k-th seeded centre.  labels_dev: n int32 (output).  scratch_dev: caller-owned
 * device memory, 256-byte aligned, at least gem_nlr_labels_spectral_scratch_bytes (about 4 n (K + 1) bytes:
 * the embedding); it also uses the handle's split-K partial area, so it must not run concurrently with an
 * iteration.  *passes_out (may be NULL): assignment passes made.  Needs r <= 2048.  Returns GEM_NLR_OK,
 * GEM_NLR_E_BREAKDOWN if U has numerical rank below K, or an argument / CUDA error.  Reads back 8 bytes per
 * Lloyd pass; synchronizes.                                                                          */
size_t gem_nlr_labels_spectral_scratch_bytes(const gem_nlr_params *params);
int gem_nlr_labels_spectral(gem_nlr_t *h, int32_t *labels_dev, void *scratch_dev, size_t scratch_bytes,
                            int32_t max_iter, int32_t *passes_out);

/* f-hat_y(U) of Eq. "normalized" at the current (U, y).  Synchronizes.                         */
int gem_nlr_objective(gem_nlr_t *h, double *fhat_out);

/* Checkpoint helpers.  get: copies y/sqrt(n) (n floats, device to device) and the iteration
 * counter; U is already in the caller's buffer.  set: the caller has written a new U into
 * U_dev; ytilde_dev (n floats, may be NULL for zeros) and t replace the dual and the counter.  */
int gem_nlr_get_state(gem_nlr_t *h, float *ytilde_dev, int32_t *t_out);
int gem_nlr_set_state(gem_nlr_t *h, const float *ytilde_dev, int32_t t);

/* Copies up to max_records per-iteration records (oldest first) to host memory; returns the
 * number copied, or a negative error.  Needs params.history == 1.  Synchronizes.               */
int gem_nlr_history(gem_nlr_t *h, gem_nlr_iter_info *records_host, int32_t max_records);

/* Device pointers into the workspace, for inspection by tests (valid until destroy):
 * which: 0 Theta (d*r floats), 1 p (r), 2 s (r), 3 ytilde (n), 4 ybar (n), 5 X-hat (n*d).      */
int gem_nlr_buffer(gem_nlr_t *h, int32_t which, void **ptr_dev);

/* Name of the kernel family chosen for the two contractions: "generic", "ffma", "mma.tf32x3",
 * "f16x3" (tcgen05, fp16 split, both products), "f16x3.tiled" (the same for r > 256), or
 * "first+second" when the two products come from different families, e.g. "generic+f16x3",
 * "generic+f16x3.tiled", "f16x3+tf32x3".  The string is static.                                  */
const char *gem_nlr_path(gem_nlr_t *h);

/* Text of the last CUDA error seen by this handle ("" if none).                                */
const char *gem_nlr_last_error(gem_nlr_t *h);

int gem_nlr_destroy(gem_nlr_t *h);

/* Measurement helpers (no counterpart in the paper's algorithm).
 * gem_nlr_profile(h, 1) makes every following iteration record CUDA events on the handle's
 * stream around its two phases: (1) vector pass + first product Theta = X-hat^T U with its
 * reductions, (2) the fused second-product kernel.  gem_nlr_profile_read returns the device
 * milliseconds accumulated per phase and the number of iterations they cover (at most 1024
 * iterations between two read-backs of the control block are recorded).
 * gem_nlr_launch_count: kernels this handle has launched since creation.                       */
int gem_nlr_profile(gem_nlr_t *h, int32_t enable);
int gem_nlr_profile_read(gem_nlr_t *h, double *ms_first_phase, double *ms_second_product,
                         int64_t *iterations);
int64_t gem_nlr_launch_count(gem_nlr_t *h);

/* ---- Row-sharded runs over several GPUs (one process and one handle per GPU) ---------------------------
 * The iteration shards by rows: rank g holds rows_g of X, U and the dual (n in its gem_nlr_params is its own
 * row count), and the small replicated quantities are summed over the ranks twice per iteration -- after the
 * first product Theta (d x r), s (r), sum q^2, sum ytilde q; after the second a, b, h and the column sums of
 * W (r) -- plus once per application of X_c^T X_c during setup and once for the column mean.  The library
 * does not link a communication library: the caller supplies two callbacks (with torch.distributed / NCCL
 * behind them in the Python binding).  The sums themselves are taken by this library's kernels, in rank
 * order, from the gathered per-rank records, so every rank obtains bit-identical replicated values and the
 * result does not depend on a library's reduction order.  The paper runs on one GPU; this is the scale-out
 * its largest data sets call for.
 *
 * gem_nlr_gather_fn: all ranks call it with the same byte count; when the work it enqueues on cuda_stream
 * has completed, recv_dev holds the world records of `bytes` bytes each, back to back in rank order
 * (an all-gather; send_dev and recv_dev are device memory of this rank).  Returns 0 on success.
 * gem_nlr_host_sum_fn: replaces buf_host[0 .. count) by its sum over the ranks, added in rank order, on
 * every rank (host memory; blocking).  Returns 0 on success.
 *
 * gem_nlr_shard_attach: call after gem_nlr_create and before anything else.  n_global = total rows.
 * exchange_dev: device memory of gem_nlr_shard_exchange_bytes(params, world) bytes, 256-byte aligned,
 * caller-owned, alive until destroy.  Afterwards gem_nlr_spectral_norm, _step, _run, _objective and _labels
 * work as on one GPU (every rank must make the same calls in the same order; rho, the gate and the stop test
 * are global and identical on all ranks; labels are those of the rank's own rows).  gem_nlr_init_range,
 * gem_nlr_labels_spectral and gem_nlr_run_host are single-GPU calls and return GEM_NLR_E_INVALID on a
 * sharded handle.                                                                                       */
typedef int (*gem_nlr_gather_fn)(void *ctx, const void *send_dev, void *recv_dev, size_t bytes, void *cuda_stream);
typedef int (*gem_nlr_host_sum_fn)(void *ctx, double *buf_host, int64_t count);
size_t gem_nlr_shard_exchange_bytes(const gem_nlr_params *params, int32_t world);
int gem_nlr_shard_attach(gem_nlr_t *h, int32_t rank, int32_t world, int64_t n_global, gem_nlr_gather_fn gather,
                         gem_nlr_host_sum_fn host_sum, void *ctx, void *exchange_dev, size_t exchange_bytes);

/* Self-test of the failure path that a healthy run never takes (no counterpart in the paper): every wait of
 * the copy / tensor-core pipelines is bounded, and when one runs out the kernel records GEM_NLR_E_TIMEOUT
 * and runs to its end instead of hanging.  This call launches a one-CTA kernel that waits, through the same
 * device code, on a barrier nothing arrives on, giving up after max_polls polls (1 .. 2^20), and then waits
 * once more with the production limit, which must return at once.  It returns GEM_NLR_E_TIMEOUT when the
 * path works (GEM_NLR_OK would mean the wait never ran out); the handle keeps that error, as after a real
 * time-out, and refuses further iterations until gem_nlr_set_state reloads the factor and the dual.
 * cycles_out (2 entries of host memory, may be NULL): SM clock cycles spent in the two waits.
 * Nothing faults, traps or spins without bound.  Synchronizes.                                     */
int gem_nlr_selftest_wait_timeout(gem_nlr_t *h, uint32_t max_polls, int64_t *cycles_out);

/* Whole job with HOST buffers: copies X_host and U_host to device_buffer_dev, runs setup, up to
 * T iterations and the label read-out, and copies U (into U_host) and the labels back.
 * device_buffer_dev must hold gem_nlr_host_job_device_bytes(params) bytes (256-byte aligned).
 * a_out, last, iters_done may be NULL.  Returns as gem_nlr_run.                                */
size_t gem_nlr_host_job_device_bytes(const gem_nlr_params *params);
int gem_nlr_run_host(const gem_nlr_params *params, const float *X_host, float *U_host,
                     int32_t *labels_host, void *device_buffer_dev, size_t device_bytes,
                     void *cuda_stream, double *a_out, gem_nlr_iter_info *last,
                     int32_t *iters_done);

/* The same job with a per-phase record (a measurement helper; the paper has no counterpart).
 * phase_ms_out: 5 doubles of host memory (may be NULL), filled from CUDA events on cuda_stream when the
 * job succeeds: [0] host-to-device copy of X; [1] setup (mean, spectral norm, normalization, operand
 * images), which overlaps the copy of the starting factor; [2] the iterations, including any wait for
 * the starting factor's copy; [3] label read-out and the device-to-host copies of U and the labels;
 * [4] the whole job from the first copy to the last.  Host-side work between the phases (handle
 * creation, the read-backs of the setup) is inside [1] and [2]; what the caller measures around the
 * call beyond [4] is host overhead (stream, event and pinned-record creation, their release).     */
int gem_nlr_run_host_timed(const gem_nlr_params *params, const float *X_host, float *U_host,
                           int32_t *labels_host, void *device_buffer_dev, size_t device_bytes,
                           void *cuda_stream, double *a_out, gem_nlr_iter_info *last,
                           int32_t *iters_done, double *phase_ms_out);

/* Column sums without any allocation: p_dev[j] = sum_i U_dev[i * r + j], j < r (FP64 sums in a
 * fixed order, rounded once to FP32) -- the p = U^T 1 of the iteration, for a factor the caller
 * holds.  The paper has no counterpart of this entry point; it exists for callers that cannot
 * allocate device memory at the time of the call: code living inside a host application that
 * distributes all device memory at start-up and forbids cudaMalloc afterwards, latency-critical
 * loops where an allocation's device-wide synchronization is not acceptable, or processes whose
 * memory already belongs to a pool they do not control.  Such callers have no workspace to hand
 * to gem_nlr_create either.
 *
 * U_dev: n x r row-major FP32 device memory (input, not modified).  p_dev: r floats of device
 * memory (output).  Both are the caller's.  The scratch for the per-block partial sums is a
 * fixed array inside the library (about 300 KB per GPU that loads the library, held until the
 * process exits); this call never calls cudaMalloc, cudaFree or any allocating routine.
 * Limit: r <= GEM_NLR_STATIC_MAX_R; a wider factor is refused with GEM_NLR_E_TOO_LARGE and
 * nothing is launched.  n is not limited.
 *
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress, with
 * that device current).  With CUDA's lazy module loading this is also the moment the driver loads
 * this entry point's module and places the array, which may synchronize the device and can fail if
 * the device has no memory left: make that first call once at start-up, as a warm-up, before any
 * stream capture begins and before memory runs short.  The device that cuda_stream belongs to must
 * be the current device on every call (the scratch address and the launch follow the current
 * device).  All calls share
 * the one array and it keeps the previous call's partial sums: every call overwrites what it
 * reads, so nothing needs clearing, but two calls whose kernels overlap on the GPU (different
 * streams without an ordering between them) race on it -- order them.
 * The work is enqueued on cuda_stream (a cudaStream_t; NULL = legacy default stream) and the
 * call does not synchronize.  Returns GEM_NLR_OK, GEM_NLR_E_INVALID (NULL pointer, n < 1 or
 * r < 1), GEM_NLR_E_TOO_LARGE, or GEM_NLR_E_CUDA.                                               */
#define GEM_NLR_STATIC_MAX_R 128
int gem_nlr_column_sums_static(const float *U_dev, int64_t n, int32_t r, float *p_dev,
                               void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* GEM_NLR_H */
