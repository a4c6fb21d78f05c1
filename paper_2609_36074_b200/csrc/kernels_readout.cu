// Label read-out for a factor with more columns than clusters (the paper's appendix "Additional Computation
// Details", paragraph "Recover cluster labels from U matrix"): the leading K left singular vectors of U as a
// spectral embedding, then K-means on its rows.
//
// The singular vectors come from the r x r Gram matrix: U^T U = Q S^2 Q^T, P_K = U Q_K S_K^{-1}.
//   1. G = U^T U in FP64: the first-product kernel with U in both places, split-K partials reduced in FP64.
//   2. Eigen-decomposition of G by parallel-order cyclic Jacobi (one CTA, FP64), the K largest eigenpairs
//      selected, E = Q_K S_K^{-1} (r x K).
//   3. Y = U E (n x K, FP32, caller-provided scratch).
//   4. K-means on the rows of Y, deterministic: farthest-point seeding (first centre = the row of largest norm,
//      then the row farthest from its nearest centre, lowest index on ties), Lloyd passes (nearest centre, lowest
//      index on ties; a centre without rows stays) until no label changes or max_iter passes.  Centre sums are
//      FP64 with a fixed owner per entry and a fixed combination order, so a run is reproducible.
// The paper does not fix the seeding or the stopping rule of its K-means; these are this library's.
#include "nlr_common.cuh"
#include "device_utils.cuh"

namespace gemnlr {

void launch_red_f64(const Problem& pb, const double* part, int g, int64_t count, double* out);

// ---------------------------------------------------------------------------------------------
// Parallel-order cyclic Jacobi on the symmetric r x r matrix A (FP64, row-major, overwritten); V receives the
// eigenvectors as columns.  A round pairs the r (or r + 1) indices like a round-robin tournament, so its
// rotations act on disjoint index pairs and are applied together: A <- J^T A J, V <- V J.
// Then the K largest eigenvalues are selected (ties: lower index first) and E[j][k] = V[j][idx_k] /
// sqrt(lambda_k) is written as FP32 (r x K row-major).  A K-th eigenvalue that is not positive relative to the
// largest (U has rank < K) raises GEM_NLR_E_BREAKDOWN in *status.
// ---------------------------------------------------------------------------------------------
constexpr int JT = 512;
__global__ void __launch_bounds__(JT)
k_jacobi_topk(double* __restrict__ A, double* __restrict__ V, int r, int K, float* __restrict__ E,
              double* __restrict__ cs /* 2 * (r + 1) / 2 */, int32_t* __restrict__ pq /* r + 1 */,
              int32_t* __restrict__ status, double* __restrict__ lambda_out)
{
    __shared__ double sred[32];
    __shared__ int s_done;
    const int tid = threadIdx.x;
    const int m = (r + 1) & ~1;                            // even number of players (index m - 1 = r is a bye when r is odd)
    const int half = m / 2;
    for (int e = tid; e < r * r; e += JT) V[e] = (e / r == e % r) ? 1.0 : 0.0;
    __syncthreads();
    for (int sweep = 0; sweep < 30; ++sweep) {
        // off-diagonal mass against the diagonal's
        double off = 0.0, dia = 0.0;
        for (int e = tid; e < r * r; e += JT) {
            const double v = A[e];
            if (e / r == e % r) dia += v * v; else off += v * v;
        }
        off = block_sum<JT>(off, sred);
        dia = block_sum<JT>(dia, sred);
        if (tid == 0) s_done = (off <= 1e-26 * dia) ? 1 : 0;
        __syncthreads();
        if (s_done) break;
        for (int round = 0; round < m - 1; ++round) {
            for (int k = tid; k < half; k += JT) {
                // player m - 1 stays and meets player `round`; the others meet symmetrically around `round`
                const int a = (k == 0) ? m - 1 : (round + k) % (m - 1);
                const int b = (k == 0) ? round : (round + (m - 1) - k) % (m - 1);
                int p = a < b ? a : b, q = a < b ? b : a;
                double c = 1.0, s = 0.0;
                if (q < r) {
                    const double apq = A[(size_t)p * r + q];
                    if (apq != 0.0) {
                        const double app = A[(size_t)p * r + p], aqq = A[(size_t)q * r + q];
                        const double tau = (aqq - app) / (2.0 * apq);
                        const double t = (tau >= 0.0 ? 1.0 : -1.0) / (fabs(tau) + sqrt(1.0 + tau * tau));
                        c = 1.0 / sqrt(1.0 + t * t);
                        s = t * c;
                    }
                } else {
                    q = -1;                                // bye
                }
                pq[2 * k] = p; pq[2 * k + 1] = q;
                cs[2 * k] = c; cs[2 * k + 1] = s;
            }
            __syncthreads();
            // rows: A <- J^T A   (row p' = c row p - s row q, row q' = s row p + c row q)
            for (int e = tid; e < half * r; e += JT) {
                const int k = e / r, j = e % r;
                const int p = pq[2 * k], q = pq[2 * k + 1];
                if (q < 0) continue;
                const double c = cs[2 * k], s = cs[2 * k + 1];
                const double x = A[(size_t)p * r + j], y = A[(size_t)q * r + j];
                A[(size_t)p * r + j] = c * x - s * y;
                A[(size_t)q * r + j] = s * x + c * y;
            }
            __syncthreads();
            // columns: A <- A J, V <- V J
            for (int e = tid; e < half * r; e += JT) {
                const int k = e / r, i = e % r;
                const int p = pq[2 * k], q = pq[2 * k + 1];
                if (q < 0) continue;
                const double c = cs[2 * k], s = cs[2 * k + 1];
                double x = A[(size_t)i * r + p], y = A[(size_t)i * r + q];
                A[(size_t)i * r + p] = c * x - s * y;
                A[(size_t)i * r + q] = s * x + c * y;
                x = V[(size_t)i * r + p]; y = V[(size_t)i * r + q];
                V[(size_t)i * r + p] = c * x - s * y;
                V[(size_t)i * r + q] = s * x + c * y;
            }
            __syncthreads();
        }
    }
    // selection of the K largest eigenvalues: rank of entry i = number of entries that beat it
    double lmax = 0.0;
    for (int i = 0; i < r; ++i) lmax = fmax(lmax, A[(size_t)i * r + i]);
    for (int i = tid; i < r; i += JT) {
        const double li = A[(size_t)i * r + i];
        int rank = 0;
        for (int j = 0; j < r; ++j) {
            const double lj = A[(size_t)j * r + j];
            if (lj > li || (lj == li && j < i)) ++rank;
        }
        if (rank < K) {
            pq[rank] = i;                                  // pq reused: index of the eigenpair of that rank
            lambda_out[rank] = li;
            if (!(li > 1e-12 * lmax)) *status = GEM_NLR_E_BREAKDOWN;
        }
    }
    __syncthreads();
    for (int e = tid; e < r * K; e += JT) {
        const int j = e / K, k = e % K;
        const int idx = pq[k];
        const double l = A[(size_t)idx * r + idx];
        E[e] = (float)(V[(size_t)j * r + idx] / sqrt(l > 0.0 ? l : 1.0));
    }
}

// ---------------------------------------------------------------------------------------------
// Y = c_f U E: n x r times r x K -> n x K (FP32 accumulation over r in tiles of 32), 64 x 64 output tiles.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
k_embed(const float* __restrict__ U, const float* __restrict__ E, const Ctl* __restrict__ ctl, int64_t n, int r, int K,
        float* __restrict__ Y)
{
    __shared__ __align__(16) float Us[64][33];
    __shared__ __align__(16) float Es[32][64];
    const float cf = ctl->c_f;
    const int k0 = blockIdx.y * 64;
    const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
    const int64_t n_tiles = (n + 63) / 64;
    for (int64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const int64_t m0 = tile * 64;
        float acc[4][4];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
        for (int j0 = 0; j0 < r; j0 += 32) {
            for (int idx = threadIdx.x; idx < 64 * 32; idx += 256) {
                const int mm = idx / 32, jj = idx % 32;
                const int64_t row = m0 + mm;
                Us[mm][jj] = (row < n && j0 + jj < r) ? cf * U[row * r + j0 + jj] : 0.f;
            }
            for (int idx = threadIdx.x; idx < 32 * 64; idx += 256) {
                const int jj = idx / 64, kk = idx % 64;
                Es[jj][kk] = (j0 + jj < r && k0 + kk < K) ? E[(size_t)(j0 + jj) * K + k0 + kk] : 0.f;
            }
            __syncthreads();
#pragma unroll 8
            for (int jj = 0; jj < 32; ++jj) {
                const float4 ev = *reinterpret_cast<const float4*>(&Es[jj][tx * 4]);
                const float ea[4] = {ev.x, ev.y, ev.z, ev.w};
#pragma unroll
                for (int a = 0; a < 4; ++a) {
                    const float x = Us[ty * 4 + a][jj];
#pragma unroll
                    for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(x, ea[b], acc[a][b]);
                }
            }
            __syncthreads();
        }
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            const int64_t row = m0 + ty * 4 + a;
            if (row >= n) continue;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int k = k0 + tx * 4 + b;
                if (k < K) Y[row * K + k] = acc[a][b];
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Farthest-point seeding.  pass 0: score_i = ||y_i||^2; pass m > 0: mind_i = min(mind_i, ||y_i - centre_{m-1}||^2),
// score_i = mind_i.  Each block reports its best (score, lowest row index); k_seed_pick takes the best block
// record (lowest row on ties), and copies that row of Y into centre m.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
k_seed_scan(const float* __restrict__ Y, int64_t n, int K, int m, const float* __restrict__ centres,
            float* __restrict__ mind, float* __restrict__ best_val, int64_t* __restrict__ best_row)
{
    extern __shared__ float sc[];                           // centre m - 1 (K floats)
    __shared__ float sv[256];
    __shared__ int64_t si[256];
    if (m > 0) {
        for (int j = threadIdx.x; j < K; j += 256) sc[j] = centres[(size_t)(m - 1) * K + j];
        __syncthreads();
    }
    float bv = -1.f;
    int64_t bi = -1;
    for (int64_t row = (int64_t)blockIdx.x * 256 + threadIdx.x; row < n; row += (int64_t)gridDim.x * 256) {
        const float* y = Y + row * K;
        float s = 0.f;
        if (m == 0) {
            for (int j = 0; j < K; ++j) s = fmaf(y[j], y[j], s);
        } else {
            for (int j = 0; j < K; ++j) { const float t = y[j] - sc[j]; s = fmaf(t, t, s); }
            const float old = (m == 1) ? s : mind[row];
            s = fminf(old, s);
            mind[row] = s;
        }
        if (s > bv) { bv = s; bi = row; }                   // rows are visited in increasing order: first maximum kept
    }
    sv[threadIdx.x] = bv; si[threadIdx.x] = bi;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) {
            const float v2 = sv[threadIdx.x + o];
            const int64_t i2 = si[threadIdx.x + o];
            if (i2 >= 0 && (v2 > sv[threadIdx.x] || (v2 == sv[threadIdx.x] && (si[threadIdx.x] < 0 || i2 < si[threadIdx.x])))) {
                sv[threadIdx.x] = v2; si[threadIdx.x] = i2;
            }
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) { best_val[blockIdx.x] = sv[0]; best_row[blockIdx.x] = si[0]; }
}

__global__ void __launch_bounds__(256)
k_seed_pick(const float* __restrict__ Y, int K, int m, int nblocks, const float* __restrict__ best_val,
            const int64_t* __restrict__ best_row, float* __restrict__ centres)
{
    __shared__ int64_t s_row;
    if (threadIdx.x == 0) {
        float bv = -1.f;
        int64_t bi = -1;
        for (int b = 0; b < nblocks; ++b) {
            const float v = best_val[b];
            const int64_t i = best_row[b];
            if (i >= 0 && (v > bv || (v == bv && i < bi) || bi < 0)) { bv = v; bi = i; }
        }
        s_row = bi < 0 ? 0 : bi;
    }
    __syncthreads();
    for (int j = threadIdx.x; j < K; j += 256) centres[(size_t)m * K + j] = Y[s_row * K + j];
}

// ---------------------------------------------------------------------------------------------
// Lloyd: assignment pass (thread per row; centres through shared memory in slabs), then centre sums.
// ---------------------------------------------------------------------------------------------
constexpr int SLAB = 32;                                    // centres per shared-memory slab
__global__ void __launch_bounds__(256)
k_lloyd_assign(const float* __restrict__ Y, int64_t n, int K, const float* __restrict__ centres,
               int32_t* __restrict__ labels, int first, unsigned long long* __restrict__ changed)
{
    extern __shared__ float sc[];                           // [SLAB][K]
    unsigned long long my_changed = 0;
    const int64_t rows_per_block = ((n + gridDim.x - 1) / gridDim.x + 255) / 256 * 256;
    const int64_t lo = (int64_t)blockIdx.x * rows_per_block;
    for (int64_t base = lo; base < lo + rows_per_block && base < n; base += 256) {
        const int64_t row = base + threadIdx.x;
        float best = 3.4e38f;
        int bk = 0;
        for (int k0 = 0; k0 < K; k0 += SLAB) {
            const int kn = (K - k0 < SLAB) ? K - k0 : SLAB;
            __syncthreads();
            for (int e = threadIdx.x; e < kn * K; e += 256) sc[e] = centres[(size_t)k0 * K + e];
            __syncthreads();
            if (row < n) {
                const float* y = Y + row * K;
                for (int k = 0; k < kn; ++k) {
                    const float* c = sc + (size_t)k * K;
                    float s = 0.f;
                    for (int j = 0; j < K; ++j) { const float t = y[j] - c[j]; s = fmaf(t, t, s); }
                    if (s < best) { best = s; bk = k0 + k; }        // strict: lowest centre index on ties
                }
            }
        }
        if (row < n) {
            if (first || labels[row] != bk) ++my_changed;
            labels[row] = bk;
        }
    }
    if (my_changed) atomicAdd(changed, my_changed);         // an integer count: order does not matter
}

// Centre sums: block b scans rows [b * span, (b + 1) * span); thread t owns entries (k, j) = t, t + 256, ... of the
// K x K sum and entry k of the counts, and adds the rows of its cluster in row order.  part[b][K * K + K].
__global__ void __launch_bounds__(256)
k_lloyd_sums(const float* __restrict__ Y, const int32_t* __restrict__ labels, int64_t n, int K, int64_t span,
             double* __restrict__ part)
{
    __shared__ int32_t sl[1024];
    const int64_t lo = (int64_t)blockIdx.x * span;
    const int64_t hi = (lo + span < n) ? lo + span : n;
    const int KK = K * K;
    double* out = part + (size_t)blockIdx.x * (KK + K);
    for (int e0 = 0; e0 < KK + K; e0 += 256 * 8) {
        double acc[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) acc[u] = 0.0;
        for (int64_t c0 = lo; c0 < hi; c0 += 1024) {
            const int cn = (int)((hi - c0 < 1024) ? hi - c0 : 1024);
            __syncthreads();
            for (int i = threadIdx.x; i < cn; i += 256) sl[i] = labels[c0 + i];
            __syncthreads();
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int e = e0 + u * 256 + threadIdx.x;
                if (e >= KK + K) continue;
                if (e < KK) {
                    const int k = e / K, j = e % K;
                    for (int i = 0; i < cn; ++i)
                        if (sl[i] == k) acc[u] += (double)Y[(c0 + i) * K + j];
                } else {
                    const int k = e - KK;
                    for (int i = 0; i < cn; ++i)
                        if (sl[i] == k) acc[u] += 1.0;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int e = e0 + u * 256 + threadIdx.x;
            if (e < KK + K) out[e] = acc[u];
        }
    }
}

__global__ void __launch_bounds__(256)
k_lloyd_centres(const double* __restrict__ part, int nblocks, int K, float* __restrict__ centres)
{
    const int KK = K * K;
    for (int e = blockIdx.x * 256 + threadIdx.x; e < KK; e += gridDim.x * 256) {
        const int k = e / K;
        double s = 0.0, cnt = 0.0;
        for (int b = 0; b < nblocks; ++b) {
            s += part[(size_t)b * (KK + K) + e];
            cnt += part[(size_t)b * (KK + K) + KK + k];
        }
        if (cnt > 0.0) centres[e] = (float)(s / cnt);       // a centre without rows stays where it is
    }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
struct ReadoutLayout {
    size_t Y, mind, centres, E, G, V, cs, pq, lam, best_val, best_row, sums, flags, total;
    int nb_scan, nb_sum;
};

static ReadoutLayout readout_layout(const gem_nlr_params& P)
{
    ReadoutLayout R;
    const size_t n = (size_t)P.n, r = (size_t)P.r, K = (size_t)P.K;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = (off + bytes + 255) / 256 * 256; return o; };
    R.nb_scan = (int)((n + 255) / 256 < (size_t)kSMs * 8 ? (n + 255) / 256 : (size_t)kSMs * 8);
    R.nb_sum = (int)((n + 4095) / 4096 < (size_t)kSMs * 2 ? (n + 4095) / 4096 : (size_t)kSMs * 2);
    R.Y = take(4 * n * K);
    R.mind = take(4 * n);
    R.centres = take(4 * K * K);
    R.E = take(4 * r * K);
    R.G = take(8 * r * r);
    R.V = take(8 * r * r);
    R.cs = take(8 * (r + 2));
    R.pq = take(4 * (r + 2 > K ? r + 2 : K));
    R.lam = take(8 * K);
    R.best_val = take(4 * (size_t)R.nb_scan);
    R.best_row = take(8 * (size_t)R.nb_scan);
    R.sums = take(8 * (size_t)R.nb_sum * (K * K + K));
    R.flags = take(64);
    R.total = off;
    return R;
}

size_t readout_scratch_bytes(const gem_nlr_params& P) { return readout_layout(P).total; }

// Enqueues the whole read-out; *passes_host / *status_host are filled after the final synchronization by the caller
// from the flags area: flags[0] = status (int32), flags[1] = passes (int32), flags[2..3] = changed counter.
// The Lloyd loop needs the count of changed labels on the host after every pass (one 8-byte read-back per pass).
int run_spectral_labels(const Problem& pb, int32_t* labels, char* scratch, int max_iter, int32_t* passes_out,
                        unsigned long long* pinned_changed /* pinned host, >= 16 bytes */)
{
    const auto& P = pb.P;
    const int r = P.r, K = P.K;
    const int64_t n = P.n;
    const ReadoutLayout R = readout_layout(P);
    float* Y = reinterpret_cast<float*>(scratch + R.Y);
    float* mind = reinterpret_cast<float*>(scratch + R.mind);
    float* centres = reinterpret_cast<float*>(scratch + R.centres);
    float* E = reinterpret_cast<float*>(scratch + R.E);
    double* G = reinterpret_cast<double*>(scratch + R.G);
    double* V = reinterpret_cast<double*>(scratch + R.V);
    double* cs = reinterpret_cast<double*>(scratch + R.cs);
    int32_t* pq = reinterpret_cast<int32_t*>(scratch + R.pq);
    double* lam = reinterpret_cast<double*>(scratch + R.lam);
    float* best_val = reinterpret_cast<float*>(scratch + R.best_val);
    int64_t* best_row = reinterpret_cast<int64_t*>(scratch + R.best_row);
    double* sums = reinterpret_cast<double*>(scratch + R.sums);
    int32_t* flags = reinterpret_cast<int32_t*>(scratch + R.flags);
    unsigned long long* changed = reinterpret_cast<unsigned long long*>(flags + 2);

    if (cudaMemsetAsync(flags, 0, 64, pb.stream) != cudaSuccess) return GEM_NLR_E_CUDA;
    // 1. G = U^T U
    {
        const int tiles = (r + G_RT - 1) / G_RT;
        const size_t cap = pb.L.part1_bytes / sizeof(double) / ((size_t)r * r);
        if (cap < 1) return GEM_NLR_E_WORKSPACE;
        int gx = pb.L.g1x;
        if ((size_t)gx > cap) gx = (int)cap;
        dim3 g1(gx, tiles * tiles);
        launch_pass1_partials(pb, pb.U, pb.U, r, r, tiles, g1);
        launch_red_f64(pb, pb.part1(), gx, (int64_t)r * r, G);
    }
    // 2. eigenpairs, E = Q_K S_K^{-1}
    k_jacobi_topk<<<1, JT, 0, pb.stream>>>(G, V, r, K, E, cs, pq, flags, lam);
    // 3. Y = U E
    {
        const int64_t n_tiles = (n + 63) / 64;
        dim3 ge((unsigned)(n_tiles < kSMs * 4 ? n_tiles : kSMs * 4), (unsigned)((K + 63) / 64));
        k_embed<<<ge, 256, 0, pb.stream>>>(pb.U, E, pb.ctl(), n, r, K, Y);
    }
    pb.count(2);
    // 4. seeding
    for (int m = 0; m < K; ++m) {
        k_seed_scan<<<R.nb_scan, 256, sizeof(float) * K, pb.stream>>>(Y, n, K, m, centres, mind, best_val, best_row);
        k_seed_pick<<<1, 256, 0, pb.stream>>>(Y, K, m, R.nb_scan, best_val, best_row, centres);
        pb.count(2);
    }
    // 5. Lloyd
    const int64_t span = (n + R.nb_sum - 1) / R.nb_sum;
    const int nb_assign = (int)((n + 255) / 256 < (int64_t)kSMs * 4 ? (n + 255) / 256 : (int64_t)kSMs * 4);
    const size_t sm_assign = sizeof(float) * SLAB * (size_t)K;
    if (sm_assign > 48 * 1024)
        cudaFuncSetAttribute(k_lloyd_assign, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm_assign);
    int passes = 0;
    for (int it = 0; it < max_iter; ++it) {
        if (cudaMemsetAsync(changed, 0, 8, pb.stream) != cudaSuccess) return GEM_NLR_E_CUDA;
        k_lloyd_assign<<<nb_assign, 256, sm_assign, pb.stream>>>(Y, n, K, centres, labels, it == 0 ? 1 : 0, changed);
        pb.count(1);
        ++passes;
        if (cudaMemcpyAsync(pinned_changed, changed, 8, cudaMemcpyDeviceToHost, pb.stream) != cudaSuccess ||
            cudaStreamSynchronize(pb.stream) != cudaSuccess)
            return GEM_NLR_E_CUDA;
        if (*pinned_changed == 0) break;
        k_lloyd_sums<<<R.nb_sum, 256, 0, pb.stream>>>(Y, labels, n, K, span, sums);
        k_lloyd_centres<<<(K * K + 255) / 256, 256, 0, pb.stream>>>(sums, R.nb_sum, K, centres);
        pb.count(2);
    }
    if (passes_out) *passes_out = passes;
    if (cudaMemcpyAsync(pinned_changed, flags, 8, cudaMemcpyDeviceToHost, pb.stream) != cudaSuccess ||
        cudaStreamSynchronize(pb.stream) != cudaSuccess)
        return GEM_NLR_E_CUDA;
    const int32_t status = *reinterpret_cast<int32_t*>(pinned_changed);
    return status < 0 ? status : GEM_NLR_OK;
}

}  // namespace gemnlr
