// Row-sharded runs: every GPU holds a block of rows of X-hat, U and the dual; the small replicated quantities are
// summed over the ranks twice per iteration (after the first product: Theta, s, sum q^2, sum ytilde q; after the
// second: a, b, h and the column sums of W).  Each rank packs its sums into an FP64 record, the caller-supplied
// gather brings all ranks' records to every rank (pure communication), and the combination runs here, in rank
// order, so every rank computes bit-identical replicated values and the result does not depend on the
// communication library's reduction order.
#include "nlr_common.cuh"
#include "device_utils.cuh"
#include "fin_logic.cuh"
#include "ffma_family.cuh"

namespace gemnlr {

size_t shard_record_doubles(const gem_nlr_params& P, int dp)
{
    const size_t first = (size_t)dp * P.r + P.r + 2, second = 3 + (size_t)P.r;
    return first > second ? first : second;
}

// rec = [dp * r Theta | r s | sum q^2 | sum ytilde q] from this rank's parked values
__global__ void __launch_bounds__(256)
k_shard_pack_first(const float* __restrict__ theta, const float* __restrict__ s, const Ctl* __restrict__ ctl, int dr, int r,
                   int mode, double* __restrict__ rec)
{
    for (int e = blockIdx.x * 256 + threadIdx.x; e < dr + r + 2; e += gridDim.x * 256) {
        double v;
        if (e < dr) v = (mode == 1) ? 0.0 : (double)theta[e];
        else if (e < dr + r) v = (double)s[e - dr];
        else v = (e == dr + r) ? ctl->qq : ctl->yq;
        rec[e] = v;
    }
}

// rec = [a, b, h | r column sums]
__global__ void __launch_bounds__(256)
k_shard_pack_second(const float* __restrict__ p, const Ctl* __restrict__ ctl, int r, double* __restrict__ rec)
{
    for (int e = blockIdx.x * 256 + threadIdx.x; e < 3 + r; e += gridDim.x * 256)
        rec[e] = (e == 0) ? ctl->sa : (e == 1) ? ctl->sb : (e == 2) ? ctl->sh : (double)p[e - 3];
}

// One CTA: the ranks' records summed in rank order, the scalar step of Algorithm 2 (d)-(e) on the sums,
// p = c * (column sums).  colsum_only: p = column sums, nothing else.
__global__ void __launch_bounds__(256)
k_shard_combine_second(Ctl* __restrict__ ctl, const double* __restrict__ recs, int world, int stride, int r, int K,
                       double eps_d, int colsum_only, float* __restrict__ p)
{
    __shared__ double sc;
    __shared__ int sok;
    if (!colsum_only && ctl->stopped) return;
    if (threadIdx.x == 0) {
        double c = 1.0;
        int ok = 1;
        if (!colsum_only) {
            double a = 0.0, b = 0.0, h = 0.0;
            for (int g = 0; g < world; ++g) {
                a += recs[(size_t)g * stride + 0];
                b += recs[(size_t)g * stride + 1];
                h += recs[(size_t)g * stride + 2];
            }
            ok = fin2_scalars(ctl, a, b, h, K, eps_d, &c, true) ? 1 : 0;
        }
        sc = c;
        sok = ok;
    }
    __syncthreads();
    if (!sok) return;
    for (int j = threadIdx.x; j < r; j += 256) {
        double v = 0.0;
        for (int g = 0; g < world; ++g) v += recs[(size_t)g * stride + 3 + j];
        p[j] = (float)(sc * v);
    }
}

static int do_gather(const Problem& pb, size_t count)
{
    const ShardInfo& S = *pb.shard;
    if (count > S.xcount) return GEM_NLR_E_WORKSPACE;
    if (S.gather(S.ctx, S.xbuf, S.xbuf + S.xcount, count * sizeof(double), (void*)pb.stream) != 0) return GEM_NLR_E_CUDA;
    return GEM_NLR_OK;
}

int shard_exchange_first(const Problem& pb, int mode)
{
    const ShardInfo& S = *pb.shard;
    const int dr = pb.P.d * pb.P.r, r = pb.P.r;
    const size_t count = (size_t)dr + r + 2;
    k_shard_pack_first<<<kSMs, 256, 0, pb.stream>>>(pb.theta(), pb.s(), pb.ctl(), dr, r, mode, S.xbuf);
    pb.count(1);
    const int rc = do_gather(pb, count);
    if (rc) return rc;
    // the gathered records sit count apart only if the area was sized for exactly this record: compact strides are
    // what the gather delivers (world records of `count` doubles, back to back)
    red1_combine_launch(pb, S.xbuf + S.xcount, S.world, S.n_global, mode);
    return GEM_NLR_OK;
}

int shard_exchange_second(const Problem& pb, int colsum_only)
{
    const ShardInfo& S = *pb.shard;
    const int r = pb.P.r;
    const size_t count = 3 + (size_t)r;
    k_shard_pack_second<<<4, 256, 0, pb.stream>>>(pb.p(), pb.ctl(), r, S.xbuf);
    const int rc = do_gather(pb, count);
    if (rc) return rc;
    k_shard_combine_second<<<1, 256, 0, pb.stream>>>(pb.ctl(), S.xbuf + S.xcount, S.world, (int)count, r, pb.P.K, pb.P.eps_d,
                                                     colsum_only, pb.p());
    pb.count(2);
    return GEM_NLR_OK;
}

}  // namespace gemnlr
