// Self-test of the bounded device-side wait: the one path of the TMA / tcgen05 pipelines that a healthy run
// never takes.  A one-CTA kernel waits, through the same mbar_wait code the iteration kernels use, on an
// mbarrier that nothing ever arrives on, with a small poll limit: the wait must run out, record
// GEM_NLR_E_TIMEOUT in the control block and return; a second wait must then return at once because the CTA's
// abort flag is up.  Nothing traps, faults or spins without bound.
#include "nlr_common.cuh"
#include "pipeline.cuh"

namespace gemnlr {

__global__ void __launch_bounds__(64)
k_selftest_wait(Ctl* __restrict__ ctl, uint32_t max_polls, long long* __restrict__ cycles_out)
{
    __shared__ __align__(8) uint64_t bar;
    __shared__ uint32_t abort_flag;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        abort_flag = 0;
        fence_barrier_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const long long t0 = clock64();
        mbar_wait_limit(b, 0, &abort_flag, ctl, max_polls);          // nobody arrives: runs out after max_polls polls
        cycles_out[0] = clock64() - t0;
    }
    __syncthreads();
    if (threadIdx.x == 32) {
        const long long t0 = clock64();
        mbar_wait(b, 0, &abort_flag, ctl);                           // production limit, but the abort flag is up
        cycles_out[1] = clock64() - t0;
    }
}

void launch_selftest_wait(const Problem& pb, uint32_t max_polls, long long* cycles_dev)
{
    k_selftest_wait<<<1, 64, 0, pb.stream>>>(pb.ctl(), max_polls, cycles_dev);
    pb.count(1);
}

}  // namespace gemnlr
