// sm_100a building blocks shared by the TMA-staged kernel families: mbarrier pipeline with
// bounded waits, TMA tile / bulk loads, tensor-map encoding on the host.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include "nlr_common.cuh"

namespace gemnlr {

// Upper bound on polls of one mbarrier wait.  A healthy wait ends within microseconds; when the
// limit is hit the kernel records GEM_NLR_E_TIMEOUT, stops waiting anywhere (all later waits
// return at once) and runs to its end, so the context stays usable.
constexpr uint32_t kSpinLimit = 1u << 20;

__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void fence_barrier_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}

// Bounded wait.  abort_flag lives in shared memory and is shared by the whole CTA; it is looked at only after
// a failed attempt (every 64th), so the common case -- the phase is already complete -- costs one instruction.
__device__ __forceinline__ void mbar_wait_limit(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                                Ctl* ctl, uint32_t limit)
{
    for (uint32_t i = 0; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return;
        if ((i & 63u) == 63u && *abort_flag) return;
    }
    *abort_flag = 1u;
    ctl->status = GEM_NLR_E_TIMEOUT;
    ctl->stopped = 1;
}

__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          Ctl* ctl)
{
    mbar_wait_limit(bar, parity, abort_flag, ctl, kSpinLimit);
}

// Bounded wait by polling (mbarrier.test_wait never suspends the thread): for the hand-overs on the critical
// path of a pipeline, where the suspension period of try_wait (of the order of a microsecond) would be
// paid on every stage.
__device__ __forceinline__ void mbar_wait_spin(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                               Ctl* ctl)
{
    // The barrier is tested first and the abort flag only every 64 polls: the caller is a single thread whose
    // instruction stream sets the stage rate, and a shared-memory read of the flag in front of every wait
    // costs it tens of cycles per stage.  Once the flag is up a wait therefore returns within 64 polls.
    for (uint32_t i = 0; i < (kSpinLimit << 4); ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return;
        if ((i & 63u) == 63u && *abort_flag) return;
    }
    *abort_flag = 1u;
    ctl->status = GEM_NLR_E_TIMEOUT;
    ctl->stopped = 1;
}

// Bounded wait by polling with a short sleep between polls: for roles that may wait long (a team waiting
// for the MMAs to free an image stage, a producer waiting for a free slot).  A pure polling loop would
// take issue slots from the single MMA-issuing thread on the same scheduler; the sleep (~100 ns) bounds
// the extra hand-over latency.
__device__ __forceinline__ void mbar_wait_backoff(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                                  Ctl* ctl)
{
    if (*abort_flag) return;
    for (uint32_t i = 0; i < (kSpinLimit << 2); ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return;
        __nanosleep(100);
    }
    *abort_flag = 1u;
    ctl->status = GEM_NLR_E_TIMEOUT;
    ctl->stopped = 1;
}

// Same bounded wait for roles that are not on the critical path of the tensor pipe: the hardware may
// suspend the thread for up to ~1 us per attempt instead of letting it poll, so that waiting warps do not
// take issue slots from the single thread that issues the MMAs on the same scheduler.
__device__ __forceinline__ bool mbar_try_wait_suspend(uint32_t bar, uint32_t parity, uint32_t hint_ns)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(hint_ns) : "memory");
    return ok != 0;
}

__device__ __forceinline__ void mbar_wait_relaxed(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                                  Ctl* ctl)
{
    if (*abort_flag) return;
    for (uint32_t i = 0; i < kSpinLimit; ++i)
        if (mbar_try_wait_suspend(bar, parity, 1000u)) return;
    *abort_flag = 1u;
    ctl->status = GEM_NLR_E_TIMEOUT;
    ctl->stopped = 1;
}

// Programmatic dependent launch.  A kernel launched with launch_pdl() may become resident while its predecessor in
// the stream is still running; grid_dep_wait() returns once that predecessor has completed and its writes are
// visible (it returns at once when the kernel was launched the ordinary way).  grid_dep_launch() lets the next
// kernel in the stream start becoming resident.  Used by the three kernels of the skinny-shape iteration, whose
// launch latencies are a few per cent of a 0.23 ms iteration.
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Tile load: box of the tensor map at element coordinates (x = column, y = row).  x * 4 bytes
// must be a multiple of 16.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tmap, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"((uint64_t)tmap), "r"(x), "r"(y), "r"(bar) : "memory");
}

// Contiguous copy global -> shared; both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"((uint64_t)src), "r"(bytes), "r"(bar) : "memory");
}

// Hint: bring `bytes` (multiple of 16) starting at the 16-byte aligned global address into L2.
// Ask for a tile of a tensor map to be brought into L2 (no shared-memory destination, no completion).
__device__ __forceinline__ void tma_prefetch_2d(const CUtensorMap* tmap, int x, int y)
{
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"((uint64_t)tmap), "r"(x), "r"(y) : "memory");
}

__device__ __forceinline__ void bulk_prefetch_l2(const void* src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"((uint64_t)src), "r"(bytes) : "memory");
}

__device__ __forceinline__ float4 lds128(uint32_t addr)
{
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}

__device__ __forceinline__ void sts128(uint32_t addr, float4 v)
{
    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}

// Host: 2-D FP32 tensor map over a row-major rows x cols matrix, box = box_rows x box_cols,
// 128-byte swizzle when box_cols * 4 == 128 (16-byte atoms: chunk index XOR row mod 8; or, with
// atom32, 32-byte atoms: 32-byte chunk index XOR row mod 4 -- the layout MN-major TF32 UMMA operands
// need), no swizzle otherwise.  Out-of-range elements read as zero.
// Returns false if the driver entry point is missing or the encode fails.
bool make_tensor_map_2d(CUtensorMap* out, const float* base, int64_t rows, int cols, int box_rows, int box_cols,
                        bool atom32 = false, int swizzle_bytes = 0);
bool make_tensor_map_2d_f16(CUtensorMap* out, const void* base, int64_t rows, int64_t cols, int64_t pitch_halves,
                            int box_rows, int box_cols);

}  // namespace gemnlr
