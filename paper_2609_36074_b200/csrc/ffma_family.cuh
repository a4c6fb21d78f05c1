// Launch interface of the TMA-staged FP32-FFMA kernel family (kernels_ffma.cu).
#pragma once
#include <cuda.h>
#include "nlr_common.cuh"

namespace gemnlr {

struct FfmaPlan {
    alignas(64) CUtensorMap tm1;   // X-hat tiles of the first product
    alignas(64) CUtensorMap tm2;   // X-hat tiles of the second product
    int shape_id;
    int g1, g2;                    // persistent grids
};

// True if (d, r, n) is covered by an instantiated shape and the tensor maps could be encoded.
bool ffma_plan(const Problem& pb, FfmaPlan* plan);
// Vector pass + Theta = X-hat^T U + reductions + the scalar step finishing the previous iteration.
void ffma_launch_first(const Problem& pb, const FfmaPlan& plan, int mode);
// Reduction of g per-CTA partial records [d*r Theta | r s | sum q^2 | sum ytilde q] (FP64) + scalar step.
void red1_fused_launch(const Problem& pb, int g, int mode);
// The same reduction over the gathered records of a row-sharded run (one per rank, rank order), followed by the
// scalar step on the combined sums; n_global is the row count over all ranks.
void red1_combine_launch(const Problem& pb, const double* records, int world, int64_t n_global, int mode);
// Fused second product, statistics, scalar step (multiplier, movement, gate, p).
void ffma_launch_second(const Problem& pb, const FfmaPlan& plan);


// Same interface for the warp-level tensor-core kernels (kernels_mma.cu: mma.sync TF32, 3-product split).
bool mma_plan(const Problem& pb, FfmaPlan* plan);
void mma_launch_first(const Problem& pb, const FfmaPlan& plan, int mode);
void mma_launch_second(const Problem& pb, const FfmaPlan& plan);

}  // namespace gemnlr
