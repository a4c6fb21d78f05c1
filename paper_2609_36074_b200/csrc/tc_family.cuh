// Launch interface of the 3xTF32 tcgen05 kernel family (kernels_tc.cu).
#pragma once
#include <cuda.h>
#include "nlr_common.cuh"

namespace gemnlr {

struct TcPlan {
    alignas(64) CUtensorMap tmX;   // X-hat boxes: 128 rows x 32 features (FP32, or the fp16 image h1)
    alignas(64) CUtensorMap tmX2;  // fp16 image h2 (fp16 split only)
    alignas(64) CUtensorMap tmU;   // U panels: 128 rows x 32 columns (load and store)
    bool f16;                      // two-term fp16 split on the static images of X-hat, else the TF32 split
    int eT;                        // Theta is scaled by 2^eT before its fp16 split
    int NP;                        // r padded to a multiple of 16 (MMA N)
    int PW;                        // columns per U panel: 16 (plain rows) or 32 (128-byte swizzle)
    int NSB, NLO, NUP;             // raw/hi box ring, lo box ring, U panel ring sizes
    int g2;                        // persistent grid
    size_t smem2;
    float* img_hi;                 // pre-split Theta^T images in the workspace
    float* img_lo;
};

// True if the shape is covered (d a multiple of 32, r a multiple of 4 in [8, 256], Theta images
// fit in shared memory) and the tensor maps could be encoded.  img_storage: 2 * d * NP floats.
bool tc_plan(const Problem& pb, TcPlan* plan, float* img_storage);
// Theta image build + fused second product, statistics, scalar step.
void tc_launch_second(const Problem& pb, const TcPlan& plan);

}  // namespace gemnlr

namespace gemnlr {

// First product + vector pass on tcgen05 (kernels_tc1.cu): d a multiple of 32 up to 256,
// r a multiple of 4 in [8, 128], d * r <= 16384.
struct Tc1Plan {
    alignas(64) CUtensorMap tmX;   // X-hat boxes: 32 rows x 32 features
    alignas(64) CUtensorMap tmU;   // U boxes: 32 rows x 32 columns
    int NSR, NLO;                  // raw stage ring, image stage ring
    bool ximg;                     // X-hat operand from the static transposed fp16 images
    int grid;
    size_t smem;
};
bool tc1_plan(const Problem& pb, Tc1Plan* plan);
// Theta partials, s, sum q^2, sum ytilde q (reduced afterwards by the FFMA family's k_red1_fused).
void tc1_launch_first(const Problem& pb, const Tc1Plan& plan);

}  // namespace gemnlr

namespace gemnlr {

// Tiled second product for wide problems (kernels_tcg.cu): d a multiple of 16, r a multiple of 4 up to
// 2048; Theta^T images of 2 * d * (r rounded up to 256) floats.
struct TcgPlan {
    alignas(64) CUtensorMap tmX1;  // X-hat image h1 (n x d fp16): boxes of 128 rows x 32 features, 64-byte swizzle
    alignas(64) CUtensorMap tmX2;  // X-hat image h2
    alignas(64) CUtensorMap tmU;   // U panels of the second product: 128 rows x 32 columns FP32, 128-byte swizzle
    int NCB;                       // 256-column blocks
    int eT;                        // Theta is scaled by 2^eT before its fp16 split
    int g2;
    size_t smem2;
    void* img_h1;                  // Theta^T images (fp16), rebuilt every iteration
    void* img_h2;
};
bool tcg_plan(const Problem& pb, TcgPlan* plan, float* img_storage);
// Builds the static fp16 images of X-hat (row-major and transposed); call whenever X-hat has become valid.
void tcg_prepare(const Problem& pb);

// Matching first product (Theta^T tiles of 128 columns x 256 features, split over row ranges): d a
// multiple of 32, (r / 128) * (d / 256) tiles at most one per SM.  The vector pass runs separately.
struct Tcg1Plan {
    alignas(64) CUtensorMap tmU;   // U slices: 32 rows x 128 columns FP32, plain rows
    int NMT, NNB, NSPLIT, grid;
    size_t smem;
};
bool tcg1_plan(const Problem& pb, Tcg1Plan* plan);
// Theta partials per row range + their reduction (Theta, ||Theta||^2 shares).
void tcg_launch_first(const Problem& pb, const Tcg1Plan& plan);
void tcg_launch_second(const Problem& pb, const TcgPlan& plan);

}  // namespace gemnlr
