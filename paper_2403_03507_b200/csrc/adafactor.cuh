// Adafactor on the compact gradient R (Sec. "GaLore with memory-efficient optimizers": Adafactor with
// first-order statistics; the update itself is Shazeer and Stern's, the paper prints none): declarations.
#pragma once

#include "common.cuh"

namespace galore {

constexpr double kAdafactorDecay = 0.8;     // beta2_t = 1 - t^-0.8
constexpr float kAdafactorEps1 = 1e-30f;    // added to R^2
constexpr float kAdafactorClip = 1.0f;      // the update is divided by max(1, rms / clip)
constexpr int kAfTileRows = 64;             // tile of the statistics pass: 64 rows x 128 columns
constexpr int kAfTileCols = 128;
constexpr int kAfSumBlocks = 592;           // fixed grid of the rms pass: its total is reproducible

// One layer's Adafactor step.  R partials, N and M are row-major with their own row pitches.
struct AdafactorItem {
  float* Rpart;            // split-K partials of R; slice 0 receives their sum
  int splits;
  int64_t split_stride;
  int rows, cols;          // shape of R and M
  int64_t r_ld, n_ld, s_ld;
  float* M;                // first moment (fp32)
  float *v_row, *v_col;    // running means of R^2 + eps_1 along rows (rows entries) and columns (cols entries)
  void* Nout;              // the new first moment once more, as the operand of the back-projection (fp32 or bf16)
  float beta1;
  double t;                // completed steps + 1
  float* scratch;          // adafactor_scratch_bytes(rows, cols) bytes
};
size_t adafactor_scratch_bytes(int64_t rows, int64_t cols);
galore_status_t launch_adafactor(const AdafactorItem& item, int32_t n_dtype, cudaStream_t st);

// Several layers in the same launches (every reduction stays inside its layer and keeps its order: a
// layer's result does not depend on what it is grouped with).  All items share the dtype of N.
constexpr int kAdafactorGroup = 32;
struct AdafactorGroup {
  AdafactorItem item[kAdafactorGroup];
  int tile_end[kAdafactorGroup];     // running totals of the statistics pass's tiles
  int vec_end[kAdafactorGroup];      // running totals of the 256-entry blocks of v_row | v_col
  float beta2t[kAdafactorGroup];
  int count;
};
galore_status_t adafactor_group_add(AdafactorGroup& g, const AdafactorItem& item);
galore_status_t launch_adafactor_group(const AdafactorGroup& g, int32_t n_dtype, cudaStream_t st);

}  // namespace galore
