// tcgen05 / TMEM / TMA projection kernels (bf16 operands, fp32 accumulation): interface.
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace galore {

// Per-layer launch state of the tensor-core path: tensor maps of the operands the library owns
// (projector, normalised update).  The map of G is encoded per call; W is accessed without TMA.
struct TensorPlan {
  bool ready = false;
  int splits = 1;             // K slices of the projection
  void* P = nullptr;
  void* Nbuf = nullptr;       // normalised update, bf16, leading dimension ld_n
  float* Rpart = nullptr;     // split-K partials of R, fp32, leading dimension ld_part
  int64_t ld_part = 0, ld_n = 0;
  CUtensorMap map_p_proj;     // projector as an operand of the projection
  CUtensorMap map_p_back;     // projector as an operand of the back-projection
  CUtensorMap map_n_back;     // normalised update as an operand of the back-projection
};

// bf16 G and P, rank a multiple of 8 (16-byte rows for TMA).
bool tensor_path_eligible(const galore_config_t& cfg);
int tensor_proj_splits(const galore_config_t& cfg, bool left);
galore_status_t tensor_plan_init(TensorPlan* plan, const galore_config_t& cfg, bool left, void* P, void* Nbuf,
                                 float* Rpart, int splits, int64_t ld_part, int64_t ld_n);
// G and W usable by this path: 16-byte aligned bases and rows.
bool tensor_operands_aligned(const galore_config_t& cfg, const void* W, int64_t ldw, const void* G, int64_t ldg);
// R partials <- P^T G (left) / G Q (right)
galore_status_t tensor_project(TensorPlan* plan, const galore_config_t& cfg, bool left, const void* G, int64_t ldg,
                               int32_t* status, cudaStream_t st);
// W <- W - scale * P N (left) / N Q^T (right), N read from plan->Nbuf
galore_status_t tensor_back_project(TensorPlan* plan, const galore_config_t& cfg, bool left, void* W, int64_t ldw,
                                    float scale, int32_t* status, cudaStream_t st);

}  // namespace galore
