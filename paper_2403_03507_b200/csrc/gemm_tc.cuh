// tcgen05 / TMEM / TMA projection kernels (bf16 operands, fp32 accumulation): interface.
#pragma once

#include <cuda.h>

#include "adam.cuh"
#include "common.cuh"

namespace galore {

// Per-layer launch state of the tensor-core path: tensor maps of the operands the library owns
// (projector, normalised update, split-K partials).  Maps of W and G are encoded per call.
struct TensorPlan {
  bool ready = false;
  int splits = 1;
  void* P = nullptr;
  void* Nbuf = nullptr;
  float* Rpart = nullptr;
  CUtensorMap map_p_proj;    // projector as an operand of the projection
  CUtensorMap map_p_back;    // projector as an operand of the back-projection
  CUtensorMap map_n_back;    // normalised update as an operand of the back-projection
};

// bf16 G and P, leading dimensions that TMA can address.
bool tensor_path_eligible(const galore_config_t& cfg);
int tensor_proj_splits(const galore_config_t& cfg, bool left);
galore_status_t tensor_plan_init(TensorPlan* plan, const galore_config_t& cfg, bool left, void* P, void* Nbuf,
                                 float* Rpart, int splits);
bool tensor_operands_aligned(const galore_config_t& cfg, const void* W, int64_t ldw, const void* G, int64_t ldg);
galore_status_t step_tensor(TensorPlan* plan, const galore_config_t& cfg, bool left, void* W, int64_t ldw,
                            const void* G, int64_t ldg, float scale, const AdamParams& ap, float* M, float* V,
                            uint8_t* Mc, float* Mam, uint8_t* Vc, float* Vam, int q_block, int64_t nel,
                            int32_t* status, cudaStream_t st);

}  // namespace galore
