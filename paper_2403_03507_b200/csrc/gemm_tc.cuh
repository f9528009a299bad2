// tcgen05 / TMEM / TMA projection kernels (bf16 operands, fp32 accumulation): interface.
#pragma once

#include <cuda.h>

#include "common.cuh"
#include "q8_code.cuh"

namespace galore {

// What the projection needs to run Adam on its output (Algorithm 1's update block and Eq. 15 in the
// epilogue): the layer's moments and where the normalised update goes.
struct TcAdamArgs {
  int32_t state_fmt;          // galore_state_fmt_t
  float *M, *V;               // fp32 moments (rows of ld_s floats), or
  uint8_t *Mc, *Vc;           // 8-bit codes (rows of ld_s bytes) with
  float *Mam, *Vam;           // one absmax per tile of q_block / 128 rows x 128 columns
  int64_t ld_s;
  int q_block;
  void* Nout;                 // bf16, leading dimension ld_n
  int64_t ld_n;
  AdamParams ap;
};

// Per-layer launch state of the tensor-core path: tensor maps of the operands the library owns
// (projector, normalised update).  The map of G is encoded per call; W is accessed without TMA.
struct TensorPlan {
  bool ready = false;
  int splits = 1;             // K slices of the projection
  int ctas = 1;               // 1: 128-row tiles per CTA; 2: 256-row tiles per CTA pair (cta_group::2)
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
int tensor_ctas(const galore_config_t& cfg);
galore_status_t tensor_plan_init(TensorPlan* plan, const galore_config_t& cfg, bool left, void* P, void* Nbuf,
                                 float* Rpart, int splits, int64_t ld_part, int64_t ld_n);
// G and W usable by this path: 16-byte aligned bases and rows.
bool tensor_operands_aligned(const galore_config_t& cfg, const void* W, int64_t ldw, const void* G, int64_t ldg);
// R partials <- P^T G (left) / G Q (right)
galore_status_t tensor_project(TensorPlan* plan, const galore_config_t& cfg, bool left, const void* G, int64_t ldg,
                               int32_t* status, cudaStream_t st);
// the same projection with Adam in its epilogue (one K slice): updates the moments, writes N, no R in memory
galore_status_t tensor_project_adam(TensorPlan* plan, const galore_config_t& cfg, bool left, const void* G, int64_t ldg,
                                    const TcAdamArgs& adam, int32_t* status, cudaStream_t st);
// W <- W - scale * P N (left) / N Q^T (right), N read from plan->Nbuf
galore_status_t tensor_back_project(TensorPlan* plan, const galore_config_t& cfg, bool left, void* W, int64_t ldw,
                                    float scale, float keep, int32_t* status, cudaStream_t st);


// ---- groups: up to tensor_group_capacity() layers per launch ------------------------------------
struct TensorGroup;   // opaque, host memory
TensorGroup* tensor_group_new();
void tensor_group_free(TensorGroup* t);
void tensor_group_reset(TensorGroup* t);
int tensor_group_count(const TensorGroup* t);
int tensor_group_capacity();
// the layer's projection with its R partials going to `part` (leading dimension ld_part, `splits` K slices)
galore_status_t tensor_group_add_project(TensorGroup* t, const TensorPlan* plan, const galore_config_t& cfg, bool left,
                                         const void* G, int64_t ldg, float* part, int64_t ld_part, int splits,
                                         int32_t* status);
// the layer's projection with Adam in its epilogue; launch with tensor_group_launch_project_adam
// (all layers of the group have the same state format)
galore_status_t tensor_group_add_project_adam(TensorGroup* t, const TensorPlan* plan, const galore_config_t& cfg, bool left,
                                              const void* G, int64_t ldg, const TcAdamArgs& adam, int32_t* status);
galore_status_t tensor_group_launch_project_adam(TensorGroup* t, int32_t state_fmt, cudaStream_t st);
// the layer's back-projection reading its normalised update from Nbuf (bf16, leading dimension ld_n)
galore_status_t tensor_group_add_back(TensorGroup* t, const TensorPlan* plan, const galore_config_t& cfg, bool left,
                                      const void* Nbuf, int64_t ld_n, void* W, int64_t ldw, float scale, float keep,
                                      int32_t* status);
// a plain GEMM: C (M x N fp32, ldc) = op(A) op(B), bf16 operands; *_mn = 1 when the operand is stored
// with M (resp. N) contiguous, 0 when K is contiguous.  Launch with tensor_group_launch_project.
galore_status_t tensor_group_add_gemm(TensorGroup* t, const void* A, int64_t lda, int a_mn, const void* B, int64_t ldb,
                                      int b_mn, int M, int N, int K, float* C, int64_t ldc, int32_t* status);
galore_status_t tensor_group_launch_project(TensorGroup* t, cudaStream_t st);
galore_status_t tensor_group_launch_back(TensorGroup* t, int32_t w_dtype, cudaStream_t st);

}  // namespace galore
