// Adam-on-R kernels and the 8-bit block-wise state format: declarations.
#pragma once

#include "common.cuh"

namespace galore {

struct AdamParams {
  float b1, b2;          // beta1, beta2
  float omb1, omb2;      // 1 - beta1, 1 - beta2
  float eps;
  float inv_bc1, inv_bc2;  // 1 / (1 - beta^t), t = completed steps + 1
};

// Where element i of the packed state (row-major, `cols` wide) sits in the R partials and in N,
// whose rows may be padded (leading dimensions r_ld, n_ld) so that TMA can address them.
struct StateGeom {
  int64_t cols = 0, r_ld = 0, n_ld = 0;   // cols == 0: everything is packed
  __host__ __device__ __forceinline__ int64_t r_index(int64_t i) const {
    return (cols == 0 || r_ld == cols) ? i : (i / cols) * r_ld + (i % cols);
  }
  __host__ __device__ __forceinline__ int64_t n_index(int64_t i) const {
    return (cols == 0 || n_ld == cols) ? i : (i / cols) * n_ld + (i % cols);
  }
};

// One layer's share of a grouped Adam launch.
struct AdamItem {
  const float* Rpart;      // split-K partials of R
  int splits;
  int64_t split_stride;
  int nel;                 // state elements
  float *M, *V;            // fp32 moments, or
  uint8_t *Mc, *Vc;        // 8-bit codes with
  float *Mam, *Vam;        // one absmax per quantisation block
  void* Nout;              // normalised update (fp32 or bf16)
  int cols, r_ld, n_ld;    // state row length and the row pitches of Rpart / Nout (cols == 0: packed)
  int aligned16;           // set by adam_group_add: all arrays allow 16-byte vector accesses
  int first_block;         // the item covers the layer's work blocks from this one on (0: the whole layer)
  AdamParams p;
  int32_t* status;
};
constexpr int kAdamGroup = 32;
struct AdamGroup {
  AdamItem item[kAdamGroup];
  int block_end[kAdamGroup];   // running total of work blocks
  int count;
};
// all items of a group share the state format, the quantisation block and the dtype of N
galore_status_t adam_group_add(AdamGroup& g, const AdamItem& item, int32_t state_fmt, int q_block);
galore_status_t launch_adam_group(const AdamGroup& g, int32_t state_fmt, int q_block, int32_t n_dtype, cudaStream_t st);

// R arrives as `splits` fp32 partial sums, each `split_stride` elements apart.
galore_status_t launch_adam_f32(const float* Rpart, int splits, int64_t split_stride, int64_t nel, float* M,
                                float* V, void* Nout, int32_t n_dtype, const AdamParams& p, int32_t* status,
                                cudaStream_t st, const StateGeom& g = StateGeom());
galore_status_t launch_adam_q8(const float* Rpart, int splits, int64_t split_stride, int64_t nel, uint8_t* Mc,
                               float* Mam, uint8_t* Vc, float* Vam, int block, void* Nout, int32_t n_dtype,
                               const AdamParams& p, int32_t* status, cudaStream_t st,
                               const StateGeom& g = StateGeom());
galore_status_t launch_q8_quantize(const float* x, int64_t nel, int is_signed, int block, uint8_t* codes,
                                   float* absmax, cudaStream_t st);
galore_status_t launch_q8_dequantize(const uint8_t* codes, const float* absmax, int64_t nel, int is_signed,
                                     int block, float* out, cudaStream_t st);
galore_status_t q8_ensure_tables();
void q8_host_codebook(bool is_signed, float* out256);

}  // namespace galore
