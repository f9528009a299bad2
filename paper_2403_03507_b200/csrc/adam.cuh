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
