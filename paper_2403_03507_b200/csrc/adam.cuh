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

// R arrives as `splits` fp32 partial sums, each `split_stride` elements apart.
galore_status_t launch_adam_f32(const float* Rpart, int splits, int64_t split_stride, int64_t nel, float* M,
                                float* V, void* Nout, int32_t n_dtype, const AdamParams& p, int32_t* status,
                                cudaStream_t st);
galore_status_t launch_adam_q8(const float* Rpart, int splits, int64_t split_stride, int64_t nel, uint8_t* Mc,
                               float* Mam, uint8_t* Vc, float* Vam, int block, void* Nout, int32_t n_dtype,
                               const AdamParams& p, int32_t* status, cudaStream_t st);
galore_status_t launch_q8_quantize(const float* x, int64_t nel, int is_signed, int block, uint8_t* codes,
                                   float* absmax, cudaStream_t st);
galore_status_t launch_q8_dequantize(const uint8_t* codes, const float* absmax, int64_t nel, int is_signed,
                                     int block, float* out, cudaStream_t st);
galore_status_t q8_ensure_tables();
void q8_host_codebook(bool is_signed, float* out256);

}  // namespace galore
