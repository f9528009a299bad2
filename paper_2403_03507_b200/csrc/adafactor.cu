// Adafactor with first-order statistics on the compact gradient R (rows x cols):
//   v_row <- b2 v_row + (1 - b2) mean_j (R^2 + eps_1),  v_col likewise along columns,  b2 = 1 - t^-0.8
//   U = R / sqrt(v_row v_col^T / mean(v_row)),  U <- U / max(1, rms(U) / d)
//   M <- beta1 M + (1 - beta1) U,  N = M
// Four passes, each a plain streaming kernel, every reduction in a fixed order (run-to-run identical):
//   1. sums the split-K partials of R and leaves per-tile row and column sums of R^2,
//   2. folds those into v_row, v_col (one thread per entry), then the mean of v_row (one CTA),
//   3. sum of U^2 over a fixed grid,
//   4. the clipped update, the momentum and N.
// R is r x n (or m x r) fp32, a small matrix beside G and W; the passes are bound by its HBM traffic.
#include "adafactor.cuh"

#include <cuda_bf16.h>

namespace galore {
namespace {

__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
// every thread of a 256-thread CTA gets the sum
__device__ __forceinline__ double block_sum_256d(double v, double* red) {
  v = warp_sum_d(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  double s = 0.0;
#pragma unroll
  for (int i = 0; i < 8; ++i) s += red[i];
  return s;
}

struct AfLayout {
  float* rowpart;    // rows x tiles_c
  float* colpart;    // tiles_r x cols
  double* sums;      // kAfSumBlocks partial sums of U^2, then [kAfSumBlocks] = mean of v_row
  int tiles_r, tiles_c;
};
__host__ __device__ inline AfLayout af_layout(float* scratch, int rows, int cols) {
  AfLayout a;
  a.tiles_r = (rows + kAfTileRows - 1) / kAfTileRows;
  a.tiles_c = (cols + kAfTileCols - 1) / kAfTileCols;
  a.sums = reinterpret_cast<double*>(scratch);
  a.rowpart = scratch + 2 * (kAfSumBlocks + 8);
  a.colpart = a.rowpart + (size_t)rows * a.tiles_c;
  return a;
}

// pass 1: one CTA per 64 x 128 tile, thread c owns column c of the tile
__global__ void __launch_bounds__(kAfTileCols) af_stats_kernel(AdafactorItem it) {
  __shared__ float rs[kAfTileCols / 32][kAfTileRows];
  const AfLayout a = af_layout(it.scratch, it.rows, it.cols);
  const int r0 = blockIdx.y * kAfTileRows, c = blockIdx.x * kAfTileCols + threadIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const bool in_c = c < it.cols;
  float col_sum = 0.f;
  for (int i = 0; i < kAfTileRows; ++i) {
    const int row = r0 + i;
    float sq = 0.f;
    if (row < it.rows && in_c) {
      const int64_t at = (int64_t)row * it.r_ld + c;
      float v = it.Rpart[at];
      for (int s = 1; s < it.splits; ++s) v += it.Rpart[at + s * it.split_stride];
      if (it.splits > 1) it.Rpart[at] = v;
      sq = v * v;
    }
    col_sum += sq;
    float row_sum = sq;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) row_sum += __shfl_xor_sync(0xffffffffu, row_sum, o);
    if (lane == 0) rs[warp][i] = row_sum;
  }
  if (in_c) a.colpart[(size_t)blockIdx.y * it.cols + c] = col_sum;
  __syncthreads();
  if (threadIdx.x < kAfTileRows && r0 + threadIdx.x < it.rows) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < kAfTileCols / 32; ++w) s += rs[w][threadIdx.x];
    a.rowpart[(size_t)(r0 + threadIdx.x) * a.tiles_c + blockIdx.x] = s;
  }
}

// pass 2a: entries 0 .. rows-1 are v_row, the next cols entries v_col
__global__ void af_vectors_kernel(AdafactorItem it, float beta2t) {
  const AfLayout a = af_layout(it.scratch, it.rows, it.cols);
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < it.rows) {
    double s = 0.0;
    for (int tc = 0; tc < a.tiles_c; ++tc) s += (double)a.rowpart[(size_t)i * a.tiles_c + tc];
    const float mean = (float)(s / (double)it.cols) + kAdafactorEps1;
    it.v_row[i] = fmaf(beta2t, it.v_row[i], (1.f - beta2t) * mean);
  } else if (i < it.rows + it.cols) {
    const int j = i - it.rows;
    double s = 0.0;
    for (int tr = 0; tr < a.tiles_r; ++tr) s += (double)a.colpart[(size_t)tr * it.cols + j];
    const float mean = (float)(s / (double)it.rows) + kAdafactorEps1;
    it.v_col[j] = fmaf(beta2t, it.v_col[j], (1.f - beta2t) * mean);
  }
}
// pass 2b: mean of v_row
__global__ void __launch_bounds__(256) af_row_mean_kernel(AdafactorItem it) {
  __shared__ double red[8];
  const AfLayout a = af_layout(it.scratch, it.rows, it.cols);
  double s = 0.0;
  for (int i = threadIdx.x; i < it.rows; i += 256) s += (double)it.v_row[i];
  s = block_sum_256d(s, red);
  if (threadIdx.x == 0) a.sums[kAfSumBlocks] = s / (double)it.rows;
}

// U^2 = R^2 mean(v_row) / (v_row v_col)
__device__ __forceinline__ float af_inv_root(float vr, float vc, float mean_r) { return rsqrtf(vr * vc / mean_r); }

// pass 3: partial sums of U^2, a fixed grid of 256-thread CTAs over the rows
__global__ void __launch_bounds__(256) af_rms_kernel(AdafactorItem it) {
  __shared__ double red[8];
  const AfLayout a = af_layout(it.scratch, it.rows, it.cols);
  const float mean_r = (float)a.sums[kAfSumBlocks];
  double s = 0.0;
  for (int row = blockIdx.x; row < it.rows; row += gridDim.x) {
    const float vr = it.v_row[row];
    const float* R = it.Rpart + (int64_t)row * it.r_ld;
    for (int c = threadIdx.x; c < it.cols; c += 256) {
      const float u = R[c] * af_inv_root(vr, it.v_col[c], mean_r);
      s += (double)u * (double)u;
    }
  }
  s = block_sum_256d(s, red);
  if (threadIdx.x == 0) a.sums[blockIdx.x] = s;
}

// pass 4
template <typename TN>
__global__ void __launch_bounds__(256) af_update_kernel(AdafactorItem it) {
  __shared__ double red[8];
  const AfLayout a = af_layout(it.scratch, it.rows, it.cols);
  double s = 0.0;
  for (int i = threadIdx.x; i < kAfSumBlocks; i += 256) s += a.sums[i];
  s = block_sum_256d(s, red);
  const float rms = (float)sqrt(s / ((double)it.rows * (double)it.cols));
  const float shrink = 1.f / fmaxf(1.f, rms / kAdafactorClip);
  const float mean_r = (float)a.sums[kAfSumBlocks];
  const float b1 = it.beta1, omb1 = 1.f - it.beta1;
  TN* N = reinterpret_cast<TN*>(it.Nout);
  for (int row = blockIdx.x; row < it.rows; row += gridDim.x) {
    const float vr = it.v_row[row];
    const float* R = it.Rpart + (int64_t)row * it.r_ld;
    float* M = it.M + (int64_t)row * it.s_ld;
    TN* Nr = N + (int64_t)row * it.n_ld;
    for (int c = threadIdx.x; c < it.cols; c += 256) {
      const float u = R[c] * af_inv_root(vr, it.v_col[c], mean_r) * shrink;
      const float m = fmaf(b1, M[c], omb1 * u);
      M[c] = m;
      Nr[c] = cvt<TN>(m);
    }
  }
}

}  // namespace

size_t adafactor_scratch_bytes(int64_t rows, int64_t cols) {
  const int64_t tiles_r = ceil_div(rows, kAfTileRows), tiles_c = ceil_div(cols, kAfTileCols);
  return align_up((size_t)(2 * (kAfSumBlocks + 8) + rows * tiles_c + tiles_r * cols) * sizeof(float), 256);
}

galore_status_t launch_adafactor(const AdafactorItem& it, int32_t n_dtype, cudaStream_t st) {
  if (it.rows <= 0 || it.cols <= 0) return GALORE_OK;
  if (!it.Rpart || !it.M || !it.v_row || !it.v_col || !it.Nout || !it.scratch || it.splits < 1) return GALORE_ERR_INVALID_ARG;
  const float beta2t = (float)(1.0 - pow(it.t, -kAdafactorDecay));
  const dim3 tiles((unsigned)ceil_div(it.cols, kAfTileCols), (unsigned)ceil_div(it.rows, kAfTileRows));
  af_stats_kernel<<<tiles, kAfTileCols, 0, st>>>(it);
  GALORE_LAUNCH_CHECK();
  af_vectors_kernel<<<(unsigned)ceil_div(it.rows + it.cols, 256), 256, 0, st>>>(it, beta2t);
  GALORE_LAUNCH_CHECK();
  af_row_mean_kernel<<<1, 256, 0, st>>>(it);
  GALORE_LAUNCH_CHECK();
  af_rms_kernel<<<kAfSumBlocks, 256, 0, st>>>(it);
  GALORE_LAUNCH_CHECK();
  if (n_dtype == GALORE_BF16)
    af_update_kernel<__nv_bfloat16><<<kAfSumBlocks, 256, 0, st>>>(it);
  else
    af_update_kernel<float><<<kAfSumBlocks, 256, 0, st>>>(it);
  GALORE_LAUNCH_CHECK();
  return GALORE_OK;
}

}  // namespace galore
