// Adafactor with first-order statistics on the compact gradient R (rows x cols):
//   v_row <- b2 v_row + (1 - b2) mean_j (R^2 + eps_1),  v_col likewise along columns,  b2 = 1 - t^-0.8
//   U = R / sqrt(v_row v_col^T / mean(v_row)),  U <- U / max(1, rms(U) / d)
//   M <- beta1 M + (1 - beta1) U,  N = M
// Four passes, each a plain streaming kernel, every reduction in a fixed order (run-to-run identical):
//   1. sums the split-K partials of R and leaves per-tile row and column sums of R^2,
//   2. folds those into v_row, v_col (one thread per entry), then the mean of v_row and the two factors
//      of 1 / sqrt(V) (one CTA per layer),
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
  float* a_row;      // rows: rsqrt(v_row / mean(v_row))
  float* b_col;      // cols: rsqrt(v_col)        (U = R a_row b_col^T)
  double* sums;      // kAfSumBlocks partial sums of U^2
  int tiles_r, tiles_c;
};
__host__ __device__ inline AfLayout af_layout(float* scratch, int rows, int cols) {
  AfLayout a;
  a.tiles_r = (rows + kAfTileRows - 1) / kAfTileRows;
  a.tiles_c = (cols + kAfTileCols - 1) / kAfTileCols;
  a.sums = reinterpret_cast<double*>(scratch);
  a.rowpart = scratch + 2 * (kAfSumBlocks + 8);
  // every section starts on a 16-byte boundary
  a.colpart = a.rowpart + ((size_t)rows * a.tiles_c + 3) / 4 * 4;
  a.a_row = a.colpart + ((size_t)a.tiles_r * cols + 3) / 4 * 4;
  a.b_col = a.a_row + (rows + 3) / 4 * 4;
  return a;
}

// pass 1: one CTA per 64 x 128 tile, thread c owns column c of the tile
// item whose running total first exceeds b, and b's position inside it
__device__ __forceinline__ int find_item(const int* end, int count, int b, int& local) {
  int i = 0;
  while (i + 1 < count && b >= end[i]) ++i;
  local = b - (i ? end[i - 1] : 0);
  return i;
}

// Warp w of the CTA takes the rows w, w + 4, ... of the tile; a lane holds four neighbouring columns
// (one 16-byte load when the rows allow it).  Row sums by warp shuffle, column sums in the lanes'
// registers, combined across the four warps in a fixed order.
__global__ void __launch_bounds__(kAfTileCols) af_stats_kernel(const __grid_constant__ AdafactorGroup g) {
  __shared__ float cs[kAfTileCols / 32][kAfTileCols];
  int tile;
  const AdafactorItem& it = g.item[find_item(g.tile_end, g.count, blockIdx.x, tile)];
  const AfLayout a = af_layout(it.scratch, it.rows, it.cols);
  const int tile_r = tile / a.tiles_c, tile_c = tile % a.tiles_c;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int r0 = tile_r * kAfTileRows, c0 = tile_c * kAfTileCols + 4 * lane;
  const bool vec = (it.r_ld % 4) == 0 && (it.split_stride % 4) == 0 && ((uintptr_t)it.Rpart & 15) == 0 && c0 + 3 < it.cols;
  float col[4] = {0.f, 0.f, 0.f, 0.f};
  // the four columns of one row: the sum of the K slices, written back when there are several
  auto load_row = [&](int row, float (&v)[4]) {
    v[0] = v[1] = v[2] = v[3] = 0.f;
    if (row >= it.rows) return;
    const int64_t at = (int64_t)row * it.r_ld + c0;
    if (vec) {
      float4 x = *reinterpret_cast<const float4*>(it.Rpart + at);
      for (int s = 1; s < it.splits; ++s) {
        const float4 y = *reinterpret_cast<const float4*>(it.Rpart + at + s * it.split_stride);
        x.x += y.x; x.y += y.y; x.z += y.z; x.w += y.w;
      }
      if (it.splits > 1) *reinterpret_cast<float4*>(it.Rpart + at) = x;
      v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
    } else {
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (c0 + k < it.cols) {
          float x = it.Rpart[at + k];
          for (int s = 1; s < it.splits; ++s) x += it.Rpart[at + k + s * it.split_stride];
          if (it.splits > 1) it.Rpart[at + k] = x;
          v[k] = x;
        }
    }
  };
  constexpr int kWarps = kAfTileCols / 32, kFlight = 4;      // four rows of a warp in flight
  for (int i = warp; i < kAfTileRows; i += kWarps * kFlight) {
    float v[kFlight][4];
#pragma unroll
    for (int u = 0; u < kFlight; ++u) load_row(r0 + i + u * kWarps, v[u]);
#pragma unroll
    for (int u = 0; u < kFlight; ++u) {
      const int row = r0 + i + u * kWarps;
      float row_sum = 0.f;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float sq = v[u][k] * v[u][k];
        col[k] += sq;
        row_sum += sq;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) row_sum += __shfl_xor_sync(0xffffffffu, row_sum, o);
      if (lane == 0 && row < it.rows) a.rowpart[(size_t)row * a.tiles_c + tile_c] = row_sum;
    }
  }
#pragma unroll
  for (int k = 0; k < 4; ++k) cs[warp][4 * lane + k] = col[k];
  __syncthreads();
  const int c = tile_c * kAfTileCols + threadIdx.x;
  if (c < it.cols) {
    float sum = 0.f;
#pragma unroll
    for (int w = 0; w < kAfTileCols / 32; ++w) sum += cs[w][threadIdx.x];
    a.colpart[(size_t)tile_r * it.cols + c] = sum;
  }
}

// pass 2a: entries 0 .. rows-1 are v_row, the next cols entries v_col
__global__ void __launch_bounds__(256) af_vectors_kernel(const __grid_constant__ AdafactorGroup g) {
  int blk;
  const int which = find_item(g.vec_end, g.count, blockIdx.x, blk);
  const AdafactorItem& it = g.item[which];
  const float beta2t = g.beta2t[which];
  const AfLayout a = af_layout(it.scratch, it.rows, it.cols);
  const int i = blk * 256 + threadIdx.x;
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
// pass 2b: the mean of v_row, then the two factors of 1 / sqrt(V): a_row = rsqrt(v_row / mean), b_col = rsqrt(v_col)
__global__ void __launch_bounds__(256) af_factors_kernel(const __grid_constant__ AdafactorGroup g) {
  __shared__ double red[8];
  const AdafactorItem& it = g.item[blockIdx.x];
  const AfLayout a = af_layout(it.scratch, it.rows, it.cols);
  double s = 0.0;
  for (int i = threadIdx.x; i < it.rows; i += 256) s += (double)it.v_row[i];
  s = block_sum_256d(s, red);
  const float mean_r = (float)(s / (double)it.rows);
  for (int i = threadIdx.x; i < it.rows; i += 256) a.a_row[i] = rsqrtf(it.v_row[i] / mean_r);
  for (int j = threadIdx.x; j < it.cols; j += 256) a.b_col[j] = rsqrtf(it.v_col[j]);
}

// rows of R in four-column groups where its rows are 16-byte aligned, the ragged end one by one
struct AfRowWalk {
  bool vec;
  int cols4;
};
__device__ __forceinline__ AfRowWalk af_walk(const AdafactorItem& it, bool with_state) {
  AfRowWalk w;
  w.vec = (it.r_ld % 4) == 0 && ((uintptr_t)it.Rpart & 15) == 0;
  if (with_state) w.vec = w.vec && (it.s_ld % 4) == 0 && (it.n_ld % 4) == 0 && ((uintptr_t)it.M & 15) == 0 && ((uintptr_t)it.Nout & 15) == 0;
  w.cols4 = w.vec ? (it.cols & ~3) : 0;
  return w;
}

// pass 3: partial sums of U^2, a fixed grid of 256-thread CTAs over the rows
__global__ void __launch_bounds__(256) af_rms_kernel(const __grid_constant__ AdafactorGroup g) {
  __shared__ double red[8];
  const AdafactorItem& it = g.item[blockIdx.y];
  const AfLayout a = af_layout(it.scratch, it.rows, it.cols);
  const AfRowWalk w = af_walk(it, false);
  double s = 0.0;
  for (int row = blockIdx.x; row < it.rows; row += gridDim.x) {
    const float ar = a.a_row[row];
    const float* R = it.Rpart + (int64_t)row * it.r_ld;
    float part = 0.f;                         // one row's share of one thread: at most a few dozen terms
    for (int c = 4 * threadIdx.x; c < w.cols4; c += 4 * 256) {
      const float4 x = *reinterpret_cast<const float4*>(R + c);
      const float4 b = *reinterpret_cast<const float4*>(a.b_col + c);
      const float u0 = x.x * ar * b.x, u1 = x.y * ar * b.y, u2 = x.z * ar * b.z, u3 = x.w * ar * b.w;
      part += u0 * u0 + u1 * u1 + u2 * u2 + u3 * u3;
    }
    for (int c = w.cols4 + threadIdx.x; c < it.cols; c += 256) {
      const float u = R[c] * ar * a.b_col[c];
      part += u * u;
    }
    s += (double)part;
  }
  s = block_sum_256d(s, red);
  if (threadIdx.x == 0) a.sums[blockIdx.x] = s;
}

template <typename TN>
__device__ __forceinline__ void af_store4(TN* dst, float m0, float m1, float m2, float m3);
template <>
__device__ __forceinline__ void af_store4<float>(float* dst, float m0, float m1, float m2, float m3) {
  *reinterpret_cast<float4*>(dst) = make_float4(m0, m1, m2, m3);
}
template <>
__device__ __forceinline__ void af_store4<__nv_bfloat16>(__nv_bfloat16* dst, float m0, float m1, float m2, float m3) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(m0, m1), hi = __floats2bfloat162_rn(m2, m3);
  uint2 v;
  v.x = *reinterpret_cast<uint32_t*>(&lo);
  v.y = *reinterpret_cast<uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(dst) = v;
}

// pass 4
template <typename TN>
__global__ void __launch_bounds__(256) af_update_kernel(const __grid_constant__ AdafactorGroup g) {
  __shared__ double red[8];
  const AdafactorItem& it = g.item[blockIdx.y];
  const AfLayout a = af_layout(it.scratch, it.rows, it.cols);
  double s = 0.0;
  for (int i = threadIdx.x; i < kAfSumBlocks; i += 256) s += a.sums[i];
  s = block_sum_256d(s, red);
  const float rms = (float)sqrt(s / ((double)it.rows * (double)it.cols));
  const float shrink = 1.f / fmaxf(1.f, rms / kAdafactorClip);
  const float b1 = it.beta1, omb1 = 1.f - it.beta1;
  const AfRowWalk w = af_walk(it, true);
  TN* N = reinterpret_cast<TN*>(it.Nout);
  for (int row = blockIdx.x; row < it.rows; row += gridDim.x) {
    const float ar = a.a_row[row] * shrink;
    const float* R = it.Rpart + (int64_t)row * it.r_ld;
    float* M = it.M + (int64_t)row * it.s_ld;
    TN* Nr = N + (int64_t)row * it.n_ld;
    for (int c = 4 * threadIdx.x; c < w.cols4; c += 4 * 256) {
      const float4 x = *reinterpret_cast<const float4*>(R + c);
      const float4 b = *reinterpret_cast<const float4*>(a.b_col + c);
      float4 m = *reinterpret_cast<const float4*>(M + c);
      m.x = fmaf(b1, m.x, omb1 * (x.x * ar * b.x));
      m.y = fmaf(b1, m.y, omb1 * (x.y * ar * b.y));
      m.z = fmaf(b1, m.z, omb1 * (x.z * ar * b.z));
      m.w = fmaf(b1, m.w, omb1 * (x.w * ar * b.w));
      *reinterpret_cast<float4*>(M + c) = m;
      af_store4<TN>(Nr + c, m.x, m.y, m.z, m.w);
    }
    for (int c = w.cols4 + threadIdx.x; c < it.cols; c += 256) {
      const float m = fmaf(b1, M[c], omb1 * (R[c] * ar * a.b_col[c]));
      M[c] = m;
      Nr[c] = cvt<TN>(m);
    }
  }
}

}  // namespace

size_t adafactor_scratch_bytes(int64_t rows, int64_t cols) {
  const int64_t tiles_r = ceil_div(rows, kAfTileRows), tiles_c = ceil_div(cols, kAfTileCols);
  return align_up((size_t)(2 * (kAfSumBlocks + 8) + rows * tiles_c + tiles_r * cols + rows + cols + 16) * sizeof(float), 256);
}

galore_status_t adafactor_group_add(AdafactorGroup& g, const AdafactorItem& it) {
  if (g.count >= kAdafactorGroup) return GALORE_ERR_INVALID_ARG;
  if (it.rows <= 0 || it.cols <= 0 || !it.Rpart || !it.M || !it.v_row || !it.v_col || !it.Nout || !it.scratch || it.splits < 1)
    return GALORE_ERR_INVALID_ARG;
  const int i = g.count;
  g.item[i] = it;
  g.beta2t[i] = (float)(1.0 - pow(it.t, -kAdafactorDecay));
  const int tiles = (int)(ceil_div(it.rows, kAfTileRows) * ceil_div(it.cols, kAfTileCols));
  const int blocks = (int)ceil_div(it.rows + it.cols, 256);
  g.tile_end[i] = (i ? g.tile_end[i - 1] : 0) + tiles;
  g.vec_end[i] = (i ? g.vec_end[i - 1] : 0) + blocks;
  g.count = i + 1;
  return GALORE_OK;
}

galore_status_t launch_adafactor_group(const AdafactorGroup& g, int32_t n_dtype, cudaStream_t st) {
  if (g.count <= 0) return GALORE_OK;
  const int n = g.count;
  af_stats_kernel<<<(unsigned)g.tile_end[n - 1], kAfTileCols, 0, st>>>(g);
  GALORE_LAUNCH_CHECK();
  af_vectors_kernel<<<(unsigned)g.vec_end[n - 1], 256, 0, st>>>(g);
  GALORE_LAUNCH_CHECK();
  af_factors_kernel<<<(unsigned)n, 256, 0, st>>>(g);
  GALORE_LAUNCH_CHECK();
  const dim3 grid(kAfSumBlocks, (unsigned)n);
  af_rms_kernel<<<grid, 256, 0, st>>>(g);
  GALORE_LAUNCH_CHECK();
  if (n_dtype == GALORE_BF16)
    af_update_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(g);
  else
    af_update_kernel<float><<<grid, 256, 0, st>>>(g);
  GALORE_LAUNCH_CHECK();
  return GALORE_OK;
}

galore_status_t launch_adafactor(const AdafactorItem& it, int32_t n_dtype, cudaStream_t st) {
  static thread_local AdafactorGroup g;
  g.count = 0;
  GALORE_TRY(adafactor_group_add(g, it));
  return launch_adafactor_group(g, n_dtype, st);
}

}  // namespace galore
