// Adam on the projected gradient R (Algorithm 1, the "update(R_t) by Adam"
// block, and Eq. 15), with fp32 or 8-bit block-wise moments (Sec. 4.3).
//
// Both kernels are streaming passes over the r x n (or m x r) state: they sum
// the split-K partials of R in a fixed order, update the stored (uncorrected)
// moments, and emit the normalised update N in the dtype the back-projection
// consumes.  The 8-bit kernel owns one quantisation block per CTA, so the
// block's absmax is a warp-shuffle + shared-memory reduction and the state
// makes exactly one round trip through HBM.
#include "adam.cuh"

#include <math.h>

#include <algorithm>
#include <mutex>
#include <vector>

namespace galore {

// ---- the 8-bit code -----------------------------------------------------------
// 256 ascending fp32 values per code.  Decade e holds 2^f linearly spaced
// magnitudes in (10^-(e+1), 10^-e]:  (2^f + 9 (j+1)) / (2^f 10^(e+1)),  f = top - e.
// Unsigned (second moment): top = 7, plus 0.  Signed (first moment): top = 6,
// both signs, 0, and one extra positive value 10^-7.
static void build_code(bool is_signed, float* out) {
  const int top = is_signed ? 6 : 7;
  std::vector<double> mags;
  for (int e = 0; e <= top; ++e) {
    const int f = top - e;
    double pow10 = 1.0;
    for (int q = 0; q < e + 1; ++q) pow10 *= 10.0;   // exact integers
    const double two_f = (double)(1 << f);
    for (int j = 0; j < (1 << f); ++j) mags.push_back((two_f + 9.0 * (j + 1)) / (two_f * pow10));
  }
  std::sort(mags.begin(), mags.end());
  std::vector<double> vals;
  if (is_signed) {
    for (auto it = mags.rbegin(); it != mags.rend(); ++it) vals.push_back(-*it);
    vals.push_back(0.0);
    vals.push_back(1.0 / 10000000.0);
    for (double v : mags) vals.push_back(v);
  } else {
    vals.push_back(0.0);
    for (double v : mags) vals.push_back(v);
  }
  for (int i = 0; i < 256; ++i) out[i] = (float)vals[i];
}

void q8_host_codebook(bool is_signed, float* out256) { build_code(is_signed, out256); }

__constant__ float c_code_s[256];
__constant__ float c_code_u[256];
__constant__ float c_mid_s[256];   // 255 thresholds used
__constant__ float c_mid_u[256];

static std::mutex g_code_mutex;
static bool g_code_ready[64] = {};

galore_status_t q8_ensure_tables() {
  int dev = 0;
  GALORE_CUDA_TRY(cudaGetDevice(&dev));
  std::lock_guard<std::mutex> lock(g_code_mutex);
  if (dev < 64 && g_code_ready[dev]) return GALORE_OK;
  float cs[256], cu[256], ms[256], mu[256];
  build_code(true, cs);
  build_code(false, cu);
  for (int i = 0; i < 255; ++i) {
    ms[i] = (float)(0.5 * ((double)cs[i] + (double)cs[i + 1]));
    mu[i] = (float)(0.5 * ((double)cu[i] + (double)cu[i + 1]));
  }
  ms[255] = mu[255] = INFINITY;
  GALORE_CUDA_TRY(cudaMemcpyToSymbol(c_code_s, cs, sizeof(cs)));
  GALORE_CUDA_TRY(cudaMemcpyToSymbol(c_code_u, cu, sizeof(cu)));
  GALORE_CUDA_TRY(cudaMemcpyToSymbol(c_mid_s, ms, sizeof(ms)));
  GALORE_CUDA_TRY(cudaMemcpyToSymbol(c_mid_u, mu, sizeof(mu)));
  if (dev < 64) g_code_ready[dev] = true;
  return GALORE_OK;
}

// number of thresholds <= y: nearest code value, ties to the larger index
__device__ __forceinline__ int q8_encode(float y, const float* __restrict__ mids) {
  int lo = 0, hi = 255;
#pragma unroll
  for (int s = 0; s < 8; ++s) {
    int mid = (lo + hi) >> 1;
    if (mids[mid] <= y) lo = mid + 1; else hi = mid;
  }
  return lo;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// max over the CTA (256 threads); every thread gets the result
__device__ __forceinline__ float block_max_256(float v, float* red /* >= 8 floats */) {
  v = warp_max(v);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = red[0];
#pragma unroll
  for (int w = 1; w < 8; ++w) r = fmaxf(r, red[w]);
  __syncthreads();
  return r;
}

template <typename TN>
__device__ __forceinline__ void store_n(TN* out, int64_t i, float v) { out[i] = cvt<TN>(v); }

__device__ __forceinline__ float adam_normalised(float m, float v, const AdamParams& p) {
  float mh = m * p.inv_bc1;
  float vh = v * p.inv_bc2;
  return mh / (sqrtf(vh) + p.eps);
}

// ---- fp32 moments -------------------------------------------------------------
template <typename TN>
__global__ void __launch_bounds__(256)
adam_f32_kernel(const float* __restrict__ Rpart, int splits, int64_t split_stride, int64_t nel,
                float* __restrict__ M, float* __restrict__ V, TN* __restrict__ Nout, AdamParams p,
                StateGeom g, int32_t* __restrict__ status) {
  bool bad = false;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nel; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t ir = g.r_index(i), in = g.n_index(i);
    float r = 0.f;
    for (int s = 0; s < splits; ++s) r += Rpart[(int64_t)s * split_stride + ir];
    bad |= !isfinite(r);
    float m = p.b1 * M[i] + p.omb1 * r;
    float v = p.b2 * V[i] + p.omb2 * (r * r);
    M[i] = m;
    V[i] = v;
    store_n(Nout, in, adam_normalised(m, v, p));
  }
  if (__syncthreads_or(bad) && threadIdx.x == 0) atomicOr(status, GALORE_DEV_NONFINITE);
}

// ---- 8-bit block-wise moments ---------------------------------------------------
// One CTA per quantisation block of EPT * 256 elements; thread t owns elements
// t, t + 256, t + 512, ... of the block, so every warp-level access is one
// contiguous run whatever the alignment of the block.
template <typename TN, int EPT>
__global__ void __launch_bounds__(256)
adam_q8_kernel(const float* __restrict__ Rpart, int splits, int64_t split_stride, int64_t nel,
               uint8_t* __restrict__ Mc, float* __restrict__ Mam, uint8_t* __restrict__ Vc,
               float* __restrict__ Vam, TN* __restrict__ Nout, AdamParams p, StateGeom g,
               int32_t* __restrict__ status) {
  __shared__ float s_code_s[256], s_code_u[256], s_mid_s[256], s_mid_u[256];
  __shared__ float red[8];
  s_code_s[threadIdx.x] = c_code_s[threadIdx.x];
  s_code_u[threadIdx.x] = c_code_u[threadIdx.x];
  s_mid_s[threadIdx.x] = c_mid_s[threadIdx.x];
  s_mid_u[threadIdx.x] = c_mid_u[threadIdx.x];
  __syncthreads();

  constexpr int QB = EPT * 256;
  const int64_t blk = blockIdx.x;
  const int64_t base = blk * QB + threadIdx.x;
  const float am_m = Mam[blk], am_v = Vam[blk];
  // position of the thread's first element in the padded R / N buffers; advanced by 256 per element
  const bool packed = (g.cols == 0) || (g.r_ld == g.cols && g.n_ld == g.cols);
  int64_t row = 0, col = 0;
  if (!packed) {
    row = base / g.cols;
    col = base - row * g.cols;
  }
  float m[EPT], v[EPT];
  bool bad = false;
  float mx_m = 0.f, mx_v = 0.f;
#pragma unroll
  for (int e = 0; e < EPT; ++e) {
    const int64_t i = base + (int64_t)e * 256;
    if (i < nel) {
      const int64_t ir = packed ? i : row * g.r_ld + col;
      const int64_t in = packed ? i : row * g.n_ld + col;
      float r = Rpart[ir];
      for (int s = 1; s < splits; ++s) r += Rpart[(int64_t)s * split_stride + ir];
      bad |= !isfinite(r);
      float m_old = s_code_s[Mc[i]] * am_m;
      float v_old = s_code_u[Vc[i]] * am_v;
      m[e] = p.b1 * m_old + p.omb1 * r;
      v[e] = p.b2 * v_old + p.omb2 * (r * r);
      store_n(Nout, in, adam_normalised(m[e], v[e], p));
      mx_m = fmaxf(mx_m, fabsf(m[e]));
      mx_v = fmaxf(mx_v, fabsf(v[e]));
    } else {
      m[e] = v[e] = 0.f;
    }
    if (!packed) {
      col += 256;
      while (col >= g.cols) { col -= g.cols; ++row; }
    }
  }
  mx_m = block_max_256(mx_m, red);
  mx_v = block_max_256(mx_v, red);
#pragma unroll
  for (int e = 0; e < EPT; ++e) {
    const int64_t i = base + (int64_t)e * 256;
    if (i < nel) {
      Mc[i] = (mx_m == 0.f) ? (uint8_t)127 : (uint8_t)q8_encode(__fdiv_rn(m[e], mx_m), s_mid_s);
      Vc[i] = (mx_v == 0.f) ? (uint8_t)0 : (uint8_t)q8_encode(__fdiv_rn(v[e], mx_v), s_mid_u);
    }
  }
  if (threadIdx.x == 0) {
    Mam[blk] = mx_m;
    Vam[blk] = mx_v;
  }
  if (__syncthreads_or(bad) && threadIdx.x == 0) atomicOr(status, GALORE_DEV_NONFINITE);
}

// ---- stand-alone quantise / dequantise (same device code as the Adam kernel) ----
template <int EPT>
__global__ void __launch_bounds__(256)
q8_quantize_kernel(const float* __restrict__ x, int64_t nel, int is_signed, uint8_t* __restrict__ codes,
                   float* __restrict__ absmax) {
  __shared__ float s_mid[256];
  __shared__ float red[8];
  s_mid[threadIdx.x] = is_signed ? c_mid_s[threadIdx.x] : c_mid_u[threadIdx.x];
  __syncthreads();
  constexpr int QB = EPT * 256;
  const int64_t blk = blockIdx.x;
  const int64_t base = blk * QB + threadIdx.x;
  float val[EPT];
  float mx = 0.f;
#pragma unroll
  for (int e = 0; e < EPT; ++e) {
    int64_t i = base + (int64_t)e * 256;
    val[e] = (i < nel) ? x[i] : 0.f;
    mx = fmaxf(mx, fabsf(val[e]));
  }
  mx = block_max_256(mx, red);
  const uint8_t zero_code = is_signed ? 127 : 0;
#pragma unroll
  for (int e = 0; e < EPT; ++e) {
    int64_t i = base + (int64_t)e * 256;
    if (i < nel) codes[i] = (mx == 0.f) ? zero_code : (uint8_t)q8_encode(__fdiv_rn(val[e], mx), s_mid);
  }
  if (threadIdx.x == 0) absmax[blk] = mx;
}

__global__ void __launch_bounds__(256)
q8_dequantize_kernel(const uint8_t* __restrict__ codes, const float* __restrict__ absmax, int64_t nel,
                     int is_signed, int block, float* __restrict__ out) {
  __shared__ float s_code[256];
  s_code[threadIdx.x] = is_signed ? c_code_s[threadIdx.x] : c_code_u[threadIdx.x];
  __syncthreads();
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nel; i += (int64_t)gridDim.x * blockDim.x)
    out[i] = s_code[codes[i]] * absmax[i / block];
}

// ---- launchers --------------------------------------------------------------------
static bool valid_block(int block) {
  return block == 256 || block == 512 || block == 1024 || block == 2048 || block == 4096;
}

template <typename TN>
static galore_status_t adam_f32_t(const float* Rpart, int splits, int64_t split_stride, int64_t nel, float* M,
                                  float* V, TN* Nout, const AdamParams& p, const StateGeom& g, int32_t* status,
                                  cudaStream_t st) {
  int64_t blocks = std::min<int64_t>(ceil_div(nel, 256), 148 * 16);
  adam_f32_kernel<TN><<<(unsigned)blocks, 256, 0, st>>>(Rpart, splits, split_stride, nel, M, V, Nout, p, g, status);
  GALORE_LAUNCH_CHECK();
  return GALORE_OK;
}

galore_status_t launch_adam_f32(const float* Rpart, int splits, int64_t split_stride, int64_t nel, float* M,
                                float* V, void* Nout, int32_t n_dtype, const AdamParams& p, int32_t* status,
                                cudaStream_t st, const StateGeom& g) {
  if (nel <= 0) return GALORE_OK;
  if (n_dtype == GALORE_BF16)
    return adam_f32_t(Rpart, splits, split_stride, nel, M, V, (__nv_bfloat16*)Nout, p, g, status, st);
  return adam_f32_t(Rpart, splits, split_stride, nel, M, V, (float*)Nout, p, g, status, st);
}

template <typename TN>
static galore_status_t adam_q8_t(const float* Rpart, int splits, int64_t split_stride, int64_t nel, uint8_t* Mc,
                                 float* Mam, uint8_t* Vc, float* Vam, int block, TN* Nout, const AdamParams& p,
                                 const StateGeom& g, int32_t* status, cudaStream_t st) {
  unsigned grid = (unsigned)ceil_div(nel, block);
#define GALORE_Q8_CASE(EPT)                                                                              \
  case EPT * 256:                                                                                        \
    adam_q8_kernel<TN, EPT><<<grid, 256, 0, st>>>(Rpart, splits, split_stride, nel, Mc, Mam, Vc, Vam,    \
                                                   Nout, p, g, status);                                  \
    break;
  switch (block) {
    GALORE_Q8_CASE(1) GALORE_Q8_CASE(2) GALORE_Q8_CASE(4) GALORE_Q8_CASE(8) GALORE_Q8_CASE(16)
    default: return GALORE_ERR_INVALID_ARG;
  }
#undef GALORE_Q8_CASE
  GALORE_LAUNCH_CHECK();
  return GALORE_OK;
}

galore_status_t launch_adam_q8(const float* Rpart, int splits, int64_t split_stride, int64_t nel, uint8_t* Mc,
                               float* Mam, uint8_t* Vc, float* Vam, int block, void* Nout, int32_t n_dtype,
                               const AdamParams& p, int32_t* status, cudaStream_t st, const StateGeom& g) {
  if (nel <= 0) return GALORE_OK;
  if (!valid_block(block)) return GALORE_ERR_INVALID_ARG;
  GALORE_TRY(q8_ensure_tables());
  if (n_dtype == GALORE_BF16)
    return adam_q8_t(Rpart, splits, split_stride, nel, Mc, Mam, Vc, Vam, block, (__nv_bfloat16*)Nout, p, g, status, st);
  return adam_q8_t(Rpart, splits, split_stride, nel, Mc, Mam, Vc, Vam, block, (float*)Nout, p, g, status, st);
}

galore_status_t launch_q8_quantize(const float* x, int64_t nel, int is_signed, int block, uint8_t* codes,
                                   float* absmax, cudaStream_t st) {
  if (nel <= 0) return GALORE_OK;
  if (!valid_block(block)) return GALORE_ERR_INVALID_ARG;
  GALORE_TRY(q8_ensure_tables());
  unsigned grid = (unsigned)ceil_div(nel, block);
  switch (block) {
    case 256: q8_quantize_kernel<1><<<grid, 256, 0, st>>>(x, nel, is_signed, codes, absmax); break;
    case 512: q8_quantize_kernel<2><<<grid, 256, 0, st>>>(x, nel, is_signed, codes, absmax); break;
    case 1024: q8_quantize_kernel<4><<<grid, 256, 0, st>>>(x, nel, is_signed, codes, absmax); break;
    case 2048: q8_quantize_kernel<8><<<grid, 256, 0, st>>>(x, nel, is_signed, codes, absmax); break;
    default: q8_quantize_kernel<16><<<grid, 256, 0, st>>>(x, nel, is_signed, codes, absmax); break;
  }
  GALORE_LAUNCH_CHECK();
  return GALORE_OK;
}

galore_status_t launch_q8_dequantize(const uint8_t* codes, const float* absmax, int64_t nel, int is_signed,
                                     int block, float* out, cudaStream_t st) {
  if (nel <= 0) return GALORE_OK;
  if (!valid_block(block)) return GALORE_ERR_INVALID_ARG;
  GALORE_TRY(q8_ensure_tables());
  int64_t blocks = std::min<int64_t>(ceil_div(nel, 256), 148 * 16);
  q8_dequantize_kernel<<<(unsigned)blocks, 256, 0, st>>>(codes, absmax, nel, is_signed, block, out);
  GALORE_LAUNCH_CHECK();
  return GALORE_OK;
}

}  // namespace galore
