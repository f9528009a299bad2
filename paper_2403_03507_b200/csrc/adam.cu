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

#include <float.h>
#include <math.h>
#include <string.h>

#include <algorithm>
#include <memory>
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

// Tables in global memory (not __constant__): every thread reads its own entry when a CTA
// stages them in shared memory, which the constant cache would serialise.
__device__ float c_code_s[256];
__device__ float c_code_u[256];
__device__ float c_mid_s[256];   // 255 thresholds used
__device__ float c_mid_u[256];
__device__ uint32_t c_enc_s[3584];   // quantiser table, one entry per bin of |y| (see q8_encode_block)
__device__ uint32_t c_enc_u[3584];

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
  // Quantiser tables.  Bin `key` holds the non-negative floats whose upper 16 bits are
  // (kLutBase >> 16) + key (bin 0 also everything below 2^-27).  With c = number of thresholds below
  // the bin and t = lower 16 bits of the one threshold inside it (0xffff if none), the entry is
  // (c << 16) + (0x10000 - t): adding the lower 16 bits of a value of the bin carries into the upper
  // half exactly when the value is at or above the threshold.
  static uint32_t enc_s[3584], enc_u[3584];
  auto build_enc = [](const float* mids, uint32_t* enc) -> bool {
    uint32_t tb[255];
    int n_nonpos = 0, n_pos = 0;
    for (int i = 0; i < 255; ++i) {
      if (mids[i] > 0.f) memcpy(&tb[n_pos++], &mids[i], 4);     // ascending, positive: bit order = value order
      else ++n_nonpos;
    }
    for (int key = 0; key < 3584; ++key) {
      const uint32_t k = (uint32_t)std::min(key, 3456);
      const uint32_t hi = (0x32000000u >> 16) + k;
      uint32_t below = 0, thr = 0xffffu;
      int inside = 0;
      for (int i = 0; i < n_pos; ++i) {
        const uint32_t th = tb[i] >> 16;
        if (th < hi && k > 0) ++below;
        else if (th == hi || (k == 0 && th < hi)) { thr = tb[i] & 0xffffu; ++inside; }
      }
      if (inside > 1 || (inside == 1 && thr > 0xfff0u)) return false;
      enc[key] = (((uint32_t)n_nonpos + below) << 16) + (0x10000u - thr);
    }
    // a threshold within 8 ulp of its bin's lower edge needs a threshold-free bin below it, so that
    // values just under the edge are sent to the exact search by the 0xffff entry
    for (int key = 1; key <= 3456; ++key) {
      const uint32_t t_here = (0x10000u - (enc[key] & 0xffffu)) & 0xffffu;       // t = 0 is stored as 0
      if (t_here < 8u && (enc[key - 1] & 0xffffu) != 1u) return false;
    }
    return true;
  };
  if (!build_enc(ms, enc_s) || !build_enc(mu, enc_u)) return GALORE_ERR_STATE;
  GALORE_CUDA_TRY(cudaMemcpyToSymbol(c_enc_s, enc_s, sizeof(enc_s)));
  GALORE_CUDA_TRY(cudaMemcpyToSymbol(c_enc_u, enc_u, sizeof(enc_u)));
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

// Same code as q8_encode(fp32(x / absmax)) at a fraction of the cost.
//  1. y' = x * (1 / absmax) is within 2 ulp of the correctly rounded quotient q.
//  2. The upper 16 bits of |y'| (exponent and 7 mantissa bits) select a bin; the spacing of the
//     thresholds is wider than a bin, so a bin holds at most one.  The bin's table entry gives the
//     number of thresholds below the bin and the lower 16 bits of the threshold inside it
//     (0xffff if there is none); comparing those with the lower 16 bits of |y'| finishes the search
//     in integer arithmetic.
//  3. If |y'| is more than 8 ulp away from the bin's threshold, q lies on the same side of it and
//     the code is final.  Otherwise (also for the top 9 values of a bin without a threshold, which
//     covers a threshold at the lower edge of the next bin) the quotient is formed with IEEE
//     division and searched exactly.
//  Signed code: its thresholds are symmetric about zero except between -1e-6 and 1e-6, so a
//  negative y' takes 255 - (code of |y'|), and goes to the exact search below 2^-19.
constexpr int kLutSize = 3584;                 // keys 0 .. 3456 used
constexpr uint32_t kLutBase = 0x32000000u;     // bits of 2^-27: below it every value maps to key 0

// Fast part: the code of y' and whether it has to be confirmed by the exact search.
template <bool SIGNED>
__device__ __forceinline__ uint32_t q8_encode_fast(float x, float inv, const uint32_t* __restrict__ enc, bool& exact) {
  const float ya = x * inv;
  const uint32_t mag = SIGNED ? (__float_as_uint(ya) & 0x7fffffffu) : __float_as_uint(ya);   // unsigned code: y' >= 0
  const uint32_t b = max(mag, kLutBase + 0x8000u);      // everything below lands mid-bin in bin 0 (no threshold there)
  const uint32_t sum = enc[min((b - kLutBase) >> 16, 3456u)] + (b & 0xffffu);
  uint32_t idx = sum >> 16;
  exact = ((sum + 8u) & 0xffffu) <= 16u;          // within 8 ulp of the threshold (modulo 2^16: errs on the safe side)
  if (SIGNED && ya < 0.f) {
    idx = 255u - idx;
    exact |= b < 0x36000000u;
  }
  return idx;
}

template <bool SIGNED>
__device__ __forceinline__ int q8_encode_block(float x, float absmax, float inv, const uint32_t* __restrict__ enc,
                                               const float* __restrict__ mids) {
  bool exact;
  const uint32_t idx = q8_encode_fast<SIGNED>(x, inv, enc, exact);
  if (!exact) return (int)idx;
  return q8_encode(__fdiv_rn(x, absmax), mids);
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

// Eq. 15 with bias correction.  The square root and the quotient use the approximate hardware
// units (about 2 ulp each): N feeds a bf16 or fp32 GEMM operand and decides no integer.
__device__ __forceinline__ float adam_normalised(float m, float v, const AdamParams& p) {
  float root, inv;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(root) : "f"(v * p.inv_bc2));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(inv) : "f"(root + p.eps));
  return (m * p.inv_bc1) * inv;
}

// ---- grouped launches ------------------------------------------------------------
// Both kernels take a group of layers (AdamGroup, passed as kernel parameters) and walk the
// blocks of all of them with one persistent grid; a single layer is a group of one.

// `it` is a cursor: a CTA's work blocks come in ascending order, so the search resumes where the
// previous one ended (a group has up to 32 layers; a scan from the start for every block cost about
// as many instructions per element as the Adam arithmetic itself).
__device__ __forceinline__ void find_item(const AdamGroup& g, int gb, int& it, int& local) {
  while (it + 1 < g.count && gb >= g.block_end[it]) ++it;
  local = gb - (it > 0 ? g.block_end[it - 1] : 0) + g.item[it].first_block;
}

// ---- fp32 moments -------------------------------------------------------------
// work block = 2048 consecutive state elements, thread t owns t, t + 256, ...
template <typename TN, bool PACKED>
__device__ __forceinline__ bool adam_f32_block(const AdamItem& a, int blk) {
  constexpr int EPT = 8;
  const int base = blk * (EPT * 256) + threadIdx.x;
  const AdamParams p = a.p;
  float* __restrict__ M = a.M;
  float* __restrict__ V = a.V;
  TN* __restrict__ Nout = (TN*)a.Nout;
  int row = 0, col = 0;
  if (!PACKED) {
    row = base / a.cols;
    col = base - row * a.cols;
  }
  float r[EPT], m[EPT], v[EPT];
  int off_r[EPT], off_n[EPT];
#pragma unroll
  for (int e = 0; e < EPT; ++e) {
    const int i = base + e * 256;
    const bool ok = i < a.nel;
    off_r[e] = PACKED ? i : row * a.r_ld + col;
    off_n[e] = PACKED ? i : row * a.n_ld + col;
    r[e] = ok ? a.Rpart[off_r[e]] : 0.f;
    m[e] = ok ? M[i] : 0.f;
    v[e] = ok ? V[i] : 0.f;
    if (!PACKED) {
      col += 256;
      while (col >= a.cols) { col -= a.cols; ++row; }
    }
  }
  for (int s = 1; s < a.splits; ++s) {
    const float* part = a.Rpart + (int64_t)s * a.split_stride;
#pragma unroll
    for (int e = 0; e < EPT; ++e)
      if (base + e * 256 < a.nel) r[e] += part[off_r[e]];
  }
  bool bad = false;
#pragma unroll
  for (int e = 0; e < EPT; ++e) {
    const int i = base + e * 256;
    if (i < a.nel) {
      bad |= !isfinite(r[e]);
      const float mn = p.b1 * m[e] + p.omb1 * r[e];
      const float vn = p.b2 * v[e] + p.omb2 * (r[e] * r[e]);
      M[i] = mn;
      V[i] = vn;
      Nout[off_n[e]] = cvt<TN>(adam_normalised(mn, vn, p));
    }
  }
  return bad;
}

// ---- 8-bit block-wise moments ---------------------------------------------------
// A CTA walks quantisation blocks of EPT * 256 elements; within a block thread t owns
// elements t, t + 256, t + 512, ... so every warp-level access is one contiguous run
// whatever the alignment of the block.  PACKED: R partials and N have the state's own
// row pitch, so one flat index serves all arrays.
#ifndef GALORE_F32_CTAS
#define GALORE_F32_CTAS 3         // fp32-state kernel: 80 registers
#endif
#ifndef GALORE_Q8_FAST_CTAS
#define GALORE_Q8_FAST_CTAS 5     // the same for the kernel that holds the full-packed-block variant alone
#endif
#ifndef GALORE_Q8_PADDED_CTAS
#define GALORE_Q8_PADDED_CTAS 5   // and for the one that holds the full-padded-block variant alone
#endif
#ifndef GALORE_Q8_CTAS
#define GALORE_Q8_CTAS 4          // resident CTAs per SM the kernel is compiled for (register budget)
#endif
struct alignas(16) Q8Tables {
  float code_s[256], code_u[256], mid_s[256], mid_u[256];
  uint32_t enc_s[kLutSize], enc_u[kLutSize];
  float red[48];          // [0, 16): the one-value reductions; [16, 32) and [32, 48): the alternating two-value ones
};

template <typename TN, int EPT, bool PACKED>
__device__ __forceinline__ bool adam_q8_block(const AdamItem& a, int blk, Q8Tables& t) {
  constexpr int QB = EPT * 256;
  const int nel = a.nel;
  const AdamParams p = a.p;
  uint8_t* __restrict__ Mc = a.Mc;
  uint8_t* __restrict__ Vc = a.Vc;
  TN* __restrict__ Nout = (TN*)a.Nout;
  const int base = blk * QB + threadIdx.x;
  const float am_m = a.Mam[blk], am_v = a.Vam[blk];
  int row = 0, col = 0;
  if (!PACKED) {
    row = base / a.cols;
    col = base - row * a.cols;
  }
  // all loads of the block are issued before anything is used: the kernel lives on memory-level
  // parallelism (EPT * (splits + 2) independent requests per thread)
  float m[EPT], v[EPT], r[EPT];
  int off_r[EPT], off_n[EPT];          // positions in the (possibly padded) R and N buffers
  uint8_t cm[EPT], cv[EPT];
#pragma unroll
  for (int e = 0; e < EPT; ++e) {
    const int i = base + e * 256;
    const bool ok = i < nel;
    off_r[e] = PACKED ? i : row * a.r_ld + col;
    off_n[e] = PACKED ? i : row * a.n_ld + col;
    r[e] = ok ? a.Rpart[off_r[e]] : 0.f;
    cm[e] = ok ? Mc[i] : (uint8_t)127;
    cv[e] = ok ? Vc[i] : (uint8_t)0;
    if (!PACKED) {
      col += 256;
      while (col >= a.cols) { col -= a.cols; ++row; }
    }
  }
  for (int s = 1; s < a.splits; ++s) {
    const float* part = a.Rpart + (int64_t)s * a.split_stride;
#pragma unroll
    for (int e = 0; e < EPT; ++e)
      if (base + e * 256 < nel) r[e] += part[off_r[e]];
  }
  bool bad = false;
  float mx_m = 0.f, mx_v = 0.f;
#pragma unroll
  for (int e = 0; e < EPT; ++e) {
    const int i = base + e * 256;
    if (i < nel) {
      bad |= !isfinite(r[e]);
      const float m_old = t.code_s[cm[e]] * am_m;
      const float v_old = t.code_u[cv[e]] * am_v;
      m[e] = p.b1 * m_old + p.omb1 * r[e];
      v[e] = p.b2 * v_old + p.omb2 * (r[e] * r[e]);
      Nout[off_n[e]] = cvt<TN>(adam_normalised(m[e], v[e], p));
      mx_m = fmaxf(mx_m, fabsf(m[e]));
      mx_v = fmaxf(mx_v, v[e]);
    } else {
      m[e] = v[e] = 0.f;
    }
  }
  mx_m = block_max_256(mx_m, t.red);
  mx_v = block_max_256(mx_v, t.red);
  const float inv_m = 1.0f / mx_m, inv_v = 1.0f / mx_v;
#pragma unroll
  for (int e = 0; e < EPT; ++e) {
    const int i = base + e * 256;
    if (i < nel) {
      Mc[i] = (mx_m == 0.f) ? (uint8_t)127 : (uint8_t)q8_encode_block<true>(m[e], mx_m, inv_m, t.enc_s, t.mid_s);
      Vc[i] = (mx_v == 0.f) ? (uint8_t)0 : (uint8_t)q8_encode_block<false>(v[e], mx_v, inv_v, t.enc_u, t.mid_u);
    }
  }
  if (threadIdx.x == 0) {
    a.Mam[blk] = mx_m;
    a.Vam[blk] = mx_v;
  }
  return bad;
}

// max of two values over the CTA (256 threads) with a single barrier; every thread gets both.
// `red` is one of two alternating 16-float buffers: a buffer is written again two calls later, and
// the barrier of the call in between separates that from the last reads of this one.
__device__ __forceinline__ void block_max2_256(float& x, float& y, float* red /* 16 floats */) {
  x = warp_max(x);
  y = warp_max(y);
  if ((threadIdx.x & 31) == 0) {
    red[threadIdx.x >> 5] = x;
    red[8 + (threadIdx.x >> 5)] = y;
  }
  __syncthreads();
  const float4* __restrict__ q = reinterpret_cast<const float4*>(red);      // 16-byte aligned (Q8Tables)
  const float4 a = q[0], b = q[1], c = q[2], d = q[3];
  x = fmaxf(fmaxf(fmaxf(a.x, a.y), fmaxf(a.z, a.w)), fmaxf(fmaxf(b.x, b.y), fmaxf(b.z, b.w)));
  y = fmaxf(fmaxf(fmaxf(c.x, c.y), fmaxf(c.z, c.w)), fmaxf(fmaxf(d.x, d.y), fmaxf(d.z, d.w)));
}

// Full block of a layer whose R and N buffers have the state's own row pitch: every array is
// addressed as base pointer + constant offset, no bounds checks, and each thread owns runs of four
// consecutive elements (one 16-byte load of R, one 4-byte load / store per code array, one 8- or
// 16-byte store of N per run).  Run j of thread t starts at element 1024 j + 4 t of the block.
template <typename TN>
__device__ __forceinline__ void store_n4(TN* dst, float a, float b, float c, float d);
template <>
__device__ __forceinline__ void store_n4<__nv_bfloat16>(__nv_bfloat16* dst, float a, float b, float c, float d) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
  uint2 v;
  v.x = *reinterpret_cast<uint32_t*>(&lo);
  v.y = *reinterpret_cast<uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(dst) = v;
}
template <>
__device__ __forceinline__ void store_n4<float>(float* dst, float a, float b, float c, float d) {
  *reinterpret_cast<float4*>(dst) = make_float4(a, b, c, d);
}

// fp32 moments, full work block of a layer with packed, 16-byte aligned arrays: runs of four as
// below, every access a 16-byte one (8 bytes for a bf16 N)
template <typename TN>
__device__ __forceinline__ bool adam_f32_block_full(const AdamItem& a, int blk) {
  const AdamParams p = a.p;
  const int base = blk * 2048 + 4 * threadIdx.x;
  const float* __restrict__ R = a.Rpart + base;
  float* __restrict__ M = a.M + base;
  float* __restrict__ V = a.V + base;
  TN* __restrict__ Nout = (TN*)a.Nout + base;
  float4 r[2], m[2], v[2];
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    r[j] = *reinterpret_cast<const float4*>(R + j * 1024);
    m[j] = *reinterpret_cast<const float4*>(M + j * 1024);
    v[j] = *reinterpret_cast<const float4*>(V + j * 1024);
  }
  for (int s = 1; s < a.splits; ++s) {
    const float* __restrict__ part = R + (int64_t)s * a.split_stride;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const float4 q = *reinterpret_cast<const float4*>(part + j * 1024);
      r[j].x += q.x; r[j].y += q.y; r[j].z += q.z; r[j].w += q.w;
    }
  }
  uint32_t top = 0u;      // largest bit pattern among the new second moments (all >= 0): a non-finite r shows here
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    const float rr[4] = {r[j].x, r[j].y, r[j].z, r[j].w};
    const float mo[4] = {m[j].x, m[j].y, m[j].z, m[j].w};
    const float vo[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
    float mn[4], vn[4], nn[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      mn[k] = p.b1 * mo[k] + p.omb1 * rr[k];
      vn[k] = p.b2 * vo[k] + p.omb2 * (rr[k] * rr[k]);
      nn[k] = adam_normalised(mn[k], vn[k], p);
      top = max(top, __float_as_uint(vn[k]));
    }
    *reinterpret_cast<float4*>(M + j * 1024) = make_float4(mn[0], mn[1], mn[2], mn[3]);
    *reinterpret_cast<float4*>(V + j * 1024) = make_float4(vn[0], vn[1], vn[2], vn[3]);
    store_n4<TN>(Nout + j * 1024, nn[0], nn[1], nn[2], nn[3]);
  }
  return top >= 0x7f800000u;
}

template <typename TN>
__global__ void __launch_bounds__(256, GALORE_F32_CTAS) adam_f32_kernel(const __grid_constant__ AdamGroup g) {
  const int total = g.block_end[g.count - 1];
  int bad_item = -1, it = 0;
  for (int gb = blockIdx.x; gb < total; gb += gridDim.x) {
    int blk;
    find_item(g, gb, it, blk);
    const AdamItem& a = g.item[it];
    const bool packed = (a.r_ld == a.cols && a.n_ld == a.cols);
    const bool full = (blk + 1) * 2048 <= a.nel;
    const bool bad = (packed && full && a.aligned16) ? adam_f32_block_full<TN>(a, blk)
                     : packed                        ? adam_f32_block<TN, true>(a, blk)
                                                     : adam_f32_block<TN, false>(a, blk);
    if (bad) bad_item = it;
  }
  if (bad_item >= 0) atomicOr(g.item[bad_item].status, GALORE_DEV_NONFINITE);
}


// PADDED: R and N have rows of a.cols elements at pitches a.r_ld and a.n_ld (the state itself is
// always contiguous).  The codes keep their 4-byte accesses; the four R and N elements of a run are
// addressed one by one, and a run may continue on the next row.
template <typename TN, int EPT, bool PADDED>
__device__ __forceinline__ bool adam_q8_block_full(const AdamItem& a, int blk, Q8Tables& t, int parity) {
  static_assert(EPT % 4 == 0, "runs of four elements");
  constexpr int RUNS = EPT / 4;
  const AdamParams p = a.p;
  const int base = blk * (EPT * 256) + 4 * threadIdx.x;
  const float* __restrict__ R = a.Rpart + (PADDED ? 0 : base);
  uint8_t* __restrict__ Mc = a.Mc + base;
  uint8_t* __restrict__ Vc = a.Vc + base;
  TN* __restrict__ Nout = (TN*)a.Nout + (PADDED ? 0 : base);
  const float am_m = a.Mam[blk], am_v = a.Vam[blk];
  float4 r[RUNS];
  uint32_t cm[RUNS], cv[RUNS];
  int run_row[PADDED ? RUNS : 1], run_col[PADDED ? RUNS : 1];      // where each run starts
  if (PADDED) {
    int row = base / a.cols;
    int col = base - row * a.cols;
    const int adv_rows = 1024 / a.cols, adv_cols = 1024 - adv_rows * a.cols;   // from one run to the next
#pragma unroll
    for (int j = 0; j < RUNS; ++j) {
      run_row[j] = row;
      run_col[j] = col;
      row += adv_rows;
      col += adv_cols;
      if (col >= a.cols) { col -= a.cols; ++row; }
    }
  }
  // element k of run j in a buffer with row pitch ld
  auto at = [&](int j, int k, int ld) {
    const bool wrap = run_col[j] + k >= a.cols;
    return (run_row[j] + (wrap ? 1 : 0)) * ld + run_col[j] + k - (wrap ? a.cols : 0);
  };
  // a run that stays inside its row (all but one or two per row) is four consecutive elements of
  // the padded buffers as well
  auto load_run = [&](const float* __restrict__ src, int j) {
    if (run_col[j] + 3 < a.cols) {
      const float* __restrict__ q = src + run_row[j] * a.r_ld + run_col[j];
      return make_float4(q[0], q[1], q[2], q[3]);
    }
    return make_float4(src[at(j, 0, a.r_ld)], src[at(j, 1, a.r_ld)], src[at(j, 2, a.r_ld)], src[at(j, 3, a.r_ld)]);
  };
#pragma unroll
  for (int j = 0; j < RUNS; ++j) {
    if (PADDED) {
      r[j] = load_run(R, j);
    } else {
      r[j] = *reinterpret_cast<const float4*>(R + j * 1024);
    }
    cm[j] = *reinterpret_cast<const uint32_t*>(Mc + j * 1024);
    cv[j] = *reinterpret_cast<const uint32_t*>(Vc + j * 1024);
  }
  for (int s = 1; s < a.splits; ++s) {
    const float* __restrict__ part = R + (int64_t)s * a.split_stride;
#pragma unroll
    for (int j = 0; j < RUNS; ++j) {
      float4 q;
      if (PADDED) q = load_run(part, j);
      else q = *reinterpret_cast<const float4*>(part + j * 1024);
      r[j].x += q.x; r[j].y += q.y; r[j].z += q.z; r[j].w += q.w;
    }
  }
  float m[EPT], v[EPT];
  float mx_m = 0.f;
  uint32_t mx_v_bits = 0u;                       // v >= 0: the order of the bit patterns is the order of the values,
                                                 // and a NaN or an infinity (from a non-finite r) ends up on top
  const float c1 = p.b1 * am_m, c2 = p.b2 * am_v;
#pragma unroll
  for (int j = 0; j < RUNS; ++j) {
    const float rr[4] = {r[j].x, r[j].y, r[j].z, r[j].w};
    float nn[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int e = 4 * j + k;
      m[e] = fmaf(t.code_s[((cm[j] >> (8 * k)) & 0xffu)], c1, p.omb1 * rr[k]);
      v[e] = fmaf(t.code_u[((cv[j] >> (8 * k)) & 0xffu)], c2, p.omb2 * (rr[k] * rr[k]));
      nn[k] = adam_normalised(m[e], v[e], p);
      mx_m = fmaxf(mx_m, fabsf(m[e]));
      mx_v_bits = max(mx_v_bits, __float_as_uint(v[e]));
    }
    if (PADDED) {
      if (run_col[j] + 3 < a.cols) {
        TN* __restrict__ q = Nout + run_row[j] * a.n_ld + run_col[j];
#pragma unroll
        for (int k = 0; k < 4; ++k) q[k] = cvt<TN>(nn[k]);
      } else {
#pragma unroll
        for (int k = 0; k < 4; ++k) Nout[at(j, k, a.n_ld)] = cvt<TN>(nn[k]);
      }
    } else {
      store_n4<TN>(Nout + j * 1024, nn[0], nn[1], nn[2], nn[3]);
    }
  }
  const bool bad = mx_v_bits >= 0x7f800000u;
  float mx_v = __uint_as_float(mx_v_bits);
  block_max2_256(mx_m, mx_v, t.red + 16 + 16 * parity);
  // an all-zero block: with 0 in place of the reciprocal every y' is 0 and takes the code of zero
  const float inv_m = mx_m != 0.f ? 1.0f / mx_m : 0.f, inv_v = mx_v != 0.f ? 1.0f / mx_v : 0.f;
#pragma unroll
  for (int j = 0; j < RUNS; ++j) {
    uint32_t pm = 0u, pv = 0u;
    uint32_t need = 0u;                              // bit k: M value k of the run, bit 4 + k: V value k
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      bool ex;
      const uint32_t c = q8_encode_fast<true>(m[4 * j + k], inv_m, t.enc_s, ex) & 0xffu;
      pm |= c << (8 * k);
      need |= (ex ? 1u : 0u) << k;
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      bool ex;
      const uint32_t c = q8_encode_fast<false>(v[4 * j + k], inv_v, t.enc_u, ex) & 0xffu;
      pv |= c << (8 * k);
      need |= (ex ? 1u : 0u) << (4 + k);
    }
    // rare (about 1 value in 15 000): one branch for the eight values of the run
    if (need != 0u) {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (need & (1u << k)) {
          const uint32_t c = (uint32_t)q8_encode(__fdiv_rn(m[4 * j + k], mx_m), t.mid_s) & 0xffu;
          pm = (pm & ~(0xffu << (8 * k))) | (c << (8 * k));
        }
        if (need & (16u << k)) {
          const uint32_t c = (uint32_t)q8_encode(__fdiv_rn(v[4 * j + k], mx_v), t.mid_u) & 0xffu;
          pv = (pv & ~(0xffu << (8 * k))) | (c << (8 * k));
        }
      }
    }
    *reinterpret_cast<uint32_t*>(Mc + j * 1024) = pm;
    *reinterpret_cast<uint32_t*>(Vc + j * 1024) = pv;
  }
  if (threadIdx.x == 0) {
    a.Mam[blk] = mx_m;
    a.Vam[blk] = mx_v;
  }
  return bad;
}

// How a quantisation block is processed depends on its layer (row pitches, alignment) and on
// whether it is a full block.  A kernel compiled with every variant inlined needs the registers of
// the most demanding one and spills in all of them, so the kernel takes the set of variants it
// contains as a template argument; the launcher sorts the layers of a group into launches whose
// kernels contain what their blocks need.
enum : int {
  kBlockFullPacked = 1,    // full block, R and N at the state's own pitch, 16-byte aligned: vector accesses
  kBlockFullPadded = 2,    // full block, padded R / N rows
  kBlockAnyPacked = 4,     // tail block or unaligned arrays, packed
  kBlockAny = 8,           // tail block or unaligned arrays, padded rows
  kBlockAll = 15
};

template <int EPT>
__host__ __device__ __forceinline__ int q8_block_kind(const AdamItem& a, int blk) {
  const bool packed = (a.r_ld == a.cols && a.n_ld == a.cols);
  const bool full = (blk + 1) * (EPT * 256) <= a.nel;
  if (EPT % 4 == 0 && full && a.aligned16) {
    if (packed) return kBlockFullPacked;
    if (a.cols >= 4) return kBlockFullPadded;
  }
  return packed ? kBlockAnyPacked : kBlockAny;
}

constexpr int q8_ctas_per_sm(int kinds) {
  return kinds == kBlockFullPacked ? GALORE_Q8_FAST_CTAS : kinds == kBlockFullPadded ? GALORE_Q8_PADDED_CTAS : GALORE_Q8_CTAS;
}

template <typename TN, int EPT, int KINDS>
__global__ void __launch_bounds__(256, q8_ctas_per_sm(KINDS)) adam_q8_kernel(const __grid_constant__ AdamGroup g) {
  __shared__ Q8Tables t;
  // 32 KiB of tables per CTA: all loads in flight at once (one L2 round trip instead of fourteen)
  static_assert(kLutSize % 256 == 0, "whole rounds");
#pragma unroll
  for (int i = 0; i < kLutSize / 256; ++i) {
    t.enc_s[i * 256 + threadIdx.x] = c_enc_s[i * 256 + threadIdx.x];
    t.enc_u[i * 256 + threadIdx.x] = c_enc_u[i * 256 + threadIdx.x];
  }
  t.code_s[threadIdx.x] = c_code_s[threadIdx.x];
  t.code_u[threadIdx.x] = c_code_u[threadIdx.x];
  t.mid_s[threadIdx.x] = c_mid_s[threadIdx.x];
  t.mid_u[threadIdx.x] = c_mid_u[threadIdx.x];
  __syncthreads();

  const int total = g.block_end[g.count - 1];
  int bad_item = -1, it = 0;
  int parity = 0;
  for (int gb = blockIdx.x; gb < total; gb += gridDim.x, parity ^= 1) {
    int blk;
    find_item(g, gb, it, blk);
    const AdamItem& a = g.item[it];
    bool bad = false;
    if constexpr (KINDS == kBlockFullPacked || KINDS == kBlockFullPadded) {
      // never launched for EPT < 4
      if constexpr (EPT % 4 == 0) bad = adam_q8_block_full<TN, EPT, KINDS == kBlockFullPadded>(a, blk, t, parity);
    } else {
      const int kind = q8_block_kind<EPT>(a, blk);           // the same for every thread of the CTA
      if constexpr (EPT % 4 == 0 && (KINDS & kBlockFullPacked) != 0)
        if (kind == kBlockFullPacked) bad = adam_q8_block_full<TN, EPT, false>(a, blk, t, parity);
      if constexpr (EPT % 4 == 0 && (KINDS & kBlockFullPadded) != 0)
        if (kind == kBlockFullPadded) bad = adam_q8_block_full<TN, EPT, true>(a, blk, t, parity);
      if constexpr ((KINDS & kBlockAnyPacked) != 0)
        if (kind == kBlockAnyPacked) bad = adam_q8_block<TN, EPT, true>(a, blk, t);
      if constexpr ((KINDS & kBlockAny) != 0)
        if (kind == kBlockAny) bad = adam_q8_block<TN, EPT, false>(a, blk, t);
    }
    if (bad) bad_item = it;      // per thread: no barrier; a non-finite input is reported by the threads that met it
  }
  if (bad_item >= 0) atomicOr(g.item[bad_item].status, GALORE_DEV_NONFINITE);
}

// ---- stand-alone quantise / dequantise (same device code as the Adam kernel) ----
template <int EPT>
__global__ void __launch_bounds__(256)
q8_quantize_kernel(const float* __restrict__ x, int64_t nel, int is_signed, uint8_t* __restrict__ codes,
                   float* __restrict__ absmax) {
  __shared__ float s_mid[256];
  __shared__ uint32_t s_enc[kLutSize];
  __shared__ float red[8];
  for (int i = threadIdx.x; i < kLutSize; i += 256) s_enc[i] = is_signed ? c_enc_s[i] : c_enc_u[i];
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
  const float inv = 1.0f / mx;
#pragma unroll
  for (int e = 0; e < EPT; ++e) {
    int64_t i = base + (int64_t)e * 256;
    if (i < nel)
      codes[i] = (mx == 0.f) ? zero_code
                             : (uint8_t)(is_signed ? q8_encode_block<true>(val[e], mx, inv, s_enc, s_mid)
                                                   : q8_encode_block<false>(val[e], mx, inv, s_enc, s_mid));
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
// the variant the full blocks of a layer take (block 0 when the layer has a full block at all)
static int q8_item_kind(const AdamItem& a, int q_block) {
  switch (q_block) {
    case 256: return q8_block_kind<1>(a, 0);
    case 512: return q8_block_kind<2>(a, 0);
    case 1024: return q8_block_kind<4>(a, 0);
    case 2048: return q8_block_kind<8>(a, 0);
    default: return q8_block_kind<16>(a, 0);
  }
}

static bool valid_block(int block) {
  return block == 256 || block == 512 || block == 1024 || block == 2048 || block == 4096;
}

galore_status_t launch_adam_group(const AdamGroup& g, int32_t state_fmt, int q_block, int32_t n_dtype, cudaStream_t st) {
  if (g.count < 1 || g.count > kAdamGroup) return GALORE_ERR_INVALID_ARG;
  const int total = g.block_end[g.count - 1];
  if (total <= 0) return GALORE_OK;
  const unsigned grid = (unsigned)std::min(total, 148 * 8);
  const bool nb = n_dtype == GALORE_BF16;
  if (state_fmt == GALORE_STATE_F32) {
    if (nb) adam_f32_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(g);
    else adam_f32_kernel<float><<<grid, 256, 0, st>>>(g);
    GALORE_LAUNCH_CHECK();
    return GALORE_OK;
  }
  if (!valid_block(q_block)) return GALORE_ERR_INVALID_ARG;
  GALORE_TRY(q8_ensure_tables());
  // The full blocks of a layer go to the kernel that holds their variant alone (packed or padded
  // rows); tail blocks and layers with unaligned arrays go to the kernel that holds all variants.
  std::unique_ptr<AdamGroup> packed(new AdamGroup), padded(new AdamGroup), rest(new AdamGroup);
  packed->count = padded->count = rest->count = 0;
  auto append = [](AdamGroup& dst, const AdamItem& a, int first, int blocks) {
    if (blocks <= 0) return;
    const int j = dst.count++;
    dst.item[j] = a;
    dst.item[j].first_block = a.first_block + first;
    dst.block_end[j] = (j > 0 ? dst.block_end[j - 1] : 0) + blocks;
  };
  for (int i = 0; i < g.count; ++i) {
    const AdamItem& a = g.item[i];
    const int blocks = g.block_end[i] - (i > 0 ? g.block_end[i - 1] : 0);
    const int kind = q8_item_kind(a, q_block);
    // whole blocks among those the item covers (it covers the layer's blocks from first_block to the last)
    const int whole = std::min(blocks, std::max(0, a.nel / q_block - a.first_block));
    if (kind == kBlockFullPacked || kind == kBlockFullPadded) {
      append(kind == kBlockFullPacked ? *packed : *padded, a, 0, whole);
      append(*rest, a, whole, blocks - whole);
    } else {
      append(*rest, a, 0, blocks);
    }
  }
#define GALORE_Q8_LAUNCH(TN, EPT, KINDS, grp)                                                                 \
  do {                                                                                                       \
    GALORE_CUDA_TRY(cudaFuncSetAttribute(adam_q8_kernel<TN, EPT, KINDS>,                                     \
                                         cudaFuncAttributePreferredSharedMemoryCarveout,                     \
                                         cudaSharedmemCarveoutMaxShared)); /* several CTAs of 32 KiB of tables per SM */ \
    const int blocks_ = (grp).block_end[(grp).count - 1];                                                    \
    adam_q8_kernel<TN, EPT, KINDS><<<(unsigned)std::min(blocks_, 148 * q8_ctas_per_sm(KINDS)), 256, 0, st>>>(grp); /* one resident wave: tables are set up once per SM slot */ \
    GALORE_LAUNCH_CHECK();                                                                                   \
  } while (0)
#define GALORE_Q8_CASE(EPT)                                                            \
  case EPT * 256:                                                                      \
    if (packed->count > 0) {                                                           \
      if (nb) GALORE_Q8_LAUNCH(__nv_bfloat16, EPT, kBlockFullPacked, *packed);         \
      else GALORE_Q8_LAUNCH(float, EPT, kBlockFullPacked, *packed);                    \
    }                                                                                  \
    if (padded->count > 0) {                                                           \
      if (nb) GALORE_Q8_LAUNCH(__nv_bfloat16, EPT, kBlockFullPadded, *padded);         \
      else GALORE_Q8_LAUNCH(float, EPT, kBlockFullPadded, *padded);                    \
    }                                                                                  \
    if (rest->count > 0) {                                                             \
      if (nb) GALORE_Q8_LAUNCH(__nv_bfloat16, EPT, kBlockAll, *rest);                  \
      else GALORE_Q8_LAUNCH(float, EPT, kBlockAll, *rest);                             \
    }                                                                                  \
    break;
  switch (q_block) {
    GALORE_Q8_CASE(1) GALORE_Q8_CASE(2) GALORE_Q8_CASE(4) GALORE_Q8_CASE(8) GALORE_Q8_CASE(16)
    default: return GALORE_ERR_INVALID_ARG;
  }
#undef GALORE_Q8_CASE
#undef GALORE_Q8_LAUNCH
  return GALORE_OK;
}

galore_status_t adam_group_add(AdamGroup& g, const AdamItem& item, int32_t state_fmt, int q_block) {
  if (g.count >= kAdamGroup) return GALORE_ERR_BUFFER_TOO_SMALL;
  AdamItem a = item;
  if (a.cols == 0) a.cols = a.r_ld = a.n_ld = a.nel > 0 ? a.nel : 1;       // packed: one long row
  // 32-bit offsets inside the kernels: the padded buffers must stay below 2^31 elements
  const int64_t rows = ceil_div(a.nel, a.cols);
  if (rows * std::max(a.r_ld, a.n_ld) >= (int64_t)1 << 31) return GALORE_ERR_SHAPE;
  const int per_block = state_fmt == GALORE_STATE_F32 ? 2048 : q_block;
  a.aligned16 = ((((uintptr_t)a.Rpart | (uintptr_t)a.Nout | (uintptr_t)a.Mc | (uintptr_t)a.Vc | (uintptr_t)a.M |
                   (uintptr_t)a.V) & 15) == 0 &&
                 (a.split_stride % 4) == 0) ? 1 : 0;
  const int i = g.count++;
  g.item[i] = a;
  g.block_end[i] = (i > 0 ? g.block_end[i - 1] : 0) + (int)ceil_div(a.nel, per_block);
  return GALORE_OK;
}

static galore_status_t single(const AdamItem& a, int32_t state_fmt, int q_block, int32_t n_dtype, cudaStream_t st) {
  if (a.nel <= 0) return GALORE_OK;
  std::unique_ptr<AdamGroup> g(new AdamGroup);
  g->count = 0;
  GALORE_TRY(adam_group_add(*g, a, state_fmt, q_block));
  return launch_adam_group(*g, state_fmt, q_block, n_dtype, st);
}

galore_status_t launch_adam_f32(const float* Rpart, int splits, int64_t split_stride, int64_t nel, float* M,
                                float* V, void* Nout, int32_t n_dtype, const AdamParams& p, int32_t* status,
                                cudaStream_t st, const StateGeom& geo) {
  if (nel >= (int64_t)1 << 31) return GALORE_ERR_SHAPE;
  AdamItem a = {};
  a.Rpart = Rpart; a.splits = splits; a.split_stride = split_stride; a.nel = (int)nel;
  a.M = M; a.V = V; a.Nout = Nout; a.p = p; a.status = status;
  a.cols = (int)geo.cols; a.r_ld = (int)geo.r_ld; a.n_ld = (int)geo.n_ld;
  return single(a, GALORE_STATE_F32, 2048, n_dtype, st);
}

galore_status_t launch_adam_q8(const float* Rpart, int splits, int64_t split_stride, int64_t nel, uint8_t* Mc,
                               float* Mam, uint8_t* Vc, float* Vam, int block, void* Nout, int32_t n_dtype,
                               const AdamParams& p, int32_t* status, cudaStream_t st, const StateGeom& geo) {
  if (nel >= (int64_t)1 << 31) return GALORE_ERR_SHAPE;
  if (!valid_block(block)) return GALORE_ERR_INVALID_ARG;
  AdamItem a = {};
  a.Rpart = Rpart; a.splits = splits; a.split_stride = split_stride; a.nel = (int)nel;
  a.Mc = Mc; a.Mam = Mam; a.Vc = Vc; a.Vam = Vam; a.Nout = Nout; a.p = p; a.status = status;
  a.cols = (int)geo.cols; a.r_ld = (int)geo.r_ld; a.n_ld = (int)geo.n_ld;
  return single(a, GALORE_STATE_Q8_BLOCK, block, n_dtype, st);
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
