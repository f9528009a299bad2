// Adam on the projected gradient R (Algorithm 1, the "update(R_t) by Adam"
// block, and Eq. 15), with fp32 or 8-bit block-wise moments (Sec. 4.3).
//
// These kernels are streaming passes over the r x n (or m x r) state for the
// cases where Adam does not run inside the projection kernel (fp32 path, K
// sliced over CTAs): they sum the split-K partials of R in a fixed order,
// update the stored (uncorrected) moments, and emit the normalised update N
// in the dtype the back-projection consumes.  A CTA handles one tile of
// tile_rows x 64 state elements at a time; for 8-bit moments that tile is
// the quantisation block, so the block's absmax is a warp-shuffle +
// shared-memory reduction and the state makes one round trip through HBM.
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


galore_status_t q8_table_ptrs(Q8TablePtrs* out) {
  GALORE_TRY(q8_ensure_tables());
  void *cs, *cu, *ms, *mu, *es, *eu;
  GALORE_CUDA_TRY(cudaGetSymbolAddress(&cs, c_code_s));
  GALORE_CUDA_TRY(cudaGetSymbolAddress(&cu, c_code_u));
  GALORE_CUDA_TRY(cudaGetSymbolAddress(&ms, c_mid_s));
  GALORE_CUDA_TRY(cudaGetSymbolAddress(&mu, c_mid_u));
  GALORE_CUDA_TRY(cudaGetSymbolAddress(&es, c_enc_s));
  GALORE_CUDA_TRY(cudaGetSymbolAddress(&eu, c_enc_u));
  out->code_s = (const float*)cs; out->code_u = (const float*)cu;
  out->mid_s = (const float*)ms; out->mid_u = (const float*)mu;
  out->enc_s = (const uint32_t*)es; out->enc_u = (const uint32_t*)eu;
  return GALORE_OK;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// max of two values over the CTA (256 threads) with a single barrier; every thread gets both.
// `red` is one of two alternating 16-float buffers: a buffer is written again two calls later, and
// the barrier of the call in between separates that from the last reads of this one.
// x and y are bit patterns of non-negative floats (their order is the order of the values): one
// hardware warp reduction each, the eight warps' results through shared memory, one more reduction.
__device__ __forceinline__ void block_max2_256(uint32_t& x, uint32_t& y, float* red /* 16 floats */) {
  uint2* __restrict__ slots = reinterpret_cast<uint2*>(red);                 // 8-byte aligned (Q8Tables)
  x = __reduce_max_sync(0xffffffffu, x);
  y = __reduce_max_sync(0xffffffffu, y);
  if ((threadIdx.x & 31) == 0) slots[threadIdx.x >> 5] = make_uint2(x, y);
  __syncthreads();
  const uint2 v = slots[threadIdx.x & 7];
  x = __reduce_max_sync(0xffffffffu, v.x);
  y = __reduce_max_sync(0xffffffffu, v.y);
}

// BYTES (a power of two) from src to dst, both aligned to min(BYTES, 16): one access up to 16 bytes
template <int BYTES>
__device__ __forceinline__ void copy_vec(void* dst, const void* src) {
  if constexpr (BYTES >= 16) {
#pragma unroll
    for (int i = 0; i < BYTES / 16; ++i) reinterpret_cast<uint4*>(dst)[i] = reinterpret_cast<const uint4*>(src)[i];
  } else if constexpr (BYTES == 8) {
    *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(src);
  } else if constexpr (BYTES == 4) {
    *reinterpret_cast<uint32_t*>(dst) = *reinterpret_cast<const uint32_t*>(src);
  } else if constexpr (BYTES == 2) {
    *reinterpret_cast<uint16_t*>(dst) = *reinterpret_cast<const uint16_t*>(src);
  } else {
    *reinterpret_cast<uint8_t*>(dst) = *reinterpret_cast<const uint8_t*>(src);
  }
}

// ---- grouped launches ------------------------------------------------------------
// The kernels take a group of layers (AdamGroup, passed as kernel parameters) and walk the tiles of
// all of them with one persistent grid; a single layer is a group of one.

// `it` is a cursor: a CTA's tiles come in ascending order, so the search resumes where the previous
// one ended.
__device__ __forceinline__ void find_item(const AdamGroup& g, int gb, int& it, int& local) {
  while (it + 1 < g.count && gb >= g.block_end[it]) ++it;
  local = gb - (it > 0 ? g.block_end[it - 1] : 0);
}

// b -> (b / sub_nc, b % sub_nc) of an item's tile numbering, by multiply-high where the launcher found it exact
__device__ __forceinline__ void tile_of(const AdamItem& a, int b, int& tile_r, int& tile_c) {
  const int q = a.sub_magic ? (int)__umulhi((uint32_t)b, a.sub_magic) : b / a.sub_nc;
  tile_r = a.sub_r0 + q;
  tile_c = a.sub_c0 + (b - q * a.sub_nc);
}
inline uint32_t tile_magic(int64_t tiles, int nc) {
  // mulhi(b, ceil(2^32 / nc)) = b / nc while b (ceil(2^32 / nc) nc - 2^32) < 2^32; the bracket is below nc
  if (nc <= 1 || tiles * nc >= ((int64_t)1 << 32)) return 0u;
  return (uint32_t)((((uint64_t)1 << 32) + (uint64_t)nc - 1) / (uint64_t)nc);
}

// Where a thread works inside a tile of 4 E rows x 64 columns: E consecutive elements of one row.
template <int E>
struct TileThread {
  static constexpr int kPerRow = kStateTileCols / E;      // threads per tile row
  static constexpr int kRows = 256 / kPerRow;             // = 4 E
  int row, col;
  __device__ __forceinline__ TileThread(int tile_r, int tile_c)
      : row(tile_r * kRows + (int)threadIdx.x / kPerRow), col(tile_c * kStateTileCols + ((int)threadIdx.x % kPerRow) * E) {}
};

template <typename TN, int E>
__device__ __forceinline__ void store_n(TN* dst, const float (&n)[E], bool fast, int valid) {
  if (fast) {
    alignas(16) TN tmp[E];
#pragma unroll
    for (int e = 0; e < E; ++e) tmp[e] = cvt<TN>(n[e]);
    copy_vec<E * (int)sizeof(TN)>(dst, tmp);
  } else {
#pragma unroll
    for (int e = 0; e < E; ++e)
      if (e < valid) dst[e] = cvt<TN>(n[e]);
  }
}

// R of the thread's E elements: the split-K partials summed in a fixed order
template <int E>
__device__ __forceinline__ void load_r(const AdamItem& a, int64_t off, bool fast, int valid, float (&r)[E]) {
  if (fast) {
    copy_vec<E * 4>(r, a.Rpart + off);
    for (int s = 1; s < a.splits; ++s) {
      alignas(16) float q[E];
      copy_vec<E * 4>(q, a.Rpart + (int64_t)s * a.split_stride + off);
#pragma unroll
      for (int e = 0; e < E; ++e) r[e] += q[e];
    }
  } else {
#pragma unroll
    for (int e = 0; e < E; ++e) r[e] = e < valid ? a.Rpart[off + e] : 0.f;
    for (int s = 1; s < a.splits; ++s) {
      const float* __restrict__ part = a.Rpart + (int64_t)s * a.split_stride + off;
#pragma unroll
      for (int e = 0; e < E; ++e)
        if (e < valid) r[e] += part[e];
    }
  }
}

// ---- fp32 moments -------------------------------------------------------------
template <typename TN>
__device__ __forceinline__ bool adam_f32_tile(const AdamItem& a, int b) {
  constexpr int E = 8;
  int tile_r, tile_c;
  tile_of(a, b, tile_r, tile_c);
  const TileThread<E> tt(tile_r, tile_c);
  const int valid = tt.row < a.rows ? min(E, a.cols - tt.col) : 0;     // elements of the run inside the matrix
  if (valid <= 0) return false;
  const bool fast = a.vec && valid == E;
  const AdamParams p = a.p;
  const int64_t so = (int64_t)tt.row * a.s_ld + tt.col;
  alignas(16) float r[E], m[E], v[E];
  float n[E];
  load_r<E>(a, (int64_t)tt.row * a.r_ld + tt.col, fast, valid, r);
  if (fast) {
    copy_vec<E * 4>(m, a.M + so);
    copy_vec<E * 4>(v, a.V + so);
  } else {
#pragma unroll
    for (int e = 0; e < E; ++e) {
      m[e] = e < valid ? a.M[so + e] : 0.f;
      v[e] = e < valid ? a.V[so + e] : 0.f;
    }
  }
  uint32_t top = 0u;      // largest bit pattern among the new second moments (all >= 0): a non-finite r shows here
#pragma unroll
  for (int e = 0; e < E; ++e) {
    m[e] = adam_m(m[e], r[e], p);
    v[e] = adam_v(v[e], r[e], p);
    n[e] = adam_normalised(m[e], v[e], p);
    top = max(top, __float_as_uint(v[e]));
  }
  if (fast) {
    copy_vec<E * 4>(a.M + so, m);
    copy_vec<E * 4>(a.V + so, v);
  } else {
#pragma unroll
    for (int e = 0; e < E; ++e)
      if (e < valid) {
        a.M[so + e] = m[e];
        a.V[so + e] = v[e];
      }
  }
  store_n<TN, E>((TN*)a.Nout + (int64_t)tt.row * a.n_ld + tt.col, n, fast, valid);
  return top >= 0x7f800000u;
}

#ifndef GALORE_F32_CTAS
#define GALORE_F32_CTAS 3
#endif
template <typename TN>
__global__ void __launch_bounds__(256, GALORE_F32_CTAS) adam_f32_kernel(const __grid_constant__ AdamGroup g) {
  const int total = g.block_end[g.count - 1];
  int bad_item = -1, it = 0;
  for (int gb = blockIdx.x; gb < total; gb += gridDim.x) {
    int tile;
    find_item(g, gb, it, tile);
    if (adam_f32_tile<TN>(g.item[it], tile)) bad_item = it;
  }
  if (bad_item >= 0) atomicOr(g.item[bad_item].status, GALORE_DEV_NONFINITE);
}

// ---- 8-bit block-wise moments ---------------------------------------------------
// One tile = one quantisation block of 256 E elements (4 E rows x 64 columns).  Elements outside
// the matrix (edge tiles) enter as zeros with the codes of zero, so they change no absmax.
#ifndef GALORE_Q8_CTAS
#define GALORE_Q8_CTAS 4          // resident CTAs per SM the kernel is compiled for (register budget)
#endif

// FAST: the launch holds interior tiles of layers whose arrays allow vector accesses only, so nothing
// is predicated (fewer registers: one more resident CTA per SM).
template <typename TN, int E, bool FAST>
__device__ __forceinline__ bool adam_q8_tile(const AdamItem& a, int b, Q8Tables& t, int parity) {
  int tile_r, tile_c;
  tile_of(a, b, tile_r, tile_c);
  const int tile = tile_r * a.tiles_c + tile_c;
  const TileThread<E> tt(tile_r, tile_c);
  const int valid = FAST ? E : (tt.row < a.rows ? max(0, min(E, a.cols - tt.col)) : 0);
  const bool fast = FAST || (a.vec && valid == E);
  const AdamParams p = a.p;
  const int64_t so = (int64_t)tt.row * a.s_ld + tt.col;
  const float am_m = a.Mam[tile], am_v = a.Vam[tile];
  alignas(16) float r[E];
  alignas(16) uint8_t cm[E], cv[E];
  if (valid > 0) load_r<E>(a, (int64_t)tt.row * a.r_ld + tt.col, fast, valid, r);
  if (fast) {
    copy_vec<E>(cm, a.Mc + so);
    copy_vec<E>(cv, a.Vc + so);
  } else {
#pragma unroll
    for (int e = 0; e < E; ++e) {
      if (valid <= 0) r[e] = 0.f;
      cm[e] = e < valid ? a.Mc[so + e] : (uint8_t)127;
      cv[e] = e < valid ? a.Vc[so + e] : (uint8_t)0;
    }
  }
  float m[E], v[E], n[E];
  float mx_m = 0.f;
  uint32_t mx_v_bits = 0u;                       // v >= 0: the order of the bit patterns is the order of the values,
                                                 // and a NaN or an infinity (from a non-finite r) ends up on top
#pragma unroll
  for (int e = 0; e < E; ++e) {
    m[e] = adam_m(__fmul_rn(t.code_s[cm[e]], am_m), r[e], p);
    v[e] = adam_v(__fmul_rn(t.code_u[cv[e]], am_v), r[e], p);
    n[e] = adam_normalised(m[e], v[e], p);
    mx_m = fmaxf(mx_m, fabsf(m[e]));
    mx_v_bits = max(mx_v_bits, __float_as_uint(v[e]));
  }
  if (valid > 0) store_n<TN, E>((TN*)a.Nout + (int64_t)tt.row * a.n_ld + tt.col, n, fast, valid);
  const bool bad = mx_v_bits >= 0x7f800000u;
  uint32_t mx_m_bits = __float_as_uint(mx_m);
  block_max2_256(mx_m_bits, mx_v_bits, t.red + 16 + 16 * parity);
  mx_m = __uint_as_float(mx_m_bits);
  const float mx_v = __uint_as_float(mx_v_bits);
  // an all-zero block: with 0 in place of the reciprocal every y' is 0 and takes the code of zero
  // (the correctly rounded reciprocal, as 1 / x would give)
  const float inv_m = mx_m != 0.f ? __frcp_rn(mx_m) : 0.f, inv_v = mx_v != 0.f ? __frcp_rn(mx_v) : 0.f;
  if constexpr (E % 4 == 0) {
    alignas(16) uint32_t pm[E / 4], pv[E / 4];
#pragma unroll
    for (int j = 0; j < E / 4; ++j) {
      const float xm[4] = {m[4 * j], m[4 * j + 1], m[4 * j + 2], m[4 * j + 3]};
      const float xv[4] = {v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]};
      pm[j] = q8_encode4<true>(xm, mx_m, inv_m, t.enc_s, t.mid_s);
      pv[j] = q8_encode4<false>(xv, mx_v, inv_v, t.enc_u, t.mid_u);
    }
    if (fast) {
      copy_vec<E>(a.Mc + so, pm);
      copy_vec<E>(a.Vc + so, pv);
    } else {
#pragma unroll
      for (int e = 0; e < E; ++e)
        if (e < valid) {
          a.Mc[so + e] = (uint8_t)(pm[e / 4] >> (8 * (e % 4)));
          a.Vc[so + e] = (uint8_t)(pv[e / 4] >> (8 * (e % 4)));
        }
    }
  } else {
#pragma unroll
    for (int e = 0; e < E; ++e)
      if (e < valid) {
        a.Mc[so + e] = (uint8_t)q8_encode_block<true>(m[e], mx_m, inv_m, t.enc_s, t.mid_s);
        a.Vc[so + e] = (uint8_t)q8_encode_block<false>(v[e], mx_v, inv_v, t.enc_u, t.mid_u);
      }
  }
  if (threadIdx.x == 0) {
    a.Mam[tile] = mx_m;
    a.Vam[tile] = mx_v;
  }
  return bad;
}

#ifndef GALORE_Q8_FAST_CTAS
#define GALORE_Q8_FAST_CTAS 6       // 40 registers with a few spills: 7.0 ms for the LLaMA-7B set against 7.5 ms at 5 or 4 (32 KiB of tables per CTA: 6 is what fits)
#endif
constexpr int q8_ctas(bool fast) { return fast ? GALORE_Q8_FAST_CTAS : GALORE_Q8_CTAS; }

template <typename TN, int E, bool FAST>
__global__ void __launch_bounds__(256, q8_ctas(FAST)) adam_q8_kernel(const __grid_constant__ AdamGroup g, const Q8TablePtrs tp) {
  __shared__ Q8Tables t;
  q8_tables_fill(t, tp, threadIdx.x, 256);
  __syncthreads();
  const int total = g.block_end[g.count - 1];
  int bad_item = -1, it = 0;
  int parity = 0;
  for (int gb = blockIdx.x; gb < total; gb += gridDim.x, parity ^= 1) {
    int tile;
    find_item(g, gb, it, tile);
    if (adam_q8_tile<TN, E, FAST>(g.item[it], tile, t, parity)) bad_item = it;   // per thread: a non-finite input is reported by the threads that met it
  }
  if (bad_item >= 0) atomicOr(g.item[bad_item].status, GALORE_DEV_NONFINITE);
}

// ---- stand-alone quantise / dequantise ------------------------------------------------
// One CTA per tile of tile_rows x tile_cols elements; two passes over the tile (absmax, then codes).
__global__ void __launch_bounds__(256)
q8_quantize_kernel(const float* __restrict__ x, int64_t rows, int64_t cols, int64_t ldx, int is_signed, int tile_rows,
                   int tile_cols, int64_t tiles_c, uint8_t* __restrict__ codes, int64_t ldc, float* __restrict__ absmax,
                   const Q8TablePtrs tp) {
  __shared__ float s_mid[256];
  __shared__ uint32_t s_enc[kLutSize];
  __shared__ float red[8];
  for (int i = threadIdx.x; i < kLutSize; i += 256) s_enc[i] = is_signed ? tp.enc_s[i] : tp.enc_u[i];
  s_mid[threadIdx.x] = is_signed ? tp.mid_s[threadIdx.x] : tp.mid_u[threadIdx.x];
  const int64_t tile = blockIdx.x;
  const int64_t r0 = (tile / tiles_c) * tile_rows, c0 = (tile % tiles_c) * tile_cols;
  const int count = tile_rows * tile_cols;
  float mx = 0.f;
  for (int e = threadIdx.x; e < count; e += 256) {
    const int64_t i = r0 + e / tile_cols, j = c0 + e % tile_cols;
    if (i < rows && j < cols) mx = fmaxf(mx, fabsf(x[i * ldx + j]));
  }
  mx = warp_max(mx);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = mx;
  __syncthreads();
  mx = red[0];
#pragma unroll
  for (int w = 1; w < 8; ++w) mx = fmaxf(mx, red[w]);
  const uint8_t zero_code = is_signed ? 127 : 0;
  const float inv = 1.0f / mx;
  for (int e = threadIdx.x; e < count; e += 256) {
    const int64_t i = r0 + e / tile_cols, j = c0 + e % tile_cols;
    if (i < rows && j < cols) {
      const float val = x[i * ldx + j];
      codes[i * ldc + j] = (mx == 0.f) ? zero_code
                                       : (uint8_t)(is_signed ? q8_encode_block<true>(val, mx, inv, s_enc, s_mid)
                                                             : q8_encode_block<false>(val, mx, inv, s_enc, s_mid));
    }
  }
  if (threadIdx.x == 0) absmax[tile] = mx;
}

__global__ void __launch_bounds__(256)
q8_dequantize_kernel(const uint8_t* __restrict__ codes, int64_t ldc, const float* __restrict__ absmax, int64_t rows,
                     int64_t cols, int is_signed, int tile_rows, int tile_cols, int64_t tiles_c, float* __restrict__ out,
                     int64_t ldo, const Q8TablePtrs tp) {
  __shared__ float s_code[256];
  s_code[threadIdx.x] = is_signed ? tp.code_s[threadIdx.x] : tp.code_u[threadIdx.x];
  __syncthreads();
  const int64_t nel = rows * cols;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < nel; e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = e / cols, j = e % cols;
    out[i * ldo + j] = s_code[codes[i * ldc + j]] * absmax[(i / tile_rows) * tiles_c + j / tile_cols];
  }
}

// ---- launchers --------------------------------------------------------------------
static bool valid_block(int block) {
  return block == 256 || block == 512 || block == 1024 || block == 2048;
}

galore_status_t launch_adam_group(const AdamGroup& g, int32_t state_fmt, int q_block, int32_t n_dtype, cudaStream_t st) {
  if (g.count < 1 || g.count > kAdamGroup) return GALORE_ERR_INVALID_ARG;
  const int total = g.block_end[g.count - 1];
  if (total <= 0) return GALORE_OK;
  const bool nb = n_dtype == GALORE_BF16;
  if (state_fmt == GALORE_STATE_F32) {
    const unsigned grid = (unsigned)std::min(total, 148 * 8);
    if (nb) adam_f32_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(g);
    else adam_f32_kernel<float><<<grid, 256, 0, st>>>(g);
    GALORE_LAUNCH_CHECK();
    return GALORE_OK;
  }
  if (!valid_block(q_block)) return GALORE_ERR_INVALID_ARG;
  Q8TablePtrs tp;
  GALORE_TRY(q8_table_ptrs(&tp));
  // The interior tiles of layers whose arrays allow vector accesses go to the kernel that holds the
  // unpredicated code alone; the ragged right and bottom strips and everything else to the general one.
  const int tile_rows = q_block / kStateTileCols;
  std::unique_ptr<AdamGroup> fast(new AdamGroup), rest(new AdamGroup);
  fast->count = rest->count = 0;
  auto launch = [&](const AdamGroup& grp, bool is_fast) -> galore_status_t {
    if (grp.count == 0) return GALORE_OK;
    const int blocks = grp.block_end[grp.count - 1];
    // one resident wave: the 32 KiB of tables are set up once per SM slot
    const unsigned grid = (unsigned)std::min(blocks, 148 * q8_ctas(is_fast));
#define GALORE_Q8_LAUNCH(TN, E, F)                                                                              \
  do {                                                                                                          \
    GALORE_CUDA_TRY(cudaFuncSetAttribute(adam_q8_kernel<TN, E, F>, cudaFuncAttributePreferredSharedMemoryCarveout, \
                                         cudaSharedmemCarveoutMaxShared));                                      \
    adam_q8_kernel<TN, E, F><<<grid, 256, 0, st>>>(grp, tp);                                                    \
    GALORE_LAUNCH_CHECK();                                                                                      \
  } while (0)
#define GALORE_Q8_CASE(E)                                        \
  case E * 256:                                                  \
    if (nb && is_fast) GALORE_Q8_LAUNCH(__nv_bfloat16, E, true); \
    else if (nb) GALORE_Q8_LAUNCH(__nv_bfloat16, E, false);      \
    else if (is_fast) GALORE_Q8_LAUNCH(float, E, true);          \
    else GALORE_Q8_LAUNCH(float, E, false);                      \
    break;
    switch (q_block) {
      GALORE_Q8_CASE(1) GALORE_Q8_CASE(2) GALORE_Q8_CASE(4) GALORE_Q8_CASE(8)
      default: return GALORE_ERR_INVALID_ARG;
    }
#undef GALORE_Q8_CASE
#undef GALORE_Q8_LAUNCH
    return GALORE_OK;
  };
  auto append = [&](AdamGroup& dst, bool is_fast, const AdamItem& a, int r0, int c0, int nr, int nc) -> galore_status_t {
    if (nr <= 0 || nc <= 0) return GALORE_OK;
    if (dst.count == kAdamGroup) {            // full: send what has been collected and start again
      GALORE_TRY(launch(dst, is_fast));
      dst.count = 0;
    }
    const int j = dst.count++;
    dst.item[j] = a;
    dst.item[j].sub_r0 = r0;
    dst.item[j].sub_c0 = c0;
    dst.item[j].sub_nc = nc;
    dst.item[j].sub_magic = tile_magic((int64_t)nr * nc, nc);
    dst.block_end[j] = (j > 0 ? dst.block_end[j - 1] : 0) + nr * nc;
    return GALORE_OK;
  };
  for (int i = 0; i < g.count; ++i) {
    const AdamItem& a = g.item[i];
    const int tr = (int)ceil_div(a.rows, tile_rows), tc = a.tiles_c;
    const int full_r = a.rows / tile_rows, full_c = a.cols / kStateTileCols;
    if (a.vec) {
      GALORE_TRY(append(*fast, true, a, 0, 0, full_r, full_c));
      GALORE_TRY(append(*rest, false, a, 0, full_c, tr, tc - full_c));            // ragged right strip
      GALORE_TRY(append(*rest, false, a, full_r, 0, tr - full_r, full_c));        // ragged bottom strip
    } else {
      GALORE_TRY(append(*rest, false, a, 0, 0, tr, tc));
    }
  }
  GALORE_TRY(launch(*fast, true));
  return launch(*rest, false);
}

galore_status_t adam_group_add(AdamGroup& g, const AdamItem& item, int32_t state_fmt, int q_block) {
  if (g.count >= kAdamGroup) return GALORE_ERR_BUFFER_TOO_SMALL;
  if (item.rows <= 0 || item.cols <= 0) return GALORE_ERR_SHAPE;
  AdamItem a = item;
  const int tile_rows = state_fmt == GALORE_STATE_F32 ? 32 : q_block / kStateTileCols;
  a.tiles_c = (int)ceil_div(a.cols, kStateTileCols);
  const int64_t tiles = ceil_div(a.rows, tile_rows) * a.tiles_c;
  const int64_t before = g.count > 0 ? g.block_end[g.count - 1] : 0;
  if (before + tiles >= (int64_t)1 << 31) return GALORE_ERR_SHAPE;
  // vector accesses of an interior tile: 16-byte aligned bases, rows of R and of fp32 moments a
  // multiple of 4 floats, rows of N a multiple of 8 elements, rows of codes a multiple of 16 bytes
  const uintptr_t bases = (uintptr_t)a.Rpart | (uintptr_t)a.Nout | (uintptr_t)a.Mc | (uintptr_t)a.Vc | (uintptr_t)a.M |
                          (uintptr_t)a.V;
  const bool pitches = (a.r_ld % 4) == 0 && (a.n_ld % 8) == 0 && (a.split_stride % 4) == 0 &&
                       (a.s_ld % (state_fmt == GALORE_STATE_F32 ? 4 : 16)) == 0;
  a.vec = ((bases & 15) == 0 && pitches) ? 1 : 0;
  a.sub_r0 = a.sub_c0 = 0;
  a.sub_nc = a.tiles_c;
  a.sub_magic = tile_magic(tiles, a.tiles_c);
  const int i = g.count++;
  g.item[i] = a;
  g.block_end[i] = (int)(before + tiles);
  return GALORE_OK;
}

galore_status_t launch_adam(const AdamItem& item, int32_t state_fmt, int q_block, int32_t n_dtype, cudaStream_t st) {
  std::unique_ptr<AdamGroup> g(new AdamGroup);
  g->count = 0;
  GALORE_TRY(adam_group_add(*g, item, state_fmt, q_block));
  return launch_adam_group(*g, state_fmt, q_block, n_dtype, st);
}

galore_status_t launch_q8_quantize(const float* x, int64_t rows, int64_t cols, int64_t ldx, int is_signed, int tile_rows,
                                   int tile_cols, uint8_t* codes, int64_t ldc, float* absmax, cudaStream_t st) {
  if (rows <= 0 || cols <= 0) return GALORE_OK;
  if (tile_rows < 1 || tile_cols < 1 || (int64_t)tile_rows * tile_cols > (1 << 20)) return GALORE_ERR_INVALID_ARG;
  Q8TablePtrs tp;
  GALORE_TRY(q8_table_ptrs(&tp));
  const int64_t tiles_c = ceil_div(cols, tile_cols);
  const int64_t tiles = ceil_div(rows, tile_rows) * tiles_c;
  if (tiles >= (int64_t)1 << 31) return GALORE_ERR_SHAPE;
  q8_quantize_kernel<<<(unsigned)tiles, 256, 0, st>>>(x, rows, cols, ldx, is_signed, tile_rows, tile_cols, tiles_c, codes,
                                                      ldc, absmax, tp);
  GALORE_LAUNCH_CHECK();
  return GALORE_OK;
}

galore_status_t launch_q8_dequantize(const uint8_t* codes, int64_t ldc, const float* absmax, int64_t rows, int64_t cols,
                                     int is_signed, int tile_rows, int tile_cols, float* out, int64_t ldo, cudaStream_t st) {
  if (rows <= 0 || cols <= 0) return GALORE_OK;
  if (tile_rows < 1 || tile_cols < 1) return GALORE_ERR_INVALID_ARG;
  Q8TablePtrs tp;
  GALORE_TRY(q8_table_ptrs(&tp));
  const int64_t blocks = std::min<int64_t>(ceil_div(rows * cols, 256), 148 * 16);
  q8_dequantize_kernel<<<(unsigned)blocks, 256, 0, st>>>(codes, ldc, absmax, rows, cols, is_signed, tile_rows, tile_cols,
                                                         ceil_div(cols, tile_cols), out, ldo, tp);
  GALORE_LAUNCH_CHECK();
  return GALORE_OK;
}

}  // namespace galore
