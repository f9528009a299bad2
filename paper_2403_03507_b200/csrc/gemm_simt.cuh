// Stride-general FMA GEMM with a pluggable epilogue.
//
// C(i, j) = sum_k A(i, k) * B(k, j),  A(i, k) = A[i*sAi + k*sAk],  B(k, j) = B[k*sBk + j*sBj]
//
// This is the library's fp32/fp64 path: it takes any operand dtype, any
// leading dimension and both transpositions, accumulates in TAcc (float or
// double) and hands each finished element to an epilogue functor
// epi(i, j, acc, split).  It carries the projections when the inputs are fp32
// (where bf16 tensor-core inputs would break the fp32 tolerance) or not
// TMA-aligned, and all fp64 work of the projector refresh.
// blockIdx.z selects a K slice of `kchunk` elements (split-K) or, when `batched`, one problem of
// a batch whose operands lie batchA / batchB elements apart; with a slot list of n entries the grid
// holds n such groups, group i with A, B and the epilogue's output shifted by id[i] * bytes.
#pragma once

#include "common.cuh"

namespace galore {

// One BM x BN tile of C over the K range [k_begin, k_end): the main loop shared by the kernels below.
template <typename TA, typename TB, typename TAcc, int BM, int BN, int BK, int TM, int TN, class Epi>
__device__ __forceinline__ void gemm_simt_tile(int M, int N, const TA* __restrict__ A, int64_t sAi, int64_t sAk,
                                               const TB* __restrict__ B, int64_t sBk, int64_t sBj, int m0, int n0, int k_begin,
                                               int k_end, int zi, const Epi& epi) {
  constexpr int NT = (BM / TM) * (BN / TN);
  constexpr int LA = BM * BK / NT;   // elements of the A tile each thread fetches
  constexpr int LB = BN * BK / NT;
  static_assert(BM * BK % NT == 0 && BN * BK % NT == 0, "tile/threads mismatch");
  static_assert(TM % 4 == 0 && TN % 4 == 0, "micro-tile is built from groups of 4");
  __shared__ TAcc As[BK][BM + 4];
  __shared__ TAcc Bs[BK][BN + 4];

  const int tid = threadIdx.x;
  const int tx = tid % (BN / TN), ty = tid / (BN / TN);
  const bool a_kfast = (sAk == 1);   // consecutive threads walk the contiguous direction
  const bool b_kfast = (sBk == 1);

  TAcc acc[TM][TN];
#pragma unroll
  for (int u = 0; u < TM; ++u)
#pragma unroll
    for (int v = 0; v < TN; ++v) acc[u][v] = TAcc(0);

  TAcc ra[LA], rb[LB];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int e = 0; e < LA; ++e) {
      int idx = tid + e * NT;
      int i = a_kfast ? idx / BK : idx % BM;
      int k = a_kfast ? idx % BK : idx / BM;
      int gi = m0 + i, gk = k0 + k;
      ra[e] = (gi < M && gk < k_end) ? cvt<TAcc>(A[(int64_t)gi * sAi + (int64_t)gk * sAk]) : TAcc(0);
    }
#pragma unroll
    for (int e = 0; e < LB; ++e) {
      int idx = tid + e * NT;
      int j = b_kfast ? idx / BK : idx % BN;
      int k = b_kfast ? idx % BK : idx / BN;
      int gj = n0 + j, gk = k0 + k;
      rb[e] = (gj < N && gk < k_end) ? cvt<TAcc>(B[(int64_t)gk * sBk + (int64_t)gj * sBj]) : TAcc(0);
    }
  };
  auto stash = [&]() {
#pragma unroll
    for (int e = 0; e < LA; ++e) {
      int idx = tid + e * NT;
      int i = a_kfast ? idx / BK : idx % BM;
      int k = a_kfast ? idx % BK : idx / BM;
      As[k][i] = ra[e];
    }
#pragma unroll
    for (int e = 0; e < LB; ++e) {
      int idx = tid + e * NT;
      int j = b_kfast ? idx / BK : idx % BN;
      int k = b_kfast ? idx % BK : idx / BN;
      Bs[k][j] = rb[e];
    }
  };

  if (k_begin < k_end) fetch(k_begin);
  for (int k0 = k_begin; k0 < k_end; k0 += BK) {
    __syncthreads();
    stash();
    __syncthreads();
    if (k0 + BK < k_end) fetch(k0 + BK);
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      TAcc a[TM], b[TN];
#pragma unroll
      for (int u = 0; u < TM; ++u) a[u] = As[k][(u / 4) * (BM / (TM / 4)) + ty * 4 + (u % 4)];
#pragma unroll
      for (int v = 0; v < TN; ++v) b[v] = Bs[k][(v / 4) * (BN / (TN / 4)) + tx * 4 + (v % 4)];
#pragma unroll
      for (int u = 0; u < TM; ++u)
#pragma unroll
        for (int v = 0; v < TN; ++v) acc[u][v] = fma(a[u], b[v], acc[u][v]);
    }
  }
  // a thread's columns come in runs of four: one 8- or 16-byte access where the epilogue's array allows it
#pragma unroll
  for (int u = 0; u < TM; ++u) {
    int i = m0 + (u / 4) * (BM / (TM / 4)) + ty * 4 + (u % 4);
    if (i >= M) continue;
#pragma unroll
    for (int vg = 0; vg < TN / 4; ++vg) {
      const int j = n0 + vg * (BN / (TN / 4)) + tx * 4;
      if (j + 3 < N && epi.can4(i, j, zi)) {
        epi.apply4(i, j, &acc[u][4 * vg], zi);
      } else {
#pragma unroll
        for (int v = 0; v < 4; ++v)
          if (j + v < N) epi(i, j + v, acc[u][4 * vg + v], zi);
      }
    }
  }
}

template <typename TA, typename TB, typename TAcc, int BM, int BN, int BK, int TM, int TN, class Epi>
__global__ void __launch_bounds__((BM / TM) * (BN / TN))
gemm_simt_kernel(int M, int N, int K, const TA* __restrict__ A, int64_t sAi, int64_t sAk,
                 const TB* __restrict__ B, int64_t sBk, int64_t sBj, int kchunk, Epi epi_in, int batched,
                 int64_t batchA, int64_t batchB, const SlotList slots, int lower_only) {
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  if (lower_only && n0 > m0 + BM - 1) return;      // the tile lies strictly above the diagonal of a square result
  const int inner = gridDim.z / slots.n;
  const int zi = blockIdx.z % inner;
  const int64_t shift = (int64_t)slots.id[blockIdx.z / inner] * slots.bytes;
  Epi epi = epi_in;
  if (shift) {
    A = slot_ptr(A, shift);
    B = slot_ptr(B, shift);
    epi.shift(shift);
  }
  const int k_begin = batched ? 0 : zi * kchunk;
  const int k_end = batched ? K : min(K, k_begin + kchunk);
  if (batched) {
    A += (int64_t)zi * batchA;
    B += (int64_t)zi * batchB;
  }
  gemm_simt_tile<TA, TB, TAcc, BM, BN, BK, TM, TN, Epi>(M, N, A, sAi, sAk, B, sBk, sBj, m0, n0, k_begin, k_end, zi, epi);
}

// ---- several problems of one operand-type combination in one launch ------------------------------
// (the projections of a layer set on the fp32 path: one launch instead of one per layer)
constexpr int kSimtGroup = 32;
template <class Epi>
struct SimtProblem {
  int M, N, K;
  const void* A;
  int64_t sAi, sAk;
  const void* B;
  int64_t sBk, sBj;
  int kchunk, splits;      // K slices of kchunk elements; slice z is handed to epi as its last argument
  Epi epi;
};
template <class Epi>
struct SimtGroup {
  SimtProblem<Epi> p[kSimtGroup];
  int cta_end[kSimtGroup];   // running totals of CTAs (tiles x K slices)
  int count;
};

template <typename TA, typename TB, typename TAcc, int BM, int BN, int BK, int TM, int TN, class Epi>
__global__ void __launch_bounds__((BM / TM) * (BN / TN))
gemm_simt_group_kernel(const __grid_constant__ SimtGroup<Epi> g) {
  int it = 0;
  while (it + 1 < g.count && (int)blockIdx.x >= g.cta_end[it]) ++it;
  const SimtProblem<Epi>& p = g.p[it];
  int local = (int)blockIdx.x - (it ? g.cta_end[it - 1] : 0);
  const int tiles_n = (p.N + BN - 1) / BN, tiles_m = (p.M + BM - 1) / BM;
  const int tn = local % tiles_n;
  local /= tiles_n;
  const int tm = local % tiles_m, zi = local / tiles_m;
  const int k_begin = zi * p.kchunk, k_end = min(p.K, k_begin + p.kchunk);
  gemm_simt_tile<TA, TB, TAcc, BM, BN, BK, TM, TN, Epi>(p.M, p.N, (const TA*)p.A, p.sAi, p.sAk, (const TB*)p.B, p.sBk, p.sBj,
                                                        tm * BM, tn * BN, k_begin, k_end, zi, p.epi);
}

// adds one problem (128 x 128 tiles); `splits` as for launch_gemm_simt
template <class Epi>
galore_status_t simt_group_add(SimtGroup<Epi>& g, int M, int N, int K, const void* A, int64_t sAi, int64_t sAk, const void* B,
                               int64_t sBk, int64_t sBj, int splits, const Epi& epi) {
  if (g.count >= kSimtGroup) return GALORE_ERR_BUFFER_TOO_SMALL;
  if (M <= 0 || N <= 0) return GALORE_ERR_SHAPE;
  if (splits < 1) splits = 1;
  int kchunk = (int)ceil_div(ceil_div(K, splits), 16) * 16;
  if (kchunk < 16) kchunk = 16;
  splits = (int)ceil_div(K > 0 ? K : 1, kchunk);
  SimtProblem<Epi>& p = g.p[g.count];
  p.M = M; p.N = N; p.K = K;
  p.A = A; p.sAi = sAi; p.sAk = sAk;
  p.B = B; p.sBk = sBk; p.sBj = sBj;
  p.kchunk = kchunk; p.splits = splits;
  p.epi = epi;
  const int64_t ctas = ceil_div(M, 128) * ceil_div(N, 128) * splits;
  const int64_t before = g.count ? g.cta_end[g.count - 1] : 0;
  if (before + ctas >= ((int64_t)1 << 31)) return GALORE_ERR_SHAPE;
  g.cta_end[g.count] = (int)(before + ctas);
  g.count += 1;
  return GALORE_OK;
}
template <typename TA, typename TB, typename TAcc, class Epi>
galore_status_t launch_gemm_simt_group(const SimtGroup<Epi>& g, cudaStream_t stream) {
  if (g.count <= 0) return GALORE_OK;
  gemm_simt_group_kernel<TA, TB, TAcc, 128, 128, 16, 8, 8, Epi><<<(unsigned)g.cta_end[g.count - 1], 256, 0, stream>>>(g);
  GALORE_LAUNCH_CHECK();
  return GALORE_OK;
}

// ---- epilogues ----------------------------------------------------------------

// C[split][i][j] = alpha * acc  (+ beta * C when beta != 0; only with one split)
template <typename TC, typename TAcc>
struct EpiStore {
  TC* C;
  int64_t ldc;
  int64_t split_stride;
  TAcc alpha, beta;
  __device__ __forceinline__ void shift(int64_t bytes) { C = slot_ptr(C, bytes); }
  __device__ __forceinline__ void operator()(int i, int j, TAcc acc, int z) const {
    TC* p = C + (int64_t)z * split_stride + (int64_t)i * ldc + j;
    TAcc v = alpha * acc;
    if (beta != TAcc(0)) v += beta * cvt<TAcc>(*p);
    *p = cvt<TC>(v);
  }
  // four neighbouring columns at once (fp32 output on a 16-byte boundary)
  __device__ __forceinline__ bool can4(int i, int j, int z) const {
    if constexpr (sizeof(TC) != 4 || sizeof(TAcc) != 4) return false;
    return ((uintptr_t)(C + (int64_t)z * split_stride + (int64_t)i * ldc + j) & 15) == 0;
  }
  __device__ __forceinline__ void apply4(int i, int j, const TAcc* acc, int z) const {
    if constexpr (sizeof(TC) == 4 && sizeof(TAcc) == 4) {
      float4* p = reinterpret_cast<float4*>(C + (int64_t)z * split_stride + (int64_t)i * ldc + j);
      float4 v = make_float4(alpha * acc[0], alpha * acc[1], alpha * acc[2], alpha * acc[3]);
      if (beta != TAcc(0)) {
        const float4 c = *p;
        v.x += beta * c.x; v.y += beta * c.y; v.z += beta * c.z; v.w += beta * c.w;
      }
      *p = v;
    }
  }
};

// W[i][j] <- keep * W[i][j] - scale * acc   (the weight update that closes Algorithm 1; keep =
// 1 - lr * weight_decay for GaLore-AdamW, exactly 1 otherwise)
template <typename TW>
struct EpiApplyW {
  TW* W;
  int64_t ldw;
  float scale;
  float keep = 1.0f;
  __device__ __forceinline__ void shift(int64_t bytes) { W = slot_ptr(W, bytes); }
  __device__ __forceinline__ void operator()(int i, int j, float acc, int) const {
    TW* p = W + (int64_t)i * ldw + j;
    *p = cvt<TW>(fmaf(-scale, acc, keep * cvt<float>(*p)));
  }
  // four neighbouring weights at once (16 bytes of fp32, 8 bytes of bf16, on their own boundary)
  __device__ __forceinline__ bool can4(int i, int j, int) const {
    return ((uintptr_t)(W + (int64_t)i * ldw + j) & (4 * sizeof(TW) - 1)) == 0;
  }
  __device__ __forceinline__ void apply4(int i, int j, const float* acc, int) const {
    TW* p = W + (int64_t)i * ldw + j;
    if constexpr (sizeof(TW) == 4) {
      float4 w = *reinterpret_cast<float4*>(p);
      w.x = fmaf(-scale, acc[0], keep * w.x);
      w.y = fmaf(-scale, acc[1], keep * w.y);
      w.z = fmaf(-scale, acc[2], keep * w.z);
      w.w = fmaf(-scale, acc[3], keep * w.w);
      *reinterpret_cast<float4*>(p) = w;
    } else {
      uint2 raw = *reinterpret_cast<uint2*>(p);
      __nv_bfloat162 lo = *reinterpret_cast<__nv_bfloat162*>(&raw.x), hi = *reinterpret_cast<__nv_bfloat162*>(&raw.y);
      const float2 a = __bfloat1622float2(lo), b = __bfloat1622float2(hi);
      lo = __floats2bfloat162_rn(fmaf(-scale, acc[0], keep * a.x), fmaf(-scale, acc[1], keep * a.y));
      hi = __floats2bfloat162_rn(fmaf(-scale, acc[2], keep * b.x), fmaf(-scale, acc[3], keep * b.y));
      raw.x = *reinterpret_cast<uint32_t*>(&lo);
      raw.y = *reinterpret_cast<uint32_t*>(&hi);
      *reinterpret_cast<uint2*>(p) = raw;
    }
  }
};

template <typename TA, typename TB, typename TAcc, class Epi>
galore_status_t launch_gemm_simt(int M, int N, int K, const TA* A, int64_t sAi, int64_t sAk, const TB* B,
                                 int64_t sBk, int64_t sBj, int splits, Epi epi, cudaStream_t stream, int batch = 0,
                                 int64_t batchA = 0, int64_t batchB = 0, const SlotList* slot_list = nullptr,
                                 bool lower_only = false) {
  if (M <= 0 || N <= 0) return GALORE_OK;
  if (batch > 0) splits = 1;       // a batch uses blockIdx.z for the problem index
  if (splits < 1) splits = 1;
  int kchunk = (int)ceil_div(ceil_div(K, splits), 16) * 16;
  if (kchunk < 16) kchunk = 16;
  splits = (int)ceil_div(K > 0 ? K : 1, kchunk);
  const SlotList slots = slot_list ? *slot_list : single_slot();
  const unsigned gz = (batch > 0 ? (unsigned)batch : (unsigned)splits) * (unsigned)slots.n;
  const bool small = (int64_t)M * N * (batch > 0 ? batch : 1) * slots.n < (int64_t)128 * 128 * 96;
  if (small) {
    dim3 grid((unsigned)ceil_div(N, 64), (unsigned)ceil_div(M, 64), gz);
    gemm_simt_kernel<TA, TB, TAcc, 64, 64, 16, 4, 4, Epi><<<grid, 256, 0, stream>>>(
        M, N, K, A, sAi, sAk, B, sBk, sBj, kchunk, epi, batch > 0 ? 1 : 0, batchA, batchB, slots, lower_only ? 1 : 0);
  } else {
    dim3 grid((unsigned)ceil_div(N, 128), (unsigned)ceil_div(M, 128), gz);
    gemm_simt_kernel<TA, TB, TAcc, 128, 128, 16, 8, 8, Epi><<<grid, 256, 0, stream>>>(
        M, N, K, A, sAi, sAk, B, sBk, sBj, kchunk, epi, batch > 0 ? 1 : 0, batchA, batchB, slots, lower_only ? 1 : 0);
  }
  GALORE_LAUNCH_CHECK();
  return GALORE_OK;
}

// number of K slices launch_gemm_simt will actually use for a request of `splits`
inline int simt_effective_splits(int K, int splits) {
  if (splits < 1) splits = 1;
  int kchunk = (int)ceil_div(ceil_div(K, splits), 16) * 16;
  if (kchunk < 16) kchunk = 16;
  return (int)ceil_div(K > 0 ? K : 1, kchunk);
}

}  // namespace galore
