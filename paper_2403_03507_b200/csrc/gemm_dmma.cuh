// Stride-general fp64 GEMM on the double-precision MMA unit, with a pluggable epilogue.
//
// C(i, j) = sum_k A(i, k) * B(k, j),  A(i, k) = A[i*sAi + k*sAk],  B(k, j) = B[k*sBk + j*sBj]
//
// Same contract as the FMA kernel of gemm_simt.cuh with a double accumulator: any operand dtype
// (converted to double while staging), any leading dimension, both transpositions, and every
// finished element handed to epi(i, j, acc, z).  blockIdx.z selects one problem of a batch whose
// operands lie `batchA` / `batchB` elements apart; with a slot list of n entries the grid holds n
// such batches, batch i with A, B and the epilogue's output shifted by id[i] * bytes.  It carries the fp64 products of the projector
// refresh (Gram matrices, triangular inverses, Rayleigh-Ritz).
#pragma once

#include "common.cuh"

namespace galore {

// D (8 x 8) += A (8 x 4, row) B (4 x 8, col), fp64.  Lane l holds A[l / 4][l % 4], B[l % 4][l / 4]
// and D[l / 4][2 (l % 4) + {0, 1}].
__device__ __forceinline__ void dmma_m8n8k4(double (&d)[2], double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};\n"
               : "+d"(d[0]), "+d"(d[1])
               : "d"(a), "d"(b));
}

template <typename TA, typename TB, int BM, int BN, int WM, int WN, class Epi>
__global__ void __launch_bounds__((BM / WM) * (BN / WN) * 32)
gemm_dmma_kernel(int M, int N, int K, const TA* __restrict__ A, int64_t sAi, int64_t sAk, int64_t batchA,
                 const TB* __restrict__ B, int64_t sBk, int64_t sBj, int64_t batchB, Epi epi_in, const SlotList slots) {
  constexpr int BK = 16;
  constexpr int NT = (BM / WM) * (BN / WN) * 32;
  constexpr int LA = BM * BK / NT, LB = BN * BK / NT;
  static_assert(BM * BK % NT == 0 && BN * BK % NT == 0, "tile/threads mismatch");
  static_assert(WM % 8 == 0 && WN % 8 == 0 && BM % 16 == 0 && BN % 16 == 0, "warp tile is built from 8 x 8 MMA tiles");
  // k-major tiles with a row stride = 4 mod 16 doubles: the 4 x 8 operand fragments (4 k, 8 m) of a
  // half-warp then touch 16 distinct banks
  __shared__ double As[BK][BM + 4];
  __shared__ double Bs[BK][BN + 4];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int wm0 = (warp / (BN / WN)) * WM, wn0 = (warp % (BN / WN)) * WN;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const int inner = gridDim.z / slots.n;
  const int zi = blockIdx.z % inner;
  const int64_t shift = (int64_t)slots.id[blockIdx.z / inner] * slots.bytes;
  Epi epi = epi_in;
  if (shift) {
    A = slot_ptr(A, shift);
    B = slot_ptr(B, shift);
    epi.shift(shift);
  }
  A += (int64_t)zi * batchA;
  B += (int64_t)zi * batchB;
  const bool a_kfast = (sAk == 1);
  const bool b_kfast = (sBk == 1);

  double acc[WM / 8][WN / 8][2];
#pragma unroll
  for (int i = 0; i < WM / 8; ++i)
#pragma unroll
    for (int j = 0; j < WN / 8; ++j) acc[i][j][0] = acc[i][j][1] = 0.0;

  double ra[LA], rb[LB];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int e = 0; e < LA; ++e) {
      const int idx = tid + e * NT;
      const int i = a_kfast ? idx / BK : idx % BM;
      const int k = a_kfast ? idx % BK : idx / BM;
      const int gi = m0 + i, gk = k0 + k;
      ra[e] = (gi < M && gk < K) ? cvt<double>(A[(int64_t)gi * sAi + (int64_t)gk * sAk]) : 0.0;
    }
#pragma unroll
    for (int e = 0; e < LB; ++e) {
      const int idx = tid + e * NT;
      const int j = b_kfast ? idx / BK : idx % BN;
      const int k = b_kfast ? idx % BK : idx / BN;
      const int gj = n0 + j, gk = k0 + k;
      rb[e] = (gj < N && gk < K) ? cvt<double>(B[(int64_t)gk * sBk + (int64_t)gj * sBj]) : 0.0;
    }
  };
  auto stash = [&]() {
#pragma unroll
    for (int e = 0; e < LA; ++e) {
      const int idx = tid + e * NT;
      const int i = a_kfast ? idx / BK : idx % BM;
      const int k = a_kfast ? idx % BK : idx / BM;
      As[k][i] = ra[e];
    }
#pragma unroll
    for (int e = 0; e < LB; ++e) {
      const int idx = tid + e * NT;
      const int j = b_kfast ? idx / BK : idx % BN;
      const int k = b_kfast ? idx % BK : idx / BN;
      Bs[k][j] = rb[e];
    }
  };

  if (K > 0) fetch(0);
  for (int k0 = 0; k0 < K; k0 += BK) {
    __syncthreads();
    stash();
    __syncthreads();
    if (k0 + BK < K) fetch(k0 + BK);
#pragma unroll
    for (int ks = 0; ks < BK / 4; ++ks) {
      double a[WM / 8], b[WN / 8];
#pragma unroll
      for (int i = 0; i < WM / 8; ++i) a[i] = As[ks * 4 + t][wm0 + i * 8 + g];
#pragma unroll
      for (int j = 0; j < WN / 8; ++j) b[j] = Bs[ks * 4 + t][wn0 + j * 8 + g];
#pragma unroll
      for (int i = 0; i < WM / 8; ++i)
#pragma unroll
        for (int j = 0; j < WN / 8; ++j) dmma_m8n8k4(acc[i][j], a[i], b[j]);
    }
  }
#pragma unroll
  for (int i = 0; i < WM / 8; ++i) {
    const int gi = m0 + wm0 + i * 8 + g;
    if (gi >= M) continue;
#pragma unroll
    for (int j = 0; j < WN / 8; ++j) {
      const int gj = n0 + wn0 + j * 8 + 2 * t;
      if (gj < N) epi(gi, gj, acc[i][j][0], zi);
      if (gj + 1 < N) epi(gi, gj + 1, acc[i][j][1], zi);
    }
  }
}

template <typename TA, typename TB, class Epi>
galore_status_t launch_gemm_dmma(int M, int N, int K, const TA* A, int64_t sAi, int64_t sAk, const TB* B, int64_t sBk,
                                 int64_t sBj, Epi epi, cudaStream_t stream, int batch = 1, int64_t batchA = 0,
                                 int64_t batchB = 0, const SlotList* slot_list = nullptr) {
  if (M <= 0 || N <= 0 || batch <= 0) return GALORE_OK;
  const SlotList slots = slot_list ? *slot_list : single_slot();
  batch *= slots.n;
  const bool small = (int64_t)M * N * batch < (int64_t)128 * 128 * 96;
  if (small) {
    dim3 grid((unsigned)ceil_div(N, 64), (unsigned)ceil_div(M, 64), (unsigned)batch);
    gemm_dmma_kernel<TA, TB, 64, 64, 32, 32, Epi><<<grid, 128, 0, stream>>>(M, N, K, A, sAi, sAk, batchA, B, sBk, sBj,
                                                                           batchB, epi, slots);
  } else {
    dim3 grid((unsigned)ceil_div(N, 128), (unsigned)ceil_div(M, 128), (unsigned)batch);
    // sixteen warps of 32 x 32 (four per scheduler hide the latency of the fragment loads better than eight of 32 x 64)
    gemm_dmma_kernel<TA, TB, 128, 128, 32, 32, Epi><<<grid, 512, 0, stream>>>(M, N, K, A, sAi, sAk, batchA, B, sBk, sBj,
                                                                             batchB, epi, slots);
  }
  GALORE_LAUNCH_CHECK();
  return GALORE_OK;
}

}  // namespace galore
