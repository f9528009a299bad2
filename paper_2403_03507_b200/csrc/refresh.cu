// Projector refresh: the top-r singular subspace of the current gradient
// (Algorithm 1, the "t mod T = 0" branch; Eq. 12-13), computed on the GPU by
// block subspace iteration instead of a full SVD.
//
// With A = G (left projector, d = m, L = n) or A = G^T (right, d = n, L = m):
//
//   Y (d x b) random, b = r + oversample                     start block
//   repeat:  Z = A^T Y ;  Y' = A Z + delta Y ;  Y = orth(Y')  power step on A A^T + delta I,
//                                                            never forming A A^T
//   Rayleigh-Ritz:  Y orthonormalised in fp64;  Z = A^T Y;  H = Z^T Z = Y^T A A^T Y;
//                   H = S Theta S^T by parallel one-sided Jacobi;  P = Y S[:, top r]
//
// orth() is CholeskyQR (Gram matrix in fp64, blocked Cholesky, blocked
// triangular solve).  The tiny shift delta keeps Y at full column rank when G
// itself has rank < b (it moves every eigenvalue by delta and no eigenvector).
// The power steps only have to bring span(Y) close to the wanted subspace, so
// they run in fp32; what fixes the accuracy of P is the last orthonormalisation
// and the Rayleigh-Ritz step, which run in fp64.
//
// Stated convergence: after q power steps the error of the top-r subspace
// decays like (theta_b / theta_r)^q (theta = Ritz values, descending); the
// iteration stops when that prediction is below the tolerance, or at the cap.
#include "refresh.cuh"
#include <type_traits>
#include "eig_jacobi.cuh"
#include "gemm_dmma.cuh"

#include <math.h>

#include <algorithm>
#include <chrono>
#include <vector>

#include "gemm_simt.cuh"
#include "gemm_tc.cuh"

namespace galore {

// ---------------------------------------------------------------------------
// small kernels
// ---------------------------------------------------------------------------

__device__ __forceinline__ uint64_t mix64(uint64_t x) {   // splitmix64 finaliser
  x += 0x9E3779B97F4A7C15ull;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}

// standard normal start block from a counter-based hash (Box-Muller)
__global__ void fill_normal_kernel(float* __restrict__ Y, int64_t count, uint64_t seed) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x) {
    uint64_t h = mix64(seed ^ mix64((uint64_t)i));
    float u1 = ((uint32_t)(h >> 40) + 1u) * (1.0f / 16777217.0f);   // (0, 1)
    float u2 = (uint32_t)(h & 0xFFFFFFu) * (1.0f / 16777216.0f);    // [0, 1)
    Y[i] = sqrtf(-2.0f * logf(u1)) * cospif(2.0f * u2);
  }
}

// first r columns of the start block <- the projector of the previous refresh (rows x r, packed)
template <typename TP>
__global__ void place_previous_kernel(float* __restrict__ Y, const TP* __restrict__ P, int64_t rows, int r, int b) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < rows * r; i += (int64_t)gridDim.x * blockDim.x)
    Y[(i / r) * b + (i % r)] = cvt<float>(P[i]);
}

__global__ void set_identity_kernel(double* __restrict__ A, int n) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < (int64_t)n * n; i += (int64_t)gridDim.x * blockDim.x)
    A[i] = (i / n == i % n) ? 1.0 : 0.0;
}

template <typename TS, typename TD>
__global__ void convert_kernel(const TS* __restrict__ src, TD* __restrict__ dst, int64_t count) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x)
    dst[i] = cvt<TD>(src[i]);
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// every thread of a 256-thread CTA gets the sum
__device__ __forceinline__ double block_sum_256(double v, double* red) {
  v = warp_sum(v);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  double r = 0.0;
#pragma unroll
  for (int w = 0; w < 8; ++w) r += red[w];
  __syncthreads();
  return r;
}

// part[blockIdx.x] = this CTA's share of the sum of squares (fixed grid, so the total is reproducible)
constexpr int kSumsqBlocks = 592;
__global__ void __launch_bounds__(256) sumsq_kernel(const float* __restrict__ x, int64_t count, double* __restrict__ part) {
  __shared__ double red[8];
  double s = 0.0;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x) {
    double v = x[i];
    s += v * v;
  }
  s = block_sum_256(s, red);
  if (threadIdx.x == 0) part[blockIdx.x] = s;
}

// Ynew += delta * Yold,  delta = max(1e-4 * rms column norm of Ynew, 1e-30)
__global__ void __launch_bounds__(256) shift_kernel(float* __restrict__ Ynew, const float* __restrict__ Yold, int64_t count,
                                                    int cols, const double* __restrict__ part) {
  __shared__ double red[8];
  double s = 0.0;
  for (int i = threadIdx.x; i < kSumsqBlocks; i += 256) s += part[i];
  s = block_sum_256(s, red);
  const float delta = fmaxf((float)(1e-4 * sqrt(s / (double)cols)), 1e-30f);
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x)
    Ynew[i] = fmaf(delta, Yold[i], Ynew[i]);
}

// ---- helpers of the tensor-core power step -----------------------------------------------------
// A value x is carried to the tensor cores as two bf16 numbers, hi = bf16(x) and lo = bf16(x - hi):
// products with exactly representable bf16 gradients then keep about 16 significant bits.
__device__ __forceinline__ void split_bf16(float x, __nv_bfloat16& hi, __nv_bfloat16& lo) {
  hi = __float2bfloat16_rn(x);
  lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}

// out = x0 + x1 (+ x2); optionally stored as fp32 and always as a hi/lo pair
__global__ void sum_split_kernel(const float* __restrict__ x0, const float* __restrict__ x1, const float* __restrict__ x2,
                                 float* __restrict__ out, __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo,
                                 int64_t count) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x) {
    float v = x0[i] + x1[i];
    if (x2) v += x2[i];
    if (out) out[i] = v;
    split_bf16(v, hi[i], lo[i]);
  }
}

// x0 += x1, and this CTA's share of the sum of squares of the result (fixed grid)
__global__ void __launch_bounds__(256) add_sumsq_kernel(float* __restrict__ x0, const float* __restrict__ x1, int64_t count,
                                                        double* __restrict__ part) {
  __shared__ double red[8];
  double s = 0.0;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x) {
    const float v = x0[i] + x1[i];
    x0[i] = v;
    s += (double)v * v;
  }
  s = block_sum_256(s, red);
  if (threadIdx.x == 0) part[blockIdx.x] = s;
}

// Ynew += delta * Yold, then the hi/lo pair of Ynew.  delta = 1e-2 x rms column norm here (1e-4 on
// the fp32 path): the pair carries about 16 bits, so directions kept alive only by the shift must
// stay well above 2^-16 of the dominant ones for the Gram matrix to remain positive definite.
__global__ void __launch_bounds__(256) shift_split_kernel(float* __restrict__ Ynew, const float* __restrict__ Yold,
                                                          int64_t count, int cols, const double* __restrict__ part,
                                                          __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo) {
  __shared__ double red[8];
  double s = 0.0;
  for (int i = threadIdx.x; i < kSumsqBlocks; i += 256) s += part[i];
  s = block_sum_256(s, red);
  const float rms = (float)sqrt(s / (double)cols);
  const float delta = fmaxf(1e-2f * rms, 1e-30f);
  const float scale = rms > 1e-30f ? 1.0f / rms : 1.0f;      // keeps magnitudes near 1 when steps are chained
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x) {
    const float v = fmaf(delta, Yold[i], Ynew[i]) * scale;
    Ynew[i] = v;
    split_bf16(v, hi[i], lo[i]);
  }
}

// One step of a degree-2 Chebyshev filter on B = A A^T over the damped interval [0, 2c] (half width c):
// first step Y1 = (B Y0 - c Y0) / c, second step Y2 = 2 (B Y1 - c Y1) / c - Y0 = T_2((B - c) / c) Y0.
// x0 + x1 is the hi/lo product B y; v = s (x0 + x1 - c y) - z (z: the block two steps back, or null),
// stored in x0 and as a hi/lo pair.
__global__ void __launch_bounds__(256) cheb_split_kernel(float* __restrict__ x0, const float* __restrict__ x1,
                                                         const float* __restrict__ y, const float* __restrict__ z, float c,
                                                         float s, int64_t count, __nv_bfloat16* __restrict__ hi,
                                                         __nv_bfloat16* __restrict__ lo) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x) {
    float v = s * fmaf(-c, y[i], x0[i] + x1[i]);
    if (z) v -= z[i];
    x0[i] = v;
    split_bf16(v, hi[i], lo[i]);
  }
}

// Rayleigh quotients of the block: ||z_i||^2 with Z = A^T Y (+ second partial of a hi/lo product).
// Slice s of kColSlices sums rows s, s + kColSlices, ...; slices are added in order afterwards.
constexpr int kColSlices = 64;
__global__ void colsumsq_partial_kernel(const float* __restrict__ z0, const float* __restrict__ z1, int64_t rows, int cols,
                                        double* __restrict__ part /* kColSlices x cols */) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= cols) return;
  double s = 0.0;
  for (int64_t i = blockIdx.y; i < rows; i += kColSlices) {
    float v = z0[i * cols + c];
    if (z1) v += z1[i * cols + c];
    s += (double)v * v;
  }
  part[(int64_t)blockIdx.y * cols + c] = s;
}
__global__ void colsumsq_final_kernel(const double* __restrict__ part, int cols, double* __restrict__ out) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= cols) return;
  double s = 0.0;
  for (int k = 0; k < kColSlices; ++k) s += part[(int64_t)k * cols + c];
  out[c] = s;
}

// C = g0 + g1 + g2 : the three bf16-pair products that make up a Gram matrix
__global__ void gram_sum_kernel(const float* __restrict__ g0, const float* __restrict__ g1, const float* __restrict__ g2,
                                float* __restrict__ C, int64_t count) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x)
    C[i] = (float)((double)g0[i] + (double)g1[i] + (double)g2[i]);
}

__global__ void split_kernel(const float* __restrict__ x, __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo,
                             int64_t count) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x)
    split_bf16(x[i], hi[i], lo[i]);
}

// ---- Cholesky of one diagonal block (nb <= 64) and the inverse of its factor ----
// C: the block inside a row-major matrix with leading dimension ld (lower triangle used and
// overwritten with L).  Linv: 64 x 64 row-major, lower triangular, zero elsewhere; rows and
// columns past nb continue the identity.
//
// Four threads per row: thread (row, part) keeps the 16 entries of its row in the columns
// 4 q + part in registers, every index a compile-time constant after unrolling.  Column j: the
// owner of the pivot publishes 1/sqrt, the rows below scale their entry and publish it, then
// every thread subtracts the rank-1 term from its entries right of j -- independent FMAs, no
// dependent chain.  The inverse is formed the same way: the threads of column c keep the running
// right-hand side of column c of L^-1, x_r = s_r / L_rr goes through shared memory to the other
// three parts, then s_k -= L_kr x_r for k > r.  (One thread per row with 64 entries each made
// the kernel four times longer in instructions, all executed once: it waited on instruction
// fetch.)
__device__ __forceinline__ double pivot_rsqrt(double x) { return rsqrt_newton(x); }
__device__ __forceinline__ float pivot_rsqrt(float x) { return rsqrtf(x); }

// blockIdx.x: position in the slot list (one CTA per workspace slot)
template <typename T>
__global__ void __launch_bounds__(256) potf2_inv_kernel(T* __restrict__ C, int ld, int nb, T* __restrict__ Linv,
                                                        int32_t* __restrict__ status, const SlotList slots) {
  {
    const int64_t shift = (int64_t)slots.id[blockIdx.x] * slots.bytes;
    C = slot_ptr(C, shift);
    Linv = slot_ptr(Linv, shift);
    status = slot_ptr(status, shift);
  }
  __shared__ T Ls[64][65];       // the factor: needed again for the inverse and for the write-back
  __shared__ T col[64];
  __shared__ T rdiag[64];
  __shared__ T xs[2][64];
  const int row = threadIdx.x & 63, part = threadIdx.x >> 6;
  T a[16];
#pragma unroll
  for (int q = 0; q < 16; ++q) {
    const int k = 4 * q + part;
    a[q] = (row < nb && k <= row) ? C[(int64_t)row * ld + k] : ((k == row) ? T(1) : T(0));
  }
#pragma unroll
  for (int j = 0; j < 64; ++j) {
    const int pj = j & 3, qj = j >> 2;
    if (row == j && part == pj) {
      T piv = a[qj];
      if (!(piv > T(0))) {             // not positive definite: keep going with a usable pivot, latch the fact
        atomicOr(status, GALORE_DEV_CHOLESKY);
        piv = (T)(fabs((double)piv) + 1e-30);
      }
      const T rs = pivot_rsqrt(piv);
      Ls[j][j] = piv * rs;
      rdiag[j] = rs;
    }
    __syncthreads();
    if (part == pj) {
      T l = T(0);
      if (row > j) {
        l = a[qj] * rdiag[j];
        Ls[row][j] = l;
      }
      col[row] = l;
    }
    __syncthreads();
    const T l = col[row];
#pragma unroll
    for (int q = qj; q < 16; ++q) {
      if (q > qj || part > pj) a[q] = fma(-l, col[4 * q + part], a[q]);
    }
  }
  __syncthreads();
  // column `row` of L^-1, entries 4 q + part
#pragma unroll
  for (int q = 0; q < 16; ++q) a[q] = (4 * q + part == row) ? T(1) : T(0);
#pragma unroll
  for (int r = 0; r < 64; ++r) {
    const int pr = r & 3, qr = r >> 2;
    if (part == pr) {
      const T x = a[qr] * rdiag[r];
      a[qr] = x;
      xs[r & 1][row] = x;
    }
    __syncthreads();
    const T x = xs[r & 1][row];
#pragma unroll
    for (int q = qr; q < 16; ++q) {
      if (q > qr || part > pr) a[q] = fma(-Ls[4 * q + part][r], x, a[q]);
    }
  }
#pragma unroll
  for (int q = 0; q < 16; ++q) Linv[(4 * q + part) * 64 + row] = a[q];
  for (int idx = threadIdx.x; idx < 64 * 64; idx += 256) {
    const int r = idx >> 6, c = idx & 63;
    if (r < nb && c <= r) C[(int64_t)r * ld + c] = Ls[r][c];
  }
}

// diagonal 64 x 64 blocks of T <- the inverses of the diagonal blocks of L (slab p = block p)
template <typename S>
__global__ void place_diag_inverse_kernel(const S* __restrict__ slabs, int b, S* __restrict__ T, const SlotList slots) {
  {
    const int64_t shift = (int64_t)slots.id[blockIdx.y] * slots.bytes;     // blockIdx.y: workspace slot
    slabs = slot_ptr(slabs, shift);
    T = slot_ptr(T, shift);
  }
  const int p = blockIdx.x, j0 = p * 64;
  const int nb = min(64, b - j0);
  for (int idx = threadIdx.x; idx < 64 * 64; idx += blockDim.x) {
    const int r = idx >> 6, c = idx & 63;
    if (r < nb && c < nb) T[(int64_t)(j0 + r) * b + j0 + c] = slabs[(int64_t)p * 4096 + idx];
  }
}

__global__ void __launch_bounds__(256) row_norm_kernel(const double* __restrict__ X, int b, double* __restrict__ lam) {
  __shared__ double red[8];
  const double* x = X + (int64_t)blockIdx.x * b;
  double s = 0.0;
  for (int j = threadIdx.x; j < b; j += 256) s += x[j] * x[j];
  s = block_sum_256(s, red);
  if (threadIdx.x == 0) lam[blockIdx.x] = sqrt(s);
}

// descending order by counting: theta[rank] = lam[i], order[rank] = i
__global__ void rank_desc_kernel(const double* __restrict__ lam, int b, double* __restrict__ theta, int* __restrict__ order) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= b) return;
  const double li = lam[i];
  int rank = 0;
  for (int j = 0; j < b; ++j) {
    double lj = lam[j];
    rank += (lj > li) || (lj == li && j < i);
  }
  theta[rank] = li;
  order[rank] = i;
}

__global__ void gather_rows_kernel(const double* __restrict__ Vt, const int* __restrict__ order, int b,
                                   double* __restrict__ Vsel) {
  const double* src = Vt + (int64_t)order[blockIdx.x] * b;
  double* dst = Vsel + (int64_t)blockIdx.x * b;
  for (int j = threadIdx.x; j < b; j += blockDim.x) dst[j] = src[j];
}

// rows of X = Theta V^T divided by their norms: the eigenvectors themselves
__global__ void gather_rows_scaled_kernel(const double* __restrict__ X, const double* __restrict__ lam,
                                          const int* __restrict__ order, int b, double* __restrict__ Vsel) {
  const int i = order[blockIdx.x];
  const double* src = X + (int64_t)i * b;
  const double inv = lam[i] > 0.0 ? 1.0 / lam[i] : 0.0;
  double* dst = Vsel + (int64_t)blockIdx.x * b;
  for (int j = threadIdx.x; j < b; j += blockDim.x) dst[j] = src[j] * inv;
}

// scal[1] += || T2 - P diag(theta) ||_F^2
__global__ void __launch_bounds__(256) residual_kernel(const double* __restrict__ T2, const double* __restrict__ P,
                                                       const double* __restrict__ theta, int64_t rows, int r,
                                                       double* __restrict__ scal) {
  __shared__ double red[8];
  double s = 0.0;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < rows * r; i += (int64_t)gridDim.x * blockDim.x) {
    double d = T2[i] - theta[i % r] * P[i];
    s += d * d;
  }
  s = block_sum_256(s, red);
  if (threadIdx.x == 0) atomicAdd(scal + 1, s);
}

// the same with T2 given as two fp32 partial products
__global__ void __launch_bounds__(256) residual_pair_kernel(const float* __restrict__ t0, const float* __restrict__ t1,
                                                            const double* __restrict__ P, const double* __restrict__ theta,
                                                            int64_t rows, int r, double* __restrict__ scal) {
  __shared__ double red[8];
  double s = 0.0;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < rows * r; i += (int64_t)gridDim.x * blockDim.x) {
    double d = ((double)t0[i] + (double)t1[i]) - theta[i % r] * P[i];
    s += d * d;
  }
  s = block_sum_256(s, red);
  if (threadIdx.x == 0) atomicAdd(scal + 1, s);
}

// GEMM epilogue: the result as a bf16 hi/lo pair
struct EpiSplitPair {
  __nv_bfloat16 *hi, *lo;
  int64_t ld;
  __device__ __forceinline__ void shift(int64_t bytes) {
    hi = slot_ptr(hi, bytes);
    lo = slot_ptr(lo, bytes);
  }
  __device__ __forceinline__ void operator()(int i, int j, double acc, int) const {
    split_bf16((float)acc, hi[(int64_t)i * ld + j], lo[(int64_t)i * ld + j]);
  }
};

// status |= flags; flags = 0  (what the slot-wise kernels latched goes to the layer's own status word)
__global__ void merge_flags_kernel(int32_t* __restrict__ status, int32_t* __restrict__ flags) {
  if (*flags) atomicOr(status, *flags);
  *flags = 0;
}

static inline unsigned grid_for(int64_t count) { return (unsigned)std::min<int64_t>(ceil_div(count, 256), 148 * 8); }

// ---------------------------------------------------------------------------
// workspace
// ---------------------------------------------------------------------------

struct RefreshBuffers {
  float* Ya;      // d x b
  float* Yb;      // d x b
  void* Zu;       // L x b, fp32 during power steps, fp64 during Rayleigh-Ritz
  double* Y64;    // d x b
  double* C;      // b x b  Gram / Cholesky factor
  double* H;      // b x b  Jacobi working matrix
  double* Vt;     // b x b
  double* P64;    // d x r
  double* Vsel;   // r x b
  double* tmp;    // d x 64
  double* Linv;   // 64 x 64
  double* lam;    // b
  double* theta;  // b
  int* order;     // b
  double* scal;   // 4 scalars
  double* part;   // kSumsqBlocks partial sums
  int* counter;   // 1
  int32_t* flags; // device status bits latched by kernels that run for several slots at once
  void* jac;      // scratch of the Jacobi eigensolver
  double* slabs;  // ceil(b / 64) inverses of 64 x 64 diagonal blocks
  // tensor-core power steps
  float* Yc;                 // d x b, third fp32 block
  __nv_bfloat16 *Yhi, *Ylo;  // d x b
  __nv_bfloat16 *Zhi, *Zlo;  // L x b
  __nv_bfloat16 *Thi, *Tlo;  // b x b, inverse Cholesky factor
};

static size_t carve(char*& p, size_t bytes) {
  size_t a = align_up(bytes, 256);
  p += a;
  return a;
}

size_t refresh_workspace_bytes(int64_t d, int64_t L, int r, int b) {
  size_t t = 0;
  t += align_up((size_t)d * b * 4, 256) * 2;
  t += align_up((size_t)L * b * 8, 256);
  t += align_up((size_t)d * b * 8, 256);
  t += align_up((size_t)b * b * 8, 256) * 3;
  t += align_up((size_t)d * r * 8, 256);
  t += align_up((size_t)r * b * 8, 256);
  t += align_up((size_t)d * 64 * 8, 256);
  t += align_up((size_t)64 * 64 * 8, 256);
  t += align_up((size_t)b * 8, 256) * 2;
  t += align_up((size_t)b * 4, 256);
  t += 256 * 2 + 8 * 1024;
  t += align_up(jacobi_scratch_bytes(b), 256);
  t += align_up((size_t)ceil_div(b, 64) * 4096 * 8, 256);
  t += align_up((size_t)d * b * 4, 256) + 2 * align_up((size_t)d * b * 2, 256) + 2 * align_up((size_t)L * b * 2, 256) +
       2 * align_up((size_t)b * b * 2, 256);
  return t;
}

static RefreshBuffers layout(void* base, int64_t d, int64_t L, int r, int b) {
  RefreshBuffers w;
  char* p = (char*)base;
  w.Ya = (float*)p; carve(p, (size_t)d * b * 4);
  w.Yb = (float*)p; carve(p, (size_t)d * b * 4);
  w.Zu = (void*)p; carve(p, (size_t)L * b * 8);
  w.Y64 = (double*)p; carve(p, (size_t)d * b * 8);
  w.C = (double*)p; carve(p, (size_t)b * b * 8);
  w.H = (double*)p; carve(p, (size_t)b * b * 8);
  w.Vt = (double*)p; carve(p, (size_t)b * b * 8);
  w.P64 = (double*)p; carve(p, (size_t)d * r * 8);
  w.Vsel = (double*)p; carve(p, (size_t)r * b * 8);
  w.tmp = (double*)p; carve(p, (size_t)d * 64 * 8);
  w.Linv = (double*)p; carve(p, (size_t)64 * 64 * 8);
  w.lam = (double*)p; carve(p, (size_t)b * 8);
  w.theta = (double*)p; carve(p, (size_t)b * 8);
  w.order = (int*)p; carve(p, (size_t)b * 4);
  w.scal = (double*)p; carve(p, 256);
  w.part = (double*)p; carve(p, 8 * 1024);
  w.counter = (int*)p; w.flags = (int32_t*)(p + 64); carve(p, 256);
  w.jac = (void*)p; carve(p, jacobi_scratch_bytes(b));
  w.slabs = (double*)p; carve(p, (size_t)ceil_div(b, 64) * 4096 * 8);
  w.Yc = (float*)p; carve(p, (size_t)d * b * 4);
  w.Yhi = (__nv_bfloat16*)p; carve(p, (size_t)d * b * 2);
  w.Ylo = (__nv_bfloat16*)p; carve(p, (size_t)d * b * 2);
  w.Zhi = (__nv_bfloat16*)p; carve(p, (size_t)L * b * 2);
  w.Zlo = (__nv_bfloat16*)p; carve(p, (size_t)L * b * 2);
  w.Thi = (__nv_bfloat16*)p; carve(p, (size_t)b * b * 2);
  w.Tlo = (__nv_bfloat16*)p; carve(p, (size_t)b * b * 2);
  return w;
}

const double* refresh_unrounded_projector(void* workspace, int64_t d, int64_t L, int r, int b) {
  return layout(workspace, d, L, r, b).P64;
}

// ---------------------------------------------------------------------------
// A group of layers of one shape refreshed together
// ---------------------------------------------------------------------------
// Each layer ("lane") owns one slot of the workspace, all slots laid out alike.  The tensor-core
// products take the lanes' problems in one grouped launch; the latency-bound small kernels
// (Cholesky panels, triangular inverses, the Jacobi eigen-solver) run for all lanes in one launch
// per kernel, their workspace pointers shifted per slot; element-wise kernels and everything that
// touches a layer's own G or P are launched lane by lane.  Every lane makes exactly the steps it
// would make on its own (its own iteration count and orthonormalisation schedule), so a layer's
// projector does not depend on what it was grouped with.

// Chebyshev acceleration of slowly converging blocks: used when the look asks for more than this many
// further plain steps, and only while T_2 at theta_1 (the growth of the block's condition number over a
// pair, which the bf16 pairs and the squared Gram matrix have to carry) stays below the second constant.
constexpr int kChebyshevFrom = 8;
constexpr double kChebyshevSpread = 150.0;
static inline double cheb_t2(double x) { return 2.0 * x * x - 1.0; }

struct TensorRefresh {
  float* F[4];          // fp32 d x b buffers; F[master] holds Y.  F[3] (the idle upper half of Y64) only ever
  int master;           // receives the second partial product of the closing step of a Chebyshev pair
  int prev = -1;        // buffer of the block one step back, between the two steps of a Chebyshev pair
};
// one run of Chebyshev pairs with a fixed interval
struct ChebSegment {
  double c;             // centre = half width of the damped interval [0, 2c]
  int pairs;
};

struct Lane {
  RefreshProblem pr;
  int slot;
  char* base;                 // start of the lane's slot
  RefreshBuffers w;
  int32_t* status;            // the layer's own status word
  float *Y, *Yn;              // current block and the other buffer (FMA path)
  TensorRefresh tr;
  int q_done = 0, q_target = 0, orth_every = 1;
  std::vector<double> theta;
  double predicted = 0.0, res_abs = 0.0;
  bool converged = false, with_vt = false, iterating = true;
  bool cheb = false;          // power steps come in pairs that apply T_2 of the shifted operator
  int q_plain = 0;            // plain power steps among q_done
  std::vector<ChebSegment> segs;
  bool p64_current = false;   // P64 holds the Ritz vectors of the lane's last Rayleigh-Ritz pass
  bool warm_check = false;    // started from the previous projector: the first Rayleigh-Ritz pass is judged by its residual
  int warm_from = 0;          // steps done when the warm start was judged, and the error bound found there
  double warm_bound = 1.0;    // (a cold start: 0 steps, error 1)
  galore_refresh_info_t info = {};
};

struct Ctx {
  char* base0;                // slot 0 of the workspace
  int64_t slot_bytes;
  int64_t d, L;
  int r, b;
  bool left, tensor;
  RefreshBuffers w0;          // slot 0's buffers: what a launch over a slot list is given
  TensorGroup* tg;
  cudaStream_t st;
};

// lanes whose pointers sit at the same place inside their slots can share a launch
struct LaneSet {
  int64_t off_a, off_b;
  SlotList list;
  std::vector<Lane*> lanes;
};
template <class KeyA, class KeyB>
static std::vector<LaneSet> sets_of(const Ctx& c, const std::vector<Lane*>& lanes, KeyA a_of, KeyB b_of) {
  std::vector<LaneSet> out;
  for (Lane* l : lanes) {
    const int64_t oa = (const char*)a_of(l) - l->base, ob = (const char*)b_of(l) - l->base;
    LaneSet* g = nullptr;
    for (LaneSet& x : out)
      if (x.off_a == oa && x.off_b == ob) g = &x;
    if (!g) {
      out.push_back(LaneSet{});
      g = &out.back();
      g->off_a = oa;
      g->off_b = ob;
      g->list = SlotList{};
      g->list.bytes = c.slot_bytes;
    }
    g->list.id[g->list.n++] = l->slot;
    g->lanes.push_back(l);
  }
  return out;
}
static SlotList slots_of(const Ctx& c, const std::vector<Lane*>& lanes) {
  SlotList s = {};
  s.bytes = c.slot_bytes;
  for (Lane* l : lanes) s.id[s.n++] = l->slot;
  return s;
}

// C (b x b, fp64, at `dst` of slot 0) = Y^T Y, Y (rows x b) at src(lane)
template <typename TY, class Src>
static galore_status_t gram(const Ctx& c, const std::vector<Lane*>& lanes, Src src, int64_t rows, double* dst0) {
  for (const LaneSet& g : sets_of(c, lanes, src, src)) {
    const TY* Y0 = (const TY*)(c.base0 + g.off_a);
    EpiStore<double, double> epi{dst0, c.b, 0, 1.0, 0.0};
    GALORE_TRY((launch_gemm_dmma<TY, TY>(c.b, c.b, (int)rows, Y0, 1, c.b, Y0, c.b, 1, epi, c.st, 1, 0, 0, &g.list)));
  }
  return GALORE_OK;
}

// Blocked Cholesky of the b x b matrix C (lower triangle, in place), then T = L^-1 (b x b, lower,
// zero above the diagonal), in every listed slot; pointers name slot 0's copies.
//   factor : per 64-wide panel the diagonal block (with its inverse, kept in w.slabs), the panel
//            below it and the trailing update;
//   invert : the inverses of the diagonal blocks are merged pairwise, level by level,
//            [T11 0; T21 T22] with T21 = -T22 L21 T11, every level two batched products.
// scratch: b*b/4 elements.
// (S = double: products on the fp64 MMA unit; S = float, used between the tensor-core power steps
// whose Gram matrices carry about 16 bits anyway: FMA products and a ten times shorter pivot chain.)
template <typename TA, typename TB, typename S, class Epi>
static galore_status_t gemm_scalar(int M, int N, int K, const TA* A, int64_t sAi, int64_t sAk, const TB* B, int64_t sBk,
                                   int64_t sBj, Epi epi, cudaStream_t st, const SlotList& sl, int batch = 1, int64_t bA = 0,
                                   int64_t bB = 0, bool lower_only = false) {
  if constexpr (std::is_same<S, double>::value)
    return launch_gemm_dmma<TA, TB>(M, N, K, A, sAi, sAk, B, sBk, sBj, epi, st, batch, bA, bB, &sl);
  else
    return launch_gemm_simt<TA, TB, float>(M, N, K, A, sAi, sAk, B, sBk, sBj, 1, epi, st, batch, bA, bB, &sl, lower_only);
}

template <typename S>
static galore_status_t cholesky_inverse(const Ctx& c, const SlotList& sl, S* C, S* T, S* scratch) {
  const int b = c.b;
  cudaStream_t st = c.st;
  const int nblk = (int)ceil_div(b, 64);
  S* slabs = (S*)c.w0.slabs;
  for (int p = 0; p < nblk; ++p) {
    const int j0 = p * 64, nb = std::min(64, b - j0), j1 = j0 + nb;
    S* slab = slabs + (int64_t)p * 4096;
    potf2_inv_kernel<S><<<sl.n, 256, 0, st>>>(C + (int64_t)j0 * b + j0, b, nb, slab, c.w0.flags, sl);
    GALORE_LAUNCH_CHECK();
    if (j1 < b) {
      const int rem = b - j1;
      S* panel = C + (int64_t)j1 * b + j0;
      // L[rest, J] = C[rest, J] Linv^T   (in place: one CTA column covers all nb columns)
      EpiStore<S, S> epi{panel, b, 0, S(1), S(0)};
      GALORE_TRY((gemm_scalar<S, S, S>(rem, nb, nb, panel, b, 1, slab, 1, 64, epi, st, sl)));
      // C[rest, rest] -= L[rest, J] L[rest, J]^T  (only the lower triangle of C is ever read: tiles above the
      // diagonal are left out where the kernel can)
      EpiStore<S, S> upd{C + (int64_t)j1 * b + j1, b, 0, S(-1), S(1)};
      GALORE_TRY((gemm_scalar<S, S, S>(rem, rem, nb, panel, b, 1, panel, 1, b, upd, st, sl, 1, 0, 0, true)));
    }
  }
  for (int i = 0; i < sl.n; ++i)
    GALORE_CUDA_TRY(cudaMemsetAsync(slot_ptr(T, (int64_t)sl.id[i] * sl.bytes), 0, sizeof(S) * b * b, st));
  place_diag_inverse_kernel<S><<<dim3(nblk, sl.n), 256, 0, st>>>(slabs, b, T, sl);
  GALORE_LAUNCH_CHECK();
  for (int64_t s = 64; s < b; s *= 2) {
    const int64_t step = 2 * s * b + 2 * s;            // from one merged block to the next, in elements
    const int full = (int)(b / (2 * s));               // blocks with a complete lower half
    const int tail = (int)(b % (2 * s)) - (int)s;      // rows of a ragged last lower half (<= 0: none)
    for (int pass = 0; pass < 2; ++pass) {
      const int count = pass == 0 ? full : (tail > 0 ? 1 : 0);
      if (count == 0) continue;
      const int s2 = pass == 0 ? (int)s : tail;
      const int64_t o = pass == 0 ? 0 : (int64_t)full * 2 * s;
      const S* L21 = C + (o + s) * b + o;
      const S* T11 = T + o * b + o;
      const S* T22 = T + (o + s) * b + (o + s);
      S* T21 = T + (o + s) * b + o;
      // W = L21 T11
      EpiStore<S, S> ew{scratch, s, s * s, S(1), S(0)};
      GALORE_TRY((gemm_scalar<S, S, S>(s2, (int)s, (int)s, L21, b, 1, T11, b, 1, ew, st, sl, count, step, step)));
      // T21 = -T22 W
      EpiStore<S, S> et{T21, b, step, S(-1), S(0)};
      GALORE_TRY((gemm_scalar<S, S, S>(s2, (int)s, s2, T22, b, 1, scratch, s, 1, et, st, sl, count, step, s * s)));
    }
  }
  return GALORE_OK;
}

// out = Y L^-T with L L^T = Y^T Y (CholeskyQR), Y at src(lane), out at dst(lane); out must not alias Y.
// Uses C, Vt, H of every lane.
template <typename TY, typename TO, class Src, class Dst>
static galore_status_t orthonormalise(const Ctx& c, const std::vector<Lane*>& lanes, Src src, Dst dst) {
  GALORE_TRY((gram<TY>(c, lanes, src, c.d, c.w0.C)));
  GALORE_TRY(cholesky_inverse<double>(c, slots_of(c, lanes), c.w0.C, c.w0.Vt, c.w0.H));
  for (const LaneSet& g : sets_of(c, lanes, src, dst)) {
    EpiStore<TO, double> epi{(TO*)(c.base0 + g.off_b), c.b, 0, 1.0, 0.0};
    GALORE_TRY((launch_gemm_dmma<TY, double>((int)c.d, c.b, c.b, (const TY*)(c.base0 + g.off_a), c.b, 1, c.w0.Vt, 1, c.b, epi,
                                             c.st, 1, 0, 0, &g.list)));
  }
  return GALORE_OK;
}

// ---- power step on the tensor cores -------------------------------------------------------------
// The block Y lives as an fp32 master (one of three d x b buffers) plus its bf16 hi/lo pair.  Every
// product below is a tcgen05 GEMM on bf16 operands with fp32 output; a product with a hi/lo operand
// is two (or three) problems of one grouped launch whose outputs are added afterwards.  The
// problems of all lanes travel in the same grouped launches.

// Y <- Y L^-T with L L^T = Y^T Y: CholeskyQR whose two big products run on the tensor cores.
// In: hi/lo pair of Y valid (the fp32 master itself is not read).  Out: master and pair updated.
static galore_status_t orth_tensor(const Ctx& c, const std::vector<Lane*>& lanes) {
  if (lanes.empty()) return GALORE_OK;
  const int b = c.b;
  const int64_t d = c.d, bb = (int64_t)b * b, yb = d * b;
  cudaStream_t st = c.st;
  tensor_group_reset(c.tg);   // Gram = (hi + lo)^T (hi + lo) without the lo^T lo term
  for (Lane* l : lanes) {
    const RefreshBuffers& w = l->w;
    float* g0 = (float*)w.H;
    float* g1 = g0 + bb;
    float* g2 = (float*)w.Y64;
    GALORE_TRY(tensor_group_add_gemm(c.tg, w.Yhi, b, 1, w.Yhi, b, 1, b, b, (int)d, g0, b, l->status));
    GALORE_TRY(tensor_group_add_gemm(c.tg, w.Yhi, b, 1, w.Ylo, b, 1, b, b, (int)d, g1, b, l->status));
    GALORE_TRY(tensor_group_add_gemm(c.tg, w.Ylo, b, 1, w.Yhi, b, 1, b, b, (int)d, g2, b, l->status));
  }
  GALORE_TRY(tensor_group_launch_project(c.tg, st));
  for (Lane* l : lanes) {
    const RefreshBuffers& w = l->w;
    gram_sum_kernel<<<grid_for(bb), 256, 0, st>>>((float*)w.H, (float*)w.H + bb, (float*)w.Y64, (float*)w.C, bb);
    GALORE_LAUNCH_CHECK();
  }
  // T = L^-1, split into a bf16 pair; as the second operand of Y L^-T it is read K-contiguous
  GALORE_TRY(cholesky_inverse<float>(c, slots_of(c, lanes), (float*)c.w0.C, (float*)c.w0.Vt, (float*)c.w0.H));
  for (Lane* l : lanes) {
    split_kernel<<<grid_for(bb), 256, 0, st>>>((const float*)l->w.Vt, l->w.Thi, l->w.Tlo, bb);
    GALORE_LAUNCH_CHECK();
  }
  tensor_group_reset(c.tg);   // Y T = hi Thi + hi Tlo + lo Thi
  for (Lane* l : lanes) {
    const RefreshBuffers& w = l->w;
    TensorRefresh& t = l->tr;
    const int m = t.master, s1 = (m + 1) % 3, s2 = (m + 2) % 3;
    GALORE_TRY(tensor_group_add_gemm(c.tg, w.Yhi, b, 0, w.Thi, b, 0, (int)d, b, b, t.F[m], b, l->status));
    GALORE_TRY(tensor_group_add_gemm(c.tg, w.Yhi, b, 0, w.Tlo, b, 0, (int)d, b, b, t.F[s1], b, l->status));
    GALORE_TRY(tensor_group_add_gemm(c.tg, w.Ylo, b, 0, w.Thi, b, 0, (int)d, b, b, t.F[s2], b, l->status));
  }
  GALORE_TRY(tensor_group_launch_project(c.tg, st));
  for (Lane* l : lanes) {
    TensorRefresh& t = l->tr;
    const int m = t.master, s1 = (m + 1) % 3, s2 = (m + 2) % 3;
    sum_split_kernel<<<grid_for(yb), 256, 0, st>>>(t.F[m], t.F[s1], t.F[s2], t.F[m], l->w.Yhi, l->w.Ylo, yb);
    GALORE_LAUNCH_CHECK();
  }
  return GALORE_OK;
}

// Z = A^T Y ; Y' = A Z + delta Y for every lane; then Y = orth(Y') for the lanes in `orth`
static galore_status_t power_step_tensor(const Ctx& c, const std::vector<Lane*>& lanes, const std::vector<Lane*>& orth) {
  if (lanes.empty()) return GALORE_OK;
  const int b = c.b;
  const int64_t d = c.d, L = c.L, zb = L * b, yb = d * b;
  cudaStream_t st = c.st;
  const int at_mn = c.left ? 1 : 0;   // A^T as the first operand: G^T (left) is M-contiguous in G, G (right) is K-contiguous
  const int a_mn = c.left ? 0 : 1;    // A as the first operand
  tensor_group_reset(c.tg);
  for (Lane* l : lanes) {
    float* z0 = (float*)l->w.Zu;
    GALORE_TRY(tensor_group_add_gemm(c.tg, l->pr.G, l->pr.ldg, at_mn, l->w.Yhi, b, 1, (int)L, b, (int)d, z0, b, l->status));
    GALORE_TRY(tensor_group_add_gemm(c.tg, l->pr.G, l->pr.ldg, at_mn, l->w.Ylo, b, 1, (int)L, b, (int)d, z0 + zb, b, l->status));
  }
  GALORE_TRY(tensor_group_launch_project(c.tg, st));
  for (Lane* l : lanes) {
    float* z0 = (float*)l->w.Zu;
    sum_split_kernel<<<grid_for(zb), 256, 0, st>>>(z0, z0 + zb, nullptr, nullptr, l->w.Zhi, l->w.Zlo, zb);
    GALORE_LAUNCH_CHECK();
  }
  // outputs of the two partial products: two buffers that hold neither Y nor, inside a Chebyshev pair, the block before it
  auto outputs = [](const TensorRefresh& t, int& o1, int& o2) {
    if (t.prev < 0) {
      o1 = (t.master + 1) % 3;
      o2 = (t.master + 2) % 3;
    } else {
      o1 = 3 - t.master - t.prev;     // the third of the buffers 0, 1, 2
      o2 = 3;
    }
  };
  tensor_group_reset(c.tg);
  for (Lane* l : lanes) {
    TensorRefresh& t = l->tr;
    int s1, s2;
    outputs(t, s1, s2);
    GALORE_TRY(tensor_group_add_gemm(c.tg, l->pr.G, l->pr.ldg, a_mn, l->w.Zhi, b, 1, (int)d, b, (int)L, t.F[s1], b, l->status));
    GALORE_TRY(tensor_group_add_gemm(c.tg, l->pr.G, l->pr.ldg, a_mn, l->w.Zlo, b, 1, (int)d, b, (int)L, t.F[s2], b, l->status));
  }
  GALORE_TRY(tensor_group_launch_project(c.tg, st));
  for (Lane* l : lanes) {
    TensorRefresh& t = l->tr;
    const int m = t.master;
    int s1, s2;
    outputs(t, s1, s2);
    if (!l->cheb) {
      add_sumsq_kernel<<<kSumsqBlocks, 256, 0, st>>>(t.F[s1], t.F[s2], yb, l->w.part);
      GALORE_LAUNCH_CHECK();
      shift_split_kernel<<<grid_for(yb), 256, 0, st>>>(t.F[s1], t.F[m], yb, b, l->w.part, l->w.Yhi, l->w.Ylo);
      GALORE_LAUNCH_CHECK();
      l->q_plain += 1;
    } else {
      const float cc = (float)l->segs.back().c, inv = (float)(1.0 / l->segs.back().c);
      if (t.prev < 0) {       // opening step of a pair: the block it starts from is needed once more
        cheb_split_kernel<<<grid_for(yb), 256, 0, st>>>(t.F[s1], t.F[s2], t.F[m], nullptr, cc, inv, yb, l->w.Yhi, l->w.Ylo);
        t.prev = m;
      } else {
        cheb_split_kernel<<<grid_for(yb), 256, 0, st>>>(t.F[s1], t.F[s2], t.F[m], t.F[t.prev], cc, 2.0f * inv, yb, l->w.Yhi,
                                                        l->w.Ylo);
        t.prev = -1;
        l->segs.back().pairs += 1;
      }
      GALORE_LAUNCH_CHECK();
    }
    t.master = s1;
    l->Y = t.F[t.master];
  }
  return orth_tensor(c, orth);
}

// the same step with FMA products (any dtype, any leading dimension); always ends orthonormal
template <typename TG>
static galore_status_t power_step_fma(const Ctx& c, const std::vector<Lane*>& lanes) {
  if (lanes.empty()) return GALORE_OK;
  const int b = c.b;
  const int64_t d = c.d, L = c.L, yb = d * b;
  cudaStream_t st = c.st;
  for (Lane* l : lanes) {
    const TG* G = (const TG*)l->pr.G;
    const int64_t sAi = c.left ? l->pr.ldg : 1;    // A(i, l) = G[i*sAi + l*sAl]
    const int64_t sAl = c.left ? 1 : l->pr.ldg;
    float* Z = (float*)l->w.Zu;
    {  // Z = A^T Y   (L x b)
      EpiStore<float, float> epi{Z, b, 0, 1.f, 0.f};
      GALORE_TRY((launch_gemm_simt<TG, float, float>((int)L, b, (int)d, G, sAl, sAi, l->Y, b, 1, 1, epi, st)));
    }
    {  // Y' = A Z     (d x b)
      EpiStore<float, float> epi{l->Yn, b, 0, 1.f, 0.f};
      GALORE_TRY((launch_gemm_simt<TG, float, float>((int)d, b, (int)L, G, sAi, sAl, Z, b, 1, 1, epi, st)));
    }
    sumsq_kernel<<<kSumsqBlocks, 256, 0, st>>>(l->Yn, yb, l->w.part);
    GALORE_LAUNCH_CHECK();
    shift_kernel<<<grid_for(yb), 256, 0, st>>>(l->Yn, l->Y, yb, b, l->w.part);
    GALORE_LAUNCH_CHECK();
  }
  // the old block is no longer needed: it receives the result
  return orthonormalise<float, float>(c, lanes, [](Lane* l) { return l->Yn; }, [](Lane* l) { return l->Y; });
}

template <typename TG>
static galore_status_t refresh_group(const RefreshProblem* prs, int count, void* workspace, size_t slot_bytes,
                                     int32_t* const* status, galore_refresh_info_t* infos, cudaStream_t st) {
  if (count < 1 || count > kMaxSlots) return GALORE_ERR_INVALID_ARG;
  NvtxRange whole("galore.refresh");
  const RefreshProblem& p0 = prs[0];
  Ctx c = {};
  c.base0 = (char*)workspace;
  c.slot_bytes = (int64_t)slot_bytes;
  c.left = p0.left;
  c.d = p0.left ? p0.m : p0.n;
  c.L = p0.left ? p0.n : p0.m;
  c.r = p0.rank;
  c.b = p0.block;
  c.st = st;
  const int64_t d = c.d, L = c.L;
  const int r = c.r, b = c.b;
  c.w0 = layout(workspace, d, L, r, b);
  const bool full_space = (b == d);
  // tensor cores carry the power steps when the gradients are bf16 and everything is TMA-addressable
  bool tensor = p0.use_tensor && !full_space && sizeof(TG) == 2 && (b % 8) == 0;
  for (int i = 0; i < count; ++i) tensor = tensor && (prs[i].ldg % 8) == 0 && (((uintptr_t)prs[i].G) & 15) == 0;
  c.tensor = tensor;
  struct GroupGuard {
    TensorGroup* g;
    ~GroupGuard() { tensor_group_free(g); }
  } guard{nullptr};
  if (tensor) {
    guard.g = c.tg = tensor_group_new();
    if (!c.tg) return GALORE_ERR_INVALID_ARG;
  }

  std::vector<Lane> store(count);
  std::vector<Lane*> all;
  const int64_t yb = d * b;
  for (int i = 0; i < count; ++i) {
    Lane& l = store[i];
    l.pr = prs[i];
    l.slot = i;
    l.base = c.base0 + (int64_t)i * c.slot_bytes;
    l.w = layout(l.base, d, L, r, b);
    l.status = status[i];
    l.Y = l.w.Ya;
    l.Yn = l.w.Yb;
    l.tr.F[0] = l.w.Ya; l.tr.F[1] = l.w.Yb; l.tr.F[2] = l.w.Yc;
    l.tr.F[3] = (float*)l.w.Y64 + yb;
    l.tr.master = 0;
    l.theta.assign(b, 0.0);
    l.info.block = b;
    l.converged = full_space;
    all.push_back(&l);
    GALORE_CUDA_TRY(cudaMemsetAsync(l.w.flags, 0, sizeof(int32_t), st));
  }

  // phase clock (only when the caller wants the record): host time at points where the stream is idle
  using clk = std::chrono::steady_clock;
  const bool timed = infos != nullptr;
  auto now_synced = [&]() {
    if (timed) cudaStreamSynchronize(st);
    return clk::now();
  };
  auto ms_between = [](clk::time_point a, clk::time_point b2) { return std::chrono::duration<double, std::milli>(b2 - a).count(); };
  double ms_ritz = 0.0, ms_jacobi = 0.0, ms_power = 0.0;
  const clk::time_point t_begin = now_synced();

  auto step = [&](const std::vector<Lane*>& lanes, const std::vector<Lane*>& orth) -> galore_status_t {
    if (tensor) return power_step_tensor(c, lanes, orth);
    return power_step_fma<TG>(c, lanes);
  };
  auto read_theta = [&](const std::vector<Lane*>& lanes) -> galore_status_t {
    for (Lane* l : lanes)
      GALORE_CUDA_TRY(cudaMemcpyAsync(l->theta.data(), l->w.theta, sizeof(double) * b, cudaMemcpyDeviceToHost, st));
    GALORE_CUDA_TRY(cudaStreamSynchronize(st));
    return GALORE_OK;
  };

  // power steps for the given lanes, every lane up to its own target on its own orthonormalisation schedule
  auto run_steps = [&](const std::vector<Lane*>& lanes) -> galore_status_t {
    for (;;) {
      std::vector<Lane*> stepping, orth;
      for (Lane* l : lanes)
        if (l->q_done < l->q_target) {
          stepping.push_back(l);
          if (((l->q_target - 1 - l->q_done) % l->orth_every) == 0) orth.push_back(l);   // the last step always ends orthonormal
        }
      if (stepping.empty()) return GALORE_OK;
      GALORE_TRY(step(stepping, orth));
      for (Lane* l : stepping) l->q_done += 1;
    }
  };

  if (!full_space) {
    for (Lane* l : all) {
      fill_normal_kernel<<<grid_for(yb), 256, 0, st>>>(l->Y, yb, l->pr.seed);
      GALORE_LAUNCH_CHECK();
      if (l->pr.warm_iters > 0) {
        // Warm start (the subspace of consecutive gradients changes slowly, Sec. 4.1): the stored
        // projector spans most of what is wanted already, the random columns carry the oversampling.
        l->warm_check = true;
        if (l->pr.p_dtype == GALORE_BF16)
          place_previous_kernel<__nv_bfloat16><<<grid_for(d * r), 256, 0, st>>>(l->Y, (const __nv_bfloat16*)l->pr.P, d, r, b);
        else
          place_previous_kernel<float><<<grid_for(d * r), 256, 0, st>>>(l->Y, (const float*)l->pr.P, d, r, b);
        GALORE_LAUNCH_CHECK();
      }
      if (tensor) {
        split_kernel<<<grid_for(yb), 256, 0, st>>>(l->Y, l->w.Yhi, l->w.Ylo, yb);
        GALORE_LAUNCH_CHECK();
      }
    }
    if (tensor) {
      GALORE_TRY(orth_tensor(c, all));
    } else {
      GALORE_TRY((orthonormalise<float, float>(c, all, [](Lane* l) { return l->Y; }, [](Lane* l) { return l->Yn; })));
      for (Lane* l : all) std::swap(l->Y, l->Yn);
    }

    // ---- first steps, then a cheap look at the spectrum ------------------------------------------
    // After a step from an orthonormal Y, ||z_i||^2 (Z = A^T Y) are the Rayleigh quotients of the
    // block's columns.  Sorted, they stand in for the Ritz values: enough to size the iteration
    // (their spread is narrower than the spectrum's, which errs towards more steps) and to decide
    // how many steps may be chained before the block has to be orthonormalised again.
    // A warm-started lane runs its given number of steps first.  If the look says that a cold start
    // would need no more than twice that, the lane goes to Rayleigh-Ritz and is judged by its residual;
    // otherwise (no gap behind the block: the gradient is dominated by noise) it carries on as a cold
    // one, which costs it nothing but keeps what its start already spans.
    for (Lane* l : all)
      l->q_target = l->warm_check ? std::min(l->pr.max_iters, l->pr.warm_iters)
                                  : std::min(l->pr.max_iters, std::max(1, l->pr.first_iters));
    GALORE_TRY(run_steps(all));
    if (b > r) {
      std::vector<Lane*> sized;
      for (Lane* l : all)
        if (l->q_done < l->pr.max_iters) sized.push_back(l);
      for (Lane* l : sized) {
        double* slices = (double*)l->w.Y64;                      // kColSlices x b doubles, Y64 is idle here
        const float* z0 = (const float*)l->w.Zu;
        const float* z1 = tensor ? z0 + L * b : nullptr;
        colsumsq_partial_kernel<<<dim3((unsigned)ceil_div(b, 128), kColSlices), 128, 0, st>>>(z0, z1, L, b, slices);
        GALORE_LAUNCH_CHECK();
        colsumsq_final_kernel<<<(unsigned)ceil_div(b, 128), 128, 0, st>>>(slices, b, l->w.lam);
        GALORE_LAUNCH_CHECK();
        rank_desc_kernel<<<(unsigned)ceil_div(b, 128), 128, 0, st>>>(l->w.lam, b, l->w.theta, l->w.order);
        GALORE_LAUNCH_CHECK();
      }
      if (!sized.empty()) GALORE_TRY(read_theta(sized));
      for (Lane* l : sized) {
        const std::vector<double>& theta = l->theta;
        const double ratio = theta[r - 1] > 0.0 ? theta[b - 1] / theta[r - 1] : 1.0;
        const int need = (ratio > 0.0 && ratio < 1.0) ? (int)ceil(log(l->pr.tol) / log(ratio)) + 1
                                                      : (ratio >= 1.0 ? l->pr.max_iters : l->q_done);
        if (l->warm_check && need > 2 * l->q_done) l->warm_check = false;
        if (!l->warm_check) l->q_target = std::min(l->pr.max_iters, std::max(need, l->q_done));
        if (tensor && !l->warm_check && need - l->q_done > kChebyshevFrom && ratio > 0.25 && ratio < 1.0) {
          // A slowly converging block (no gap behind it): the remaining steps come in pairs that apply
          // T_2 of the operator mapped so that [0, theta_b] falls on [-1, 1].  What lies in the interval stays
          // bounded by 1 while theta_r grows by T_2(2 theta_r / theta_b - 1) per pair, against
          // (theta_r / theta_b)^2 of two plain steps.  The look's theta_b is on the high side, which
          // widens the interval: slower than it could be, never wrong.
          const double beta = theta[b - 1];
          const double gain = cheb_t2(2.0 * theta[r - 1] / beta - 1.0), spread = cheb_t2(2.0 * theta[0] / beta - 1.0);
          if (gain > 1.0 && spread <= kChebyshevSpread) {
            const double left = pow(ratio, (double)l->q_done);            // what the plain steps have achieved
            const int pairs = std::max(1, (int)ceil(log(left / l->pr.tol) / log(gain)) + 1);
            l->cheb = true;
            l->segs.push_back(ChebSegment{0.5 * beta, 0});
            l->q_target = std::min(l->q_done + 2 * pairs, l->q_done + (l->pr.max_iters - l->q_done) / 2 * 2);
          }
        }
        if (l->cheb) {
          l->orth_every = 2;           // the filter's own growth of the block's condition number was checked above
        } else if (tensor && theta[b - 1] > 0.0) {
          // chained steps multiply the block's condition number by theta_1/theta_b each; the bf16 pair
          // carries 16 bits and the Gram matrix squares the product, so keep it below about 100
          const double spread = theta[0] / theta[b - 1];
          l->orth_every = spread > 1.0 ? (int)floor(log(100.0) / log(spread)) : 8;
          l->orth_every = std::max(1, std::min(l->orth_every, 8));
        }
      }
    }
  }

  // P64 = Y64 S[:, top r] from the last Rayleigh-Ritz pass of the given lanes
  const int64_t pc = d * r;
  auto make_p64 = [&](const std::vector<Lane*>& lanes) -> galore_status_t {
    if (lanes.empty()) return GALORE_OK;
    for (Lane* l : lanes) {
      const RefreshBuffers& w = l->w;
      l->p64_current = true;
      if (l->with_vt)
        gather_rows_kernel<<<r, 256, 0, st>>>(w.Vt, w.order, b, w.Vsel);
      else
        gather_rows_scaled_kernel<<<r, 256, 0, st>>>(w.H, w.lam, w.order, b, w.Vsel);
      GALORE_LAUNCH_CHECK();
    }
    EpiStore<double, double> epi{c.w0.P64, r, 0, 1.0, 0.0};
    const SlotList sl = slots_of(c, lanes);
    return launch_gemm_dmma<double, double>((int)d, r, b, c.w0.Y64, b, 1, c.w0.Vsel, 1, b, epi, st, 1, 0, 0, &sl);
  };
  // res_abs = || A A^T P - P Theta ||_F of the given lanes (after make_p64; synchronises the stream).
  // On the tensor path A^T P = Z S is formed from the products already at hand and A (A^T P) runs on
  // the tensor cores in bf16 pairs.  Leaves the iteration's block Y untouched.
  auto residuals = [&](const std::vector<Lane*>& lanes) -> galore_status_t {
    if (lanes.empty()) return GALORE_OK;
    const bool tensor_residual = tensor && (r % 8) == 0;
    for (Lane* l : lanes) {
      const RefreshBuffers& w = l->w;
      const TG* G = (const TG*)l->pr.G;
      const int64_t sAi = c.left ? l->pr.ldg : 1, sAl = c.left ? 1 : l->pr.ldg;
      if (tensor_residual) {
        EpiSplitPair e1{w.Zhi, w.Zlo, r};
        GALORE_TRY((launch_gemm_dmma<double, double>((int)L, r, b, (const double*)w.Zu, b, 1, w.Vsel, 1, b, e1, st)));
        const int a_mn = c.left ? 0 : 1;
        const int s1 = (l->tr.master + 1) % 3, s2 = (l->tr.master + 2) % 3;
        tensor_group_reset(c.tg);
        GALORE_TRY(tensor_group_add_gemm(c.tg, l->pr.G, l->pr.ldg, a_mn, w.Zhi, r, 1, (int)d, r, (int)L, l->tr.F[s1], r, l->status));
        GALORE_TRY(tensor_group_add_gemm(c.tg, l->pr.G, l->pr.ldg, a_mn, w.Zlo, r, 1, (int)d, r, (int)L, l->tr.F[s2], r, l->status));
        GALORE_TRY(tensor_group_launch_project(c.tg, st));
        GALORE_CUDA_TRY(cudaMemsetAsync(w.scal, 0, 32, st));
        residual_pair_kernel<<<grid_for(d * r), 256, 0, st>>>(l->tr.F[s1], l->tr.F[s2], w.P64, w.theta, d, r, w.scal);
        GALORE_LAUNCH_CHECK();
      } else {
        double* T1 = (double*)w.Zu;   // L x r
        double* T2 = w.Y64;           // d x r (Y64 is no longer needed once P64 exists)
        EpiStore<double, double> e1{T1, r, 0, 1.0, 0.0};
        GALORE_TRY((launch_gemm_dmma<TG, double>((int)L, r, (int)d, G, sAl, sAi, w.P64, r, 1, e1, st)));
        EpiStore<double, double> e2{T2, r, 0, 1.0, 0.0};
        GALORE_TRY((launch_gemm_dmma<TG, double>((int)d, r, (int)L, G, sAi, sAl, T1, r, 1, e2, st)));
        GALORE_CUDA_TRY(cudaMemsetAsync(w.scal, 0, 32, st));
        residual_kernel<<<grid_for(pc), 256, 0, st>>>(T2, w.P64, w.theta, d, r, w.scal);
        GALORE_LAUNCH_CHECK();
      }
    }
    std::vector<double> sc(2 * lanes.size(), 0.0);
    for (size_t i = 0; i < lanes.size(); ++i)
      GALORE_CUDA_TRY(cudaMemcpyAsync(&sc[2 * i], lanes[i]->w.scal, 2 * sizeof(double), cudaMemcpyDeviceToHost, st));
    GALORE_CUDA_TRY(cudaStreamSynchronize(st));
    for (size_t i = 0; i < lanes.size(); ++i) lanes[i]->res_abs = sqrt(sc[2 * i + 1]);
    return GALORE_OK;
  };

  std::vector<Lane*> live = all;            // lanes that still iterate
  while (!live.empty()) {
    // ---- power steps: every lane up to its own target, on its own orthonormalisation schedule ----
    {
      NvtxRange range("galore.refresh.steps");
      GALORE_TRY(run_steps(live));
    }
    NvtxRange range("galore.refresh.rayleigh_ritz");
    for (Lane* l : live) {
      l->p64_current = false;
      l->info.ritz_passes += 1;
    }
    // ---- Rayleigh-Ritz in fp64 --------------------------------------------------
    const clk::time_point t_rr = now_synced();
    ms_power = ms_between(t_begin, t_rr) - ms_ritz - ms_jacobi;
    if (full_space) {
      for (Lane* l : live) {
        set_identity_kernel<<<grid_for(yb), 256, 0, st>>>(l->w.Y64, (int)d);
        GALORE_LAUNCH_CHECK();
      }
    } else {
      // Y left the last power step orthonormal to working precision (1e-7 on the FMA path, about 1e-4 from the
      // bf16 pairs); one CholeskyQR pass in fp64 from there is orthonormal to double rounding
      GALORE_TRY((orthonormalise<float, double>(c, live, [](Lane* l) { return l->Y; }, [](Lane* l) { return l->w.Y64; })));
    }
    for (Lane* l : live) {   // Z = A^T Y   (L x b), fp64
      const TG* G = (const TG*)l->pr.G;
      const int64_t sAi = c.left ? l->pr.ldg : 1, sAl = c.left ? 1 : l->pr.ldg;
      EpiStore<double, double> epi{(double*)l->w.Zu, b, 0, 1.0, 0.0};
      GALORE_TRY((launch_gemm_dmma<TG, double>((int)L, b, (int)d, G, sAl, sAi, l->w.Y64, b, 1, epi, st)));
    }
    const clk::time_point t_jac = now_synced();
    ms_ritz += ms_between(t_rr, t_jac);
    // Eigenvectors are read off the rotated rows Theta V^T; only when wanted eigenvalues are tiny
    // against the largest (a gradient of rank below r) are the rotations accumulated separately.
    std::vector<Lane*> solving = live;
    while (!solving.empty()) {
      GALORE_TRY((gram<double>(c, solving, [](Lane* l) { return (double*)l->w.Zu; }, L, c.w0.H)));     // H = Z^T Z
      std::vector<Lane*> plain, with_vt;
      for (Lane* l : solving) (l->with_vt ? with_vt : plain).push_back(l);
      for (Lane* l : with_vt) {
        set_identity_kernel<<<grid_for((int64_t)b * b), 256, 0, st>>>(l->w.Vt, b);
        GALORE_LAUNCH_CHECK();
      }
      for (int pass = 0; pass < 2; ++pass) {
        const std::vector<Lane*>& set = pass == 0 ? plain : with_vt;
        if (set.empty()) continue;
        const SlotList sl = slots_of(c, set);
        int sweeps[kMaxSlots] = {};
        GALORE_TRY(jacobi_eigh(c.w0.H, pass == 0 ? nullptr : c.w0.Vt, b, c.w0.jac, c.w0.counter, 1e-11, 40, sweeps, st, &sl));
        for (size_t i = 0; i < set.size(); ++i) set[i]->info.jacobi_sweeps = sweeps[i];
      }
      for (Lane* l : solving) {
        row_norm_kernel<<<b, 256, 0, st>>>(l->w.H, b, l->w.lam);
        GALORE_LAUNCH_CHECK();
        rank_desc_kernel<<<(unsigned)ceil_div(b, 128), 128, 0, st>>>(l->w.lam, b, l->w.theta, l->w.order);
        GALORE_LAUNCH_CHECK();
      }
      GALORE_TRY(read_theta(solving));
      std::vector<Lane*> again;
      for (Lane* l : solving)
        if (!l->with_vt && !(l->theta[r - 1] > 1e-8 * l->theta[0])) {
          l->with_vt = true;
          again.push_back(l);
        }
      solving = again;
    }
    ms_jacobi += ms_between(t_jac, now_synced());

    std::vector<Lane*> more;
    if (!full_space) {
      // A warm-started lane is judged by what it reached, not by a prediction from a random start:
      // the residual of its Ritz pairs over the gap behind the r-th Ritz value bounds the sine of the
      // largest angle to the exact invariant subspace (Davis-Kahan, with Frobenius for spectral norm:
      // on the safe side).  If that is not within the tolerance the lane goes on like a cold one, its
      // remaining steps sized from the bound instead of from 1.
      std::vector<Lane*> judged;
      for (Lane* l : live)
        if (l->warm_check) judged.push_back(l);
      if (!judged.empty()) {
        GALORE_TRY(make_p64(judged));
        GALORE_TRY(residuals(judged));
      }
      for (Lane* l : judged) {
        l->warm_check = false;
        const double th_r = l->theta[r - 1], th_b = l->theta[b - 1];
        const double gap = b > r ? th_r - l->theta[r] : 0.0;
        const double bound = gap > 0.0 ? l->res_abs / gap : 1.0;
        l->predicted = std::min(1.0, bound);
        // a prediction from a random start is held to the tolerance itself, which leaves a margin of ten to
        // the 1e-3 rad the projector has to meet; a bound on what was reached needs no such margin
        l->converged = bound <= 10.0 * l->pr.tol;
        const double ratio = (b > r && th_r > 0.0) ? th_b / th_r : 1.0;
        if (!l->converged && l->q_done < l->pr.max_iters && ratio < 1.0 && ratio > 0.0) {
          const int need = (int)ceil(log(l->pr.tol / l->predicted) / log(ratio)) + 1;
          l->q_target = std::min(l->pr.max_iters, l->q_done + std::max(1, need));
          l->warm_from = l->q_done;
          l->warm_bound = l->predicted;
          more.push_back(l);
        }
      }
      for (Lane* l : live) {
        if (std::find(judged.begin(), judged.end(), l) != judged.end()) continue;
        const double th_r = l->theta[r - 1], th_b = l->theta[b - 1];
        const double ratio = (b > r && th_r > 0.0) ? th_b / th_r : 1.0;
        if (l->cheb) {
          // plain steps as below; every Chebyshev pair divides the error by T_2 at theta_r over the largest
          // value the filter takes on what is to be damped (1 inside its interval, T_2 at theta_b beyond it)
          double log_err = (ratio < 1.0 && ratio > 0.0) ? l->q_plain * log(ratio) : 0.0;
          for (const ChebSegment& sg : l->segs) {
            const double num = std::max(1.0, fabs(cheb_t2(th_b / sg.c - 1.0))), den = cheb_t2(th_r / sg.c - 1.0);
            if (den > num) log_err += sg.pairs * log(num / den);
          }
          l->predicted = ratio < 1.0 ? std::min(1.0, exp(log_err)) : 1.0;
          l->converged = l->predicted <= l->pr.tol;
          if (!l->converged && l->q_done + 1 < l->pr.max_iters && ratio < 1.0 && ratio > 0.0) {
            const double c2 = 0.5 * 1.02 * th_b;                   // the interval now ends just above the b-th Ritz value
            const double gain = cheb_t2(th_r / c2 - 1.0);
            const int pairs = gain > 1.0 ? std::max(1, (int)ceil(log(l->predicted / l->pr.tol) / log(gain)) + 1) : 1;
            l->segs.push_back(ChebSegment{c2, 0});
            l->q_target = std::min(l->q_done + 2 * pairs, l->q_done + (l->pr.max_iters - l->q_done) / 2 * 2);
            more.push_back(l);
          }
          continue;
        }
        // from a random start the error begins at 1; after a warm start at the bound found above
        l->predicted = (ratio < 1.0) ? l->warm_bound * pow(ratio, (double)(l->q_done - l->warm_from)) : 1.0;
        l->converged = l->predicted <= l->pr.tol;
        if (!l->converged && l->q_done < l->pr.max_iters && ratio < 1.0 && ratio > 0.0) {
          const int need = (int)ceil(log(l->pr.tol) / log(ratio)) + 2;
          l->q_target = std::min(l->pr.max_iters, std::max(need, l->q_done + 1));
          more.push_back(l);                                       // more power steps, then Rayleigh-Ritz again
        }
      }
    }
    live = more;
  }

  // ---- P = Y S[:, top r], rounded to the stored dtype ------------------------------------------
  // (a lane judged by its residual and found converged has its P64 already, and the residual used Y64 as scratch)
  std::vector<Lane*> unmade;
  for (Lane* l : all)
    if (!l->p64_current) unmade.push_back(l);
  GALORE_TRY(make_p64(unmade));
  for (Lane* l : all) {
    if (l->pr.p_dtype == GALORE_BF16)
      convert_kernel<double, __nv_bfloat16><<<grid_for(pc), 256, 0, st>>>(l->w.P64, (__nv_bfloat16*)l->pr.P, pc);
    else
      convert_kernel<double, float><<<grid_for(pc), 256, 0, st>>>(l->w.P64, (float*)l->pr.P, pc);
    GALORE_LAUNCH_CHECK();
    merge_flags_kernel<<<1, 1, 0, st>>>(l->status, l->w.flags);
    GALORE_LAUNCH_CHECK();
  }
  // the a-posteriori residual of the kept Ritz pairs is a diagnostic: only when the record is wanted
  if (infos) {
    GALORE_TRY(residuals(all));
    for (Lane* l : all) l->info.residual = l->theta[0] > 0.0 ? l->res_abs / (l->theta[0] * sqrt((double)r)) : 0.0;
  }
  GALORE_CUDA_TRY(cudaStreamSynchronize(st));      // the refresh is complete when the call returns
  const double ms_total = ms_between(t_begin, clk::now());
  galore_status_t worst = GALORE_OK;
  for (int i = 0; i < count; ++i) {
    Lane& l = store[i];
    // times of the group as a whole, divided evenly among its layers
    l.info.ms_total = ms_total / count;
    l.info.ms_power = ms_power / count;
    l.info.ms_jacobi = ms_jacobi / count;
    l.info.ms_ritz = (ms_total - ms_power - ms_jacobi) / count;
    l.info.iterations = l.q_done;
    l.info.converged = l.converged ? 1 : 0;
    l.info.predicted_error = l.predicted;
    l.info.sigma_1 = sqrt(l.theta[0]);
    l.info.sigma_r = sqrt(l.theta[r - 1]);
    l.info.sigma_next = (b > r) ? sqrt(l.theta[r]) : 0.0;
    if (infos) infos[i] = l.info;
    if (!l.converged) worst = GALORE_WARN_NOT_CONVERGED;
  }
  return worst;
}

galore_status_t refresh_projector_group(const RefreshProblem* prs, int count, void* workspace, size_t slot_bytes,
                                        int32_t* const* status, galore_refresh_info_t* infos, cudaStream_t st) {
  if (!prs || count < 1) return GALORE_ERR_INVALID_ARG;
  for (int i = 1; i < count; ++i) {
    const RefreshProblem &a = prs[0], &b = prs[i];
    if (a.m != b.m || a.n != b.n || a.left != b.left || a.rank != b.rank || a.block != b.block || a.g_dtype != b.g_dtype ||
        a.use_tensor != b.use_tensor || a.max_iters != b.max_iters || a.first_iters != b.first_iters)
      return GALORE_ERR_INVALID_ARG;
  }
  if (prs[0].g_dtype == GALORE_BF16) return refresh_group<__nv_bfloat16>(prs, count, workspace, slot_bytes, status, infos, st);
  return refresh_group<float>(prs, count, workspace, slot_bytes, status, infos, st);
}

galore_status_t refresh_projector(const RefreshProblem& pr, void* workspace, int32_t* status,
                                  galore_refresh_info_t* info, cudaStream_t st) {
  const int64_t d = pr.left ? pr.m : pr.n, L = pr.left ? pr.n : pr.m;
  return refresh_projector_group(&pr, 1, workspace, refresh_workspace_bytes(d, L, pr.rank, pr.block), &status, info, st);
}

}  // namespace galore
