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

template <typename T>
__global__ void __launch_bounds__(256) potf2_inv_kernel(T* __restrict__ C, int ld, int nb, T* __restrict__ Linv,
                                                        int32_t* __restrict__ status) {
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
__global__ void place_diag_inverse_kernel(const S* __restrict__ slabs, int b, S* __restrict__ T) {
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
  __device__ __forceinline__ void operator()(int i, int j, double acc, int) const {
    split_bf16((float)acc, hi[(int64_t)i * ld + j], lo[(int64_t)i * ld + j]);
  }
};

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
  w.counter = (int*)p; carve(p, 256);
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
// building blocks
// ---------------------------------------------------------------------------

// C (b x b, fp64) = Y^T Y
template <typename TY>
static galore_status_t gram(const TY* Y, int64_t d, int b, double* C, cudaStream_t st) {
  EpiStore<double, double> epi{C, b, 0, 1.0, 0.0};
  return launch_gemm_dmma<TY, TY>(b, b, (int)d, Y, 1, b, Y, b, 1, epi, st);
}

// Blocked Cholesky of the b x b matrix C (lower triangle, in place), then T = L^-1 (b x b, lower,
// zero above the diagonal).
//   factor : per 64-wide panel the diagonal block (with its inverse, kept in w.slabs), the panel
//            below it and the trailing update;
//   invert : the inverses of the diagonal blocks are merged pairwise, level by level,
//            [T11 0; T21 T22] with T21 = -T22 L21 T11, every level two batched products.
// scratch: b*b/4 doubles.
// (S = double: products on the fp64 MMA unit; S = float, used between the tensor-core power steps
// whose Gram matrices carry about 16 bits anyway: FMA products and a ten times shorter pivot chain.)
template <typename TA, typename TB, typename S, class Epi>
static galore_status_t gemm_scalar(int M, int N, int K, const TA* A, int64_t sAi, int64_t sAk, const TB* B, int64_t sBk,
                                   int64_t sBj, Epi epi, cudaStream_t st, int batch = 1, int64_t bA = 0, int64_t bB = 0) {
  if constexpr (std::is_same<S, double>::value)
    return launch_gemm_dmma<TA, TB>(M, N, K, A, sAi, sAk, B, sBk, sBj, epi, st, batch, bA, bB);
  else
    return launch_gemm_simt<TA, TB, float>(M, N, K, A, sAi, sAk, B, sBk, sBj, 1, epi, st, batch, bA, bB);
}

template <typename S>
static galore_status_t cholesky_inverse(S* C, int b, S* T, S* scratch, const RefreshBuffers& w, int32_t* status,
                                        cudaStream_t st) {
  const int nblk = (int)ceil_div(b, 64);
  S* slabs = (S*)w.slabs;
  for (int p = 0; p < nblk; ++p) {
    const int j0 = p * 64, nb = std::min(64, b - j0), j1 = j0 + nb;
    S* slab = slabs + (int64_t)p * 4096;
    potf2_inv_kernel<S><<<1, 256, 0, st>>>(C + (int64_t)j0 * b + j0, b, nb, slab, status);
    GALORE_LAUNCH_CHECK();
    if (j1 < b) {
      const int rem = b - j1;
      S* panel = C + (int64_t)j1 * b + j0;
      // L[rest, J] = C[rest, J] Linv^T   (in place: one CTA column covers all nb columns)
      EpiStore<S, S> epi{panel, b, 0, S(1), S(0)};
      GALORE_TRY((gemm_scalar<S, S, S>(rem, nb, nb, panel, b, 1, slab, 1, 64, epi, st)));
      // C[rest, rest] -= L[rest, J] L[rest, J]^T
      EpiStore<S, S> upd{C + (int64_t)j1 * b + j1, b, 0, S(-1), S(1)};
      GALORE_TRY((gemm_scalar<S, S, S>(rem, rem, nb, panel, b, 1, panel, 1, b, upd, st)));
    }
  }
  GALORE_CUDA_TRY(cudaMemsetAsync(T, 0, sizeof(S) * b * b, st));
  place_diag_inverse_kernel<S><<<nblk, 256, 0, st>>>(slabs, b, T);
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
      GALORE_TRY((gemm_scalar<S, S, S>(s2, (int)s, (int)s, L21, b, 1, T11, b, 1, ew, st, count, step, step)));
      // T21 = -T22 W
      EpiStore<S, S> et{T21, b, step, S(-1), S(0)};
      GALORE_TRY((gemm_scalar<S, S, S>(s2, (int)s, s2, T22, b, 1, scratch, s, 1, et, st, count, step, s * s)));
    }
  }
  return GALORE_OK;
}

// out = Y L^-T with L L^T = Y^T Y (CholeskyQR); out must not alias Y.  Uses w.C, w.Vt, w.H.
template <typename TY, typename TO>
static galore_status_t orthonormalise(const TY* Y, TO* out, int64_t d, int b, const RefreshBuffers& w, int32_t* status,
                                      cudaStream_t st) {
  GALORE_TRY(gram(Y, d, b, w.C, st));
  GALORE_TRY(cholesky_inverse<double>(w.C, b, w.Vt, w.H, w, status, st));
  EpiStore<TO, double> epi{out, b, 0, 1.0, 0.0};
  return launch_gemm_dmma<TY, double>((int)d, b, b, Y, b, 1, w.Vt, 1, b, epi, st);
}

// ---- power step on the tensor cores -------------------------------------------------------------
// The block Y lives as an fp32 master (one of three d x b buffers) plus its bf16 hi/lo pair.  Every
// product below is a tcgen05 GEMM on bf16 operands with fp32 output; a product with a hi/lo operand
// is two (or three) problems of one grouped launch whose outputs are added afterwards.

struct TensorRefresh {
  TensorGroup* tg;
  float* F[3];          // fp32 d x b buffers; F[master] holds Y
  int master;
  int32_t* status;
};

// Y <- Y L^-T with L L^T = Y^T Y: CholeskyQR whose two big products run on the tensor cores.
// In: hi/lo pair of Y valid (the fp32 master itself is not read).  Out: master and pair updated.
static galore_status_t orth_tensor(TensorRefresh& t, const RefreshBuffers& w, int64_t d, int b, cudaStream_t st) {
  const int64_t bb = (int64_t)b * b, yb = d * b;
  float* g0 = (float*)w.H;
  float* g1 = g0 + bb;
  float* g2 = (float*)w.Y64;
  tensor_group_reset(t.tg);   // Gram = (hi + lo)^T (hi + lo) without the lo^T lo term
  GALORE_TRY(tensor_group_add_gemm(t.tg, w.Yhi, b, 1, w.Yhi, b, 1, b, b, (int)d, g0, b, t.status));
  GALORE_TRY(tensor_group_add_gemm(t.tg, w.Yhi, b, 1, w.Ylo, b, 1, b, b, (int)d, g1, b, t.status));
  GALORE_TRY(tensor_group_add_gemm(t.tg, w.Ylo, b, 1, w.Yhi, b, 1, b, b, (int)d, g2, b, t.status));
  GALORE_TRY(tensor_group_launch_project(t.tg, st));
  gram_sum_kernel<<<grid_for(bb), 256, 0, st>>>(g0, g1, g2, (float*)w.C, bb);
  GALORE_LAUNCH_CHECK();
  // T = L^-1, split into a bf16 pair; as the second operand of Y L^-T it is read K-contiguous
  GALORE_TRY(cholesky_inverse<float>((float*)w.C, b, (float*)w.Vt, (float*)w.H, w, t.status, st));
  split_kernel<<<grid_for(bb), 256, 0, st>>>((const float*)w.Vt, w.Thi, w.Tlo, bb);
  GALORE_LAUNCH_CHECK();
  const int m = t.master, s1 = (m + 1) % 3, s2 = (m + 2) % 3;
  tensor_group_reset(t.tg);   // Y T = hi Thi + hi Tlo + lo Thi
  GALORE_TRY(tensor_group_add_gemm(t.tg, w.Yhi, b, 0, w.Thi, b, 0, (int)d, b, b, t.F[m], b, t.status));
  GALORE_TRY(tensor_group_add_gemm(t.tg, w.Yhi, b, 0, w.Tlo, b, 0, (int)d, b, b, t.F[s1], b, t.status));
  GALORE_TRY(tensor_group_add_gemm(t.tg, w.Ylo, b, 0, w.Thi, b, 0, (int)d, b, b, t.F[s2], b, t.status));
  GALORE_TRY(tensor_group_launch_project(t.tg, st));
  sum_split_kernel<<<grid_for(yb), 256, 0, st>>>(t.F[m], t.F[s1], t.F[s2], t.F[m], w.Yhi, w.Ylo, yb);
  GALORE_LAUNCH_CHECK();
  return GALORE_OK;
}

// Z = A^T Y ; Y' = A Z + delta Y ; Y = orth(Y')
static galore_status_t power_step_tensor(TensorRefresh& t, const RefreshProblem& pr, const RefreshBuffers& w, int64_t d,
                                         int64_t L, int b, bool orth, cudaStream_t st) {
  const int64_t zb = L * b, yb = d * b;
  float* z0 = (float*)w.Zu;
  float* z1 = z0 + zb;
  const int at_mn = pr.left ? 1 : 0;   // A^T as the first operand: G^T (left) is M-contiguous in G, G (right) is K-contiguous
  const int a_mn = pr.left ? 0 : 1;    // A as the first operand
  tensor_group_reset(t.tg);
  GALORE_TRY(tensor_group_add_gemm(t.tg, pr.G, pr.ldg, at_mn, w.Yhi, b, 1, (int)L, b, (int)d, z0, b, t.status));
  GALORE_TRY(tensor_group_add_gemm(t.tg, pr.G, pr.ldg, at_mn, w.Ylo, b, 1, (int)L, b, (int)d, z1, b, t.status));
  GALORE_TRY(tensor_group_launch_project(t.tg, st));
  sum_split_kernel<<<grid_for(zb), 256, 0, st>>>(z0, z1, nullptr, nullptr, w.Zhi, w.Zlo, zb);
  GALORE_LAUNCH_CHECK();
  const int m = t.master, s1 = (m + 1) % 3, s2 = (m + 2) % 3;
  tensor_group_reset(t.tg);
  GALORE_TRY(tensor_group_add_gemm(t.tg, pr.G, pr.ldg, a_mn, w.Zhi, b, 1, (int)d, b, (int)L, t.F[s1], b, t.status));
  GALORE_TRY(tensor_group_add_gemm(t.tg, pr.G, pr.ldg, a_mn, w.Zlo, b, 1, (int)d, b, (int)L, t.F[s2], b, t.status));
  GALORE_TRY(tensor_group_launch_project(t.tg, st));
  add_sumsq_kernel<<<kSumsqBlocks, 256, 0, st>>>(t.F[s1], t.F[s2], yb, w.part);
  GALORE_LAUNCH_CHECK();
  shift_split_kernel<<<grid_for(yb), 256, 0, st>>>(t.F[s1], t.F[m], yb, b, w.part, w.Yhi, w.Ylo);
  GALORE_LAUNCH_CHECK();
  t.master = s1;
  return orth ? orth_tensor(t, w, d, b, st) : GALORE_OK;
}

template <typename TG>
static galore_status_t refresh_typed(const RefreshProblem& pr, void* workspace, int32_t* status,
                                     galore_refresh_info_t* info, cudaStream_t st) {
  const TG* G = (const TG*)pr.G;
  const int64_t d = pr.left ? pr.m : pr.n;
  const int64_t L = pr.left ? pr.n : pr.m;
  const int64_t sAi = pr.left ? pr.ldg : 1;    // A(i, l) = G[i*sAi + l*sAl]
  const int64_t sAl = pr.left ? 1 : pr.ldg;
  const int r = pr.rank, b = pr.block;
  RefreshBuffers w = layout(workspace, d, L, r, b);
  galore_refresh_info_t local = {};
  local.block = b;
  // phase clock: host time at points where the stream is synchronised anyway
  using clk = std::chrono::steady_clock;
  auto now_synced = [&]() {
    cudaStreamSynchronize(st);
    return clk::now();
  };
  auto ms_between = [](clk::time_point a, clk::time_point b2) { return std::chrono::duration<double, std::milli>(b2 - a).count(); };
  const clk::time_point t_begin = now_synced();

  float* Y = w.Ya;
  float* Yn = w.Yb;
  const int64_t yb = d * b;
  int q_done = 0;
  std::vector<double> theta(b);
  const bool full_space = (b == d);

  // tensor cores carry the power steps when the gradient is bf16 and everything is TMA-addressable
  const bool tensor = pr.use_tensor && !full_space && sizeof(TG) == 2 && (b % 8) == 0 && (pr.ldg % 8) == 0 &&
                      (((uintptr_t)pr.G) & 15) == 0;
  TensorRefresh tr = {};
  struct GroupGuard {
    TensorGroup* g;
    ~GroupGuard() { tensor_group_free(g); }
  } guard{nullptr};
  if (!full_space) {
    fill_normal_kernel<<<grid_for(yb), 256, 0, st>>>(Y, yb, pr.seed);
    GALORE_LAUNCH_CHECK();
    if (tensor) {
      guard.g = tr.tg = tensor_group_new();
      if (!tr.tg) return GALORE_ERR_INVALID_ARG;
      tr.F[0] = w.Ya; tr.F[1] = w.Yb; tr.F[2] = w.Yc;
      tr.master = 0;
      tr.status = status;
      split_kernel<<<grid_for(yb), 256, 0, st>>>(Y, w.Yhi, w.Ylo, yb);
      GALORE_LAUNCH_CHECK();
      GALORE_TRY(orth_tensor(tr, w, d, b, st));
    } else {
      GALORE_TRY(orthonormalise(Y, Yn, d, b, w, status, st));
      std::swap(Y, Yn);
    }
  }
  double predicted = 0.0;
  bool converged = full_space;

  // one power step, Z = A^T Y ; Y' = A Z + delta Y ; optionally Y = orth(Y')
  auto one_step = [&](bool orth) -> galore_status_t {
    if (tensor) {
      GALORE_TRY(power_step_tensor(tr, pr, w, d, L, b, orth, st));
      Y = tr.F[tr.master];
      return GALORE_OK;
    }
    float* Z = (float*)w.Zu;
    {  // Z = A^T Y   (L x b)
      EpiStore<float, float> epi{Z, b, 0, 1.f, 0.f};
      GALORE_TRY((launch_gemm_simt<TG, float, float>((int)L, b, (int)d, G, sAl, sAi, Y, b, 1, 1, epi, st)));
    }
    {  // Y' = A Z     (d x b)
      EpiStore<float, float> epi{Yn, b, 0, 1.f, 0.f};
      GALORE_TRY((launch_gemm_simt<TG, float, float>((int)d, b, (int)L, G, sAi, sAl, Z, b, 1, 1, epi, st)));
    }
    sumsq_kernel<<<kSumsqBlocks, 256, 0, st>>>(Yn, yb, w.part);
    GALORE_LAUNCH_CHECK();
    shift_kernel<<<grid_for(yb), 256, 0, st>>>(Yn, Y, yb, b, w.part);
    GALORE_LAUNCH_CHECK();
    return orthonormalise(Yn, Y, d, b, w, status, st);    // the old block is no longer needed: reuse it for the result
  };

  // ---- first steps, then a cheap look at the spectrum ------------------------------------------
  // After a step from an orthonormal Y, ||z_i||^2 (Z = A^T Y) are the Rayleigh quotients of the
  // block's columns.  Sorted, they stand in for the Ritz values: enough to size the iteration
  // (their spread is narrower than the spectrum's, which errs towards more steps) and to decide
  // how many steps may be chained before the block has to be orthonormalised again.
  int q_target = 0;
  int orth_every = 1;
  if (!full_space) {
    const int q0 = std::min(pr.max_iters, std::max(1, pr.first_iters));
    for (; q_done < q0; ++q_done) GALORE_TRY(one_step(true));
    q_target = q_done;
    if (b > r && q_done < pr.max_iters) {
      double* slices = (double*)w.Y64;                      // kColSlices x b doubles, Y64 is idle here
      const float* z0 = (const float*)w.Zu;
      const float* z1 = tensor ? z0 + L * b : nullptr;
      colsumsq_partial_kernel<<<dim3((unsigned)ceil_div(b, 128), kColSlices), 128, 0, st>>>(z0, z1, L, b, slices);
      GALORE_LAUNCH_CHECK();
      colsumsq_final_kernel<<<(unsigned)ceil_div(b, 128), 128, 0, st>>>(slices, b, w.lam);
      GALORE_LAUNCH_CHECK();
      rank_desc_kernel<<<(unsigned)ceil_div(b, 128), 128, 0, st>>>(w.lam, b, w.theta, w.order);
      GALORE_LAUNCH_CHECK();
      GALORE_CUDA_TRY(cudaMemcpyAsync(theta.data(), w.theta, sizeof(double) * b, cudaMemcpyDeviceToHost, st));
      GALORE_CUDA_TRY(cudaStreamSynchronize(st));
      const double ratio = theta[r - 1] > 0.0 ? theta[b - 1] / theta[r - 1] : 1.0;
      if (ratio > 0.0 && ratio < 1.0) {
        const int need = (int)ceil(log(pr.tol) / log(ratio)) + 1;
        q_target = std::min(pr.max_iters, std::max(need, q_done));
      } else if (ratio >= 1.0) {
        q_target = pr.max_iters;
      }
      if (tensor && theta[b - 1] > 0.0) {
        // chained steps multiply the block's condition number by theta_1/theta_b each; the bf16 pair
        // carries 16 bits and the Gram matrix squares the product, so keep it below about 100
        const double spread = theta[0] / theta[b - 1];
        orth_every = spread > 1.0 ? (int)floor(log(100.0) / log(spread)) : 8;
        orth_every = std::max(1, std::min(orth_every, 8));
      }
    }
  }
  bool with_vt = false;

  for (;;) {
    // ---- power steps ---------------------------------------------------------
    for (; q_done < q_target; ++q_done) {
      const bool orth = ((q_target - 1 - q_done) % orth_every) == 0;      // the last step always ends orthonormal
      GALORE_TRY(one_step(orth));
    }
    // ---- Rayleigh-Ritz in fp64 --------------------------------------------------
    const clk::time_point t_rr = now_synced();
    local.ms_power = ms_between(t_begin, t_rr) - local.ms_ritz - local.ms_jacobi;
    if (full_space) {
      set_identity_kernel<<<grid_for(yb), 256, 0, st>>>(w.Y64, (int)d);
      GALORE_LAUNCH_CHECK();
    } else {
      // Y left the last power step orthonormal to working precision (1e-7 on the FMA path, about 1e-4 from the
      // bf16 pairs); one CholeskyQR pass in fp64 from there is orthonormal to double rounding
      GALORE_TRY(orthonormalise(Y, w.Y64, d, b, w, status, st));
    }
    double* Z64 = (double*)w.Zu;
    {  // Z = A^T Y   (L x b), fp64
      EpiStore<double, double> epi{Z64, b, 0, 1.0, 0.0};
      GALORE_TRY((launch_gemm_dmma<TG, double>((int)L, b, (int)d, G, sAl, sAi, w.Y64, b, 1, epi, st)));
    }
    const clk::time_point t_jac = now_synced();
    local.ms_ritz += ms_between(t_rr, t_jac);
    // Eigenvectors are read off the rotated rows Theta V^T; only when wanted eigenvalues are tiny
    // against the largest (a gradient of rank below r) are the rotations accumulated separately.
    for (;;) {
      GALORE_TRY(gram(Z64, L, b, w.H, st));                   // H = Z^T Z
      if (with_vt) {
        set_identity_kernel<<<grid_for((int64_t)b * b), 256, 0, st>>>(w.Vt, b);
        GALORE_LAUNCH_CHECK();
      }
      int sweeps = 0;
      GALORE_TRY(jacobi_eigh(w.H, with_vt ? w.Vt : nullptr, b, w.jac, w.counter, 1e-11, 40, &sweeps, st));
      local.jacobi_sweeps = sweeps;
      row_norm_kernel<<<b, 256, 0, st>>>(w.H, b, w.lam);
      GALORE_LAUNCH_CHECK();
      rank_desc_kernel<<<(unsigned)ceil_div(b, 128), 128, 0, st>>>(w.lam, b, w.theta, w.order);
      GALORE_LAUNCH_CHECK();
      GALORE_CUDA_TRY(cudaMemcpyAsync(theta.data(), w.theta, sizeof(double) * b, cudaMemcpyDeviceToHost, st));
      GALORE_CUDA_TRY(cudaStreamSynchronize(st));
      if (with_vt || theta[r - 1] > 1e-8 * theta[0]) break;
      with_vt = true;
    }
    local.ms_jacobi += ms_between(t_jac, now_synced());

    if (!full_space) {
      const double th_r = theta[r - 1], th_b = theta[b - 1];
      const double ratio = (b > r && th_r > 0.0) ? th_b / th_r : 1.0;
      predicted = (ratio < 1.0) ? pow(ratio, (double)q_done) : 1.0;
      converged = predicted <= pr.tol;
      if (!converged && q_done < pr.max_iters && ratio < 1.0 && ratio > 0.0) {
        int need = (int)ceil(log(pr.tol) / log(ratio)) + 2;
        q_target = std::min(pr.max_iters, std::max(need, q_done + 1));
        continue;                                              // more power steps, then Rayleigh-Ritz again
      }
    }
    break;
  }

  // ---- P = Y S[:, top r] ------------------------------------------------------------
  if (with_vt)
    gather_rows_kernel<<<r, 256, 0, st>>>(w.Vt, w.order, b, w.Vsel);
  else
    gather_rows_scaled_kernel<<<r, 256, 0, st>>>(w.H, w.lam, w.order, b, w.Vsel);
  GALORE_LAUNCH_CHECK();
  {
    EpiStore<double, double> epi{w.P64, r, 0, 1.0, 0.0};
    GALORE_TRY((launch_gemm_dmma<double, double>((int)d, r, b, w.Y64, b, 1, w.Vsel, 1, b, epi, st)));
  }
  const int64_t pc = d * r;
  if (pr.p_dtype == GALORE_BF16)
    convert_kernel<double, __nv_bfloat16><<<grid_for(pc), 256, 0, st>>>(w.P64, (__nv_bfloat16*)pr.P, pc);
  else
    convert_kernel<double, float><<<grid_for(pc), 256, 0, st>>>(w.P64, (float*)pr.P, pc);
  GALORE_LAUNCH_CHECK();

  // ---- a-posteriori residual of the kept Ritz pairs -----------------------------------
  // || A A^T P - P Theta ||.  It is a diagnostic: on the tensor path A^T P = Z S is formed from the
  // products already at hand and A (A^T P) runs on the tensor cores in bf16 pairs.
  const bool tensor_residual = tensor && (r % 8) == 0;
  if (tensor_residual) {
    EpiSplitPair e1{w.Zhi, w.Zlo, r};
    GALORE_TRY((launch_gemm_dmma<double, double>((int)L, r, b, (const double*)w.Zu, b, 1, w.Vsel, 1, b, e1, st)));
    const int a_mn = pr.left ? 0 : 1;
    const int s1 = (tr.master + 1) % 3, s2 = (tr.master + 2) % 3;
    tensor_group_reset(tr.tg);
    GALORE_TRY(tensor_group_add_gemm(tr.tg, pr.G, pr.ldg, a_mn, w.Zhi, r, 1, (int)d, r, (int)L, tr.F[s1], r, status));
    GALORE_TRY(tensor_group_add_gemm(tr.tg, pr.G, pr.ldg, a_mn, w.Zlo, r, 1, (int)d, r, (int)L, tr.F[s2], r, status));
    GALORE_TRY(tensor_group_launch_project(tr.tg, st));
    GALORE_CUDA_TRY(cudaMemsetAsync(w.scal, 0, 32, st));
    residual_pair_kernel<<<grid_for(d * r), 256, 0, st>>>(tr.F[s1], tr.F[s2], w.P64, w.theta, d, r, w.scal);
    GALORE_LAUNCH_CHECK();
  } else {
    double* T1 = (double*)w.Zu;   // L x r
    double* T2 = w.Y64;           // d x r (Y64 is no longer needed)
    EpiStore<double, double> e1{T1, r, 0, 1.0, 0.0};
    GALORE_TRY((launch_gemm_dmma<TG, double>((int)L, r, (int)d, G, sAl, sAi, w.P64, r, 1, e1, st)));
    EpiStore<double, double> e2{T2, r, 0, 1.0, 0.0};
    GALORE_TRY((launch_gemm_dmma<TG, double>((int)d, r, (int)L, G, sAi, sAl, T1, r, 1, e2, st)));
    GALORE_CUDA_TRY(cudaMemsetAsync(w.scal, 0, 32, st));
    residual_kernel<<<grid_for(pc), 256, 0, st>>>(T2, w.P64, w.theta, d, r, w.scal);
    GALORE_LAUNCH_CHECK();
  }
  {
    double sc[2] = {0, 0};
    GALORE_CUDA_TRY(cudaMemcpyAsync(sc, w.scal, sizeof(sc), cudaMemcpyDeviceToHost, st));
    GALORE_CUDA_TRY(cudaStreamSynchronize(st));
    local.residual = theta[0] > 0.0 ? sqrt(sc[1]) / (theta[0] * sqrt((double)r)) : 0.0;
  }
  local.ms_total = ms_between(t_begin, now_synced());
  local.ms_ritz = local.ms_total - local.ms_power - local.ms_jacobi;
  local.iterations = q_done;
  local.converged = converged ? 1 : 0;
  local.predicted_error = predicted;
  local.sigma_1 = sqrt(theta[0]);
  local.sigma_r = sqrt(theta[r - 1]);
  local.sigma_next = (b > r) ? sqrt(theta[r]) : 0.0;
  if (info) *info = local;
  return converged ? GALORE_OK : GALORE_WARN_NOT_CONVERGED;
}

galore_status_t refresh_projector(const RefreshProblem& pr, void* workspace, int32_t* status,
                                  galore_refresh_info_t* info, cudaStream_t st) {
  if (pr.g_dtype == GALORE_BF16) return refresh_typed<__nv_bfloat16>(pr, workspace, status, info, st);
  return refresh_typed<float>(pr, workspace, status, info, st);
}

}  // namespace galore
