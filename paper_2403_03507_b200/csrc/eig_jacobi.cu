// Block one-sided Jacobi for the symmetric eigenproblem of the Rayleigh-Ritz step (Eq. 12-13).
//
// The rows of X (initially H) are made mutually orthogonal by plane rotations, as in the Hestenes
// method; at convergence X = Theta V^T.  Rows are grouped in blocks of 32.  One round pairs the
// blocks by a round-robin schedule; for every pair of blocks
//   1. the 64 x 64 Gram matrix of its rows is formed (fp64 tensor-core MMA, columns split over CTAs),
//   2. one cyclic sweep of rotations is run on that Gram matrix in shared memory, which is exactly
//      the sequence of rotations the 64 rows themselves would receive, accumulated into a 64 x 64
//      orthogonal matrix,
//   3. the accumulated rotation is applied to the 64 rows (again an fp64 MMA product).
// All blocks meet once per sweep; a sweep without any rotation ends the iteration.  Compared with
// rotating two rows per CTA and round, the matrix is read and written twice per block round instead
// of once per row round: 32 times less traffic for the same rotations.
#include "eig_jacobi.cuh"

#include <algorithm>

namespace galore {
namespace {

constexpr int kBlockRows = 32;
constexpr int kPairRows = 64;
constexpr int kGramChunk = 256;   // columns summed by one CTA of the Gram kernel
constexpr int kApplyCols = 128;   // columns transformed by one CTA of the apply kernel
constexpr int kGramLd = 36;       // shared-memory row strides, all = 4 mod 16 doubles: the 8 x 4 operand
constexpr int kRotLd = 68;        // fragments of the fp64 MMA then fall on distinct banks
constexpr int kApplyHalf = 64;    // columns in shared memory at a time
constexpr int kHalfLd = 68;

// D (8 x 8) += A (8 x 4, row) B (4 x 8, col), fp64.  Lane l holds A[l / 4][l % 4], B[l % 4][l / 4]
// and D[l / 4][2 (l % 4) + {0, 1}].
__device__ __forceinline__ void dmma(double (&d)[2], double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};\n"
               : "+d"(d[0]), "+d"(d[1])
               : "d"(a), "d"(b));
}

// Round-robin tournament of n players (n even): in `round`, position k meets position n - 1 - k.
__host__ __device__ __forceinline__ int rr_player(int pos, int round, int n) {
  if (pos == 0) return 0;
  const int m = n - 1;
  int v = (pos - 1 - round) % m;
  if (v < 0) v += m;
  return 1 + v;
}

struct BlockPair {
  int I, J;   // I < J
  __device__ __forceinline__ int row(int l) const { return l < kBlockRows ? I * kBlockRows + l : J * kBlockRows + (l - kBlockRows); }
};
__device__ __forceinline__ BlockPair block_pair(int pair, int round, int nblk) {
  int I = rr_player(pair, round, nblk), J = rr_player(nblk - 1 - pair, round, nblk);
  if (I > J) { const int t = I; I = J; J = t; }
  return BlockPair{I, J};
}

// part[(pair * chunks + chunk)] (64 x 64) = rows(pair)[:, chunk] rows(pair)[:, chunk]^T
__global__ void __launch_bounds__(128) jb_gram_kernel(const double* __restrict__ X, int b, int nblk, int round, int chunks,
                                                      double* __restrict__ part, const SlotList slots) {
  __shared__ __align__(16) double Xs[2][kPairRows][kGramLd];
  const int pair = blockIdx.x, chunk = blockIdx.y;
  {
    const int64_t shift = (int64_t)slots.id[blockIdx.z] * slots.bytes;     // blockIdx.z: workspace slot
    X = slot_ptr(X, shift);
    part = slot_ptr(part, shift);
  }
  const BlockPair bp = block_pair(pair, round, nblk);
  if (bp.I * kBlockRows >= b) return;                 // both blocks are padding
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  // The Gram matrix is symmetric and the sweep reads its upper triangle only: of the 8 x 8 grid of 8 x 8
  // tiles the 36 with tile row <= tile column are formed.  Warps 0 and 3 take the upper halves of the two
  // diagonal 32 x 32 quadrants (10 tiles each), warps 1 and 2 the two column halves of the off-diagonal one.
  const bool diagonal = warp == 0 || warp == 3;
  const int rb = warp == 3 ? 1 : 0, cb = rb;                     // the diagonal quadrant of warps 0 and 3
  const int jbase = warp == 2 ? 2 : 0;                           // first tile column of warps 1 and 2
  const int c_begin = chunk * kGramChunk;
  const int c_end = min(b, c_begin + kGramChunk);
  const int tiles = (c_end - c_begin + 31) / 32;
  const bool vec = (b & 1) == 0;

  double acc[4][4][2];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j][0] = acc[i][j][1] = 0.0;

  double2 stage[8];
  auto fetch = [&](int tile) {
    const int c0 = c_begin + tile * 32;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int id = tid + 128 * i;
      const int l = id >> 4, col = c0 + (id & 15) * 2;
      const int row = bp.row(l);
      double2 v = make_double2(0.0, 0.0);
      if (row < b) {
        const double* src = X + (int64_t)row * b + col;
        if (vec && col + 1 < c_end) {
          v = *reinterpret_cast<const double2*>(src);
        } else {
          if (col < c_end) v.x = src[0];
          if (col + 1 < c_end) v.y = src[1];
        }
      }
      stage[i] = v;
    }
  };
  auto stash = [&](int buf) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int id = tid + 128 * i;
      *reinterpret_cast<double2*>(&Xs[buf][id >> 4][(id & 15) * 2]) = stage[i];
    }
  };

  fetch(0);
  stash(0);
  __syncthreads();
  for (int tile = 0; tile < tiles; ++tile) {
    const int buf = tile & 1;
    if (tile + 1 < tiles) fetch(tile + 1);
#pragma unroll
    if (diagonal) {            // upper half of a diagonal quadrant: tiles (i, j) with i <= j
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        double a[4], bb[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) a[i] = Xs[buf][rb * 32 + i * 8 + g][ks * 4 + t];
#pragma unroll
        for (int j = 0; j < 4; ++j) bb[j] = Xs[buf][cb * 32 + j * 8 + g][ks * 4 + t];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = i; j < 4; ++j) dmma(acc[i][j], a[i], bb[j]);
      }
    } else {                   // two of the four tile columns of the off-diagonal quadrant (kept in acc[.][0..1])
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        double a[4], bb[2];
#pragma unroll
        for (int i = 0; i < 4; ++i) a[i] = Xs[buf][i * 8 + g][ks * 4 + t];
#pragma unroll
        for (int j = 0; j < 2; ++j) bb[j] = Xs[buf][32 + (jbase + j) * 8 + g][ks * 4 + t];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 2; ++j) dmma(acc[i][j], a[i], bb[j]);
      }
    }
    if (tile + 1 < tiles) stash(buf ^ 1);
    __syncthreads();
  }

  double* out = part + ((int64_t)pair * chunks + chunk) * (kPairRows * kPairRows);
  if (diagonal) {
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = i; j < 4; ++j) {
        const int r = rb * 32 + i * 8 + g, c = cb * 32 + j * 8 + 2 * t;
        *reinterpret_cast<double2*>(out + r * kPairRows + c) = make_double2(acc[i][j][0], acc[i][j][1]);
      }
  } else {
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int r = i * 8 + g, c = 32 + (jbase + j) * 8 + 2 * t;
        *reinterpret_cast<double2*>(out + r * kPairRows + c) = make_double2(acc[i][j][0], acc[i][j][1]);
      }
  }
}

// One cyclic sweep over the 64 rows of a block pair, run on their Gram matrix A, with the rotations
// accumulated into Rot (Rot <- R Rot, so that the rows themselves become Rot x rows).
//
// The 64 rows sit at the 64 positions of a round-robin table; slot k pairs positions k and 63 - k.
// After every round the rows move on by one position (position 0 stays), and the data moves with
// them: a round reads A and Rot from one shared-memory copy and writes the other copy at the next
// positions, so every address a thread touches is the same in all rounds and is computed once.
// After the 63 rounds of a sweep all rows are back where they started.
//   * A is kept as its upper triangle in position space (entry (i, j) at [min][max]).  The 32
//     rotations of a round split it into 2 x 2 blocks (positions of slot u x positions of slot v)
//     that transform independently, B <- R_u B R_v^T; the 528 blocks with u <= v are the work.
//   * Rot: the two rows of a slot are rotated, 64 columns each.
//   * The angle is computed in single precision (after scaling by the exponent of the larger of
//     aqq - app and 2 apq) and (c, s) are then renormalised in double precision: the rotation is
//     orthogonal to double rounding, its angle accurate to about 1e-7, which leaves the pair
//     orthogonal to 1e-7 of what it was.
// flags[pair] = rotations applied (0: Rot is the identity and is not written).
constexpr int kSweepRounds = kPairRows - 1;
constexpr int kSlots = kPairRows / 2;
constexpr int kBlockTasks = kSlots * (kSlots + 1) / 2;
constexpr int kSweepThreads = 512;
constexpr int kALd = kPairRows + 1;
constexpr size_t kSweepSmem = 2 * (size_t)kPairRows * kALd * sizeof(double);   // A and Rot: three CTAs fit on an SM

__host__ __device__ __forceinline__ int next_position(int pos) { return pos == 0 ? 0 : (pos == kPairRows - 1 ? 1 : pos + 1); }
__host__ __device__ __forceinline__ int upper_offset(int i, int j) { return i < j ? i * kALd + j : j * kALd + i; }

struct BlockTask {
  int u, v;        // slots
  int rd[4];       // offsets of (fu, fv), (fu, gv), (gu, fv), (gu, gv) in the current copy
  int wr[4];       // offsets of the same entries, one position on, in the other copy
};
__device__ __forceinline__ BlockTask make_block_task(int task) {
  BlockTask t;
  int u = 0, start = 0;
  while (u + 1 < kSlots && start + (kSlots - u) <= task) { start += kSlots - u; ++u; }
  t.u = u;
  t.v = min(kSlots - 1, u + (task - start));
  const int fu = t.u, gu = kPairRows - 1 - t.u, fv = t.v, gv = kPairRows - 1 - t.v;
  t.rd[0] = upper_offset(fu, fv);
  t.rd[1] = upper_offset(fu, gv);
  t.rd[2] = upper_offset(gu, fv);
  t.rd[3] = upper_offset(gu, gv);
  const int nfu = next_position(fu), ngu = next_position(gu), nfv = next_position(fv), ngv = next_position(gv);
  t.wr[0] = upper_offset(nfu, nfv);
  t.wr[1] = upper_offset(nfu, ngv);
  t.wr[2] = upper_offset(ngu, nfv);
  t.wr[3] = upper_offset(ngu, ngv);
  return t;
}

// B <- R_u B R_v^T for one 2 x 2 block, in two halves with a barrier between them: the results go back
// into the same copy of A, one position on, once every thread has read its entries.
struct BlockValues {
  double a0, a1, a2, a3;
};
__device__ __forceinline__ BlockValues block_read(const BlockTask& t, const double* A) {
  return BlockValues{A[t.rd[0]], A[t.rd[1]], A[t.rd[2]], A[t.rd[3]]};
}
__device__ __forceinline__ void block_write(const BlockTask& t, const double2* cs, const BlockValues& b, double* A) {
  const double2 ru = cs[t.u], rv = cs[t.v];
  // For u == v the two off-diagonal entries are one stored value; both results agree.
  const double r00 = ru.x * b.a0 - ru.y * b.a2, r01 = ru.x * b.a1 - ru.y * b.a3;
  const double r10 = ru.y * b.a0 + ru.x * b.a2, r11 = ru.y * b.a1 + ru.x * b.a3;
  A[t.wr[0]] = rv.x * r00 - rv.y * r01;
  A[t.wr[1]] = rv.y * r00 + rv.x * r01;
  A[t.wr[2]] = rv.x * r10 - rv.y * r11;
  A[t.wr[3]] = rv.y * r10 + rv.x * r11;
}

__global__ void __launch_bounds__(kSweepThreads, 2) jb_sweep_kernel(const double* __restrict__ part, int chunks, int b, int nblk,
                                                                 int round, double tol, double* __restrict__ rot_out,
                                                                 int* __restrict__ flags, int* __restrict__ rotations,
                                                                 const SlotList slots) {
  extern __shared__ __align__(16) double jb_smem[];
  {
    const int64_t shift = (int64_t)slots.id[blockIdx.y] * slots.bytes;     // blockIdx.y: workspace slot
    part = slot_ptr(part, shift);
    rot_out = slot_ptr(rot_out, shift);
    flags = slot_ptr(flags, shift);
    rotations = slot_ptr(rotations, shift);
  }
  double* const As = jb_smem;                          // the Gram matrix (upper triangle used)
  double* const Rs = jb_smem + kPairRows * kALd;       // the accumulated rotation
  __shared__ double2 cs[2][kSlots];     // the rotations of the current round and of the next
  const int pair = blockIdx.x, tid = threadIdx.x;
  const BlockPair bp = block_pair(pair, round, nblk);
  if (bp.I * kBlockRows >= b) {
    if (tid == 0) flags[pair] = 0;
    return;
  }
  const double* src = part + (int64_t)pair * chunks * (kPairRows * kPairRows);
  {
    double sum[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) sum[i] = 0.0;
    for (int c = 0; c < chunks; c += 4) {     // four partial matrices in flight
      double v[4][8];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const double* sc = src + (int64_t)(c + j) * (kPairRows * kPairRows);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int idx = tid + kSweepThreads * i;
          const bool upper = ((idx >> 9) <= ((idx >> 3) & 7));       // tile row <= tile column: the rest is not written
          v[j][i] = (c + j < chunks && upper) ? sc[idx] : 0.0;
        }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int i = 0; i < 8; ++i) sum[i] += v[j][i];
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int idx = tid + kSweepThreads * i;
      As[(idx >> 6) * kALd + (idx & 63)] = sum[i];
      Rs[(idx >> 6) * kALd + (idx & 63)] = ((idx >> 6) == (idx & 63)) ? 1.0 : 0.0;
    }
  }
  const BlockTask t0 = make_block_task(tid);                                   // tasks 0 .. 511
  const bool second = tid < kBlockTasks - kSweepThreads;
  const BlockTask t1 = make_block_task(second ? kSweepThreads + tid : 0);      // tasks 512 .. 527
  // Rot: slot tid / 16, columns tid % 16 + 16 i
  const int rslot = tid >> 4, rcol = tid & 15;
  const int rf = rslot * kALd + rcol, rg = (kPairRows - 1 - rslot) * kALd + rcol;
  const int wf = next_position(rslot) * kALd + rcol, wg = next_position(kPairRows - 1 - rslot) * kALd + rcol;
  __syncthreads();
  int applied = 0;
  const double tol2 = tol * tol;
  // the rotation of slot `tid` (positions tid and 63 - tid) from the current A
  auto rotation = [&]() -> double2 {
    const int f = tid, g = kPairRows - 1 - tid;
    const double app = As[f * kALd + f], aqq = As[g * kALd + g], apq = As[f * kALd + g];
    double c = 1.0, s = 0.0;
    if (apq != 0.0 && apq * apq > tol2 * app * aqq) {
      // tan(2 phi) = 2 apq / (aqq - app), |phi| <= pi/4.  With h = hypot(d, o): cos(2 phi) = |d| / h,
      // c = sqrt((1 + |d|/h) / 2), s = sign(d) o / (2 h c).
      const double d = aqq - app, o = 2.0 * apq;
      const int ex = (__double2hiint(fmax(fabs(d), fabs(o))) >> 20) & 0x7ff;
      if (ex >= 1 && ex <= 2045) {
        const double sc = __hiloint2double((2046 - ex) << 20, 0);
        const float df = (float)(d * sc), of = (float)(o * sc);
        const float rh = rsqrtf(fmaf(df, df, of * of));
        const float v = fmaf(0.5f * fabsf(df), rh, 0.5f);
        const float rc = rsqrtf(v);
        const float c0 = v * rc, s0 = (d >= 0.0 ? 0.5f : -0.5f) * of * rh * rc;
        if (s0 != 0.0f) {
          c = (double)c0;
          s = (double)s0;
          const double eps = fma(c, c, fma(s, s, -1.0));          // c0^2 + s0^2 = 1 + eps, |eps| ~ 1e-7
          const double fix = fma(eps, fma(eps, 0.375, -0.5), 1.0);  // (1 + eps)^-1/2 to O(eps^3)
          c *= fix;
          s *= fix;
          ++applied;
        }
      }
    }
    return make_double2(c, s);
  };
  // A round: A <- rotated A (every entry also moves one position on, the round-robin order of the rows),
  // then, side by side, the first warp works out the next round's rotations from the new A while everybody
  // rotates Rot.  Both matrices are updated in place: read, barrier, write.
  //   barrier X: this round's rotations are visible, every thread has read its entries of A, and the previous
  //              round's writes of Rot have landed;
  //   barrier Y: the new A is visible and every thread has read its entries of Rot.
  if (tid < kSlots) cs[0][tid] = rotation();
  for (int rr = 0; rr < kSweepRounds; ++rr) {
    const double2* cur = cs[rr & 1];
    const BlockValues v0 = block_read(t0, As);
    BlockValues v1 = v0;
    if (second) v1 = block_read(t1, As);
    __syncthreads();                                   // X
    block_write(t0, cur, v0, As);
    if (second) block_write(t1, cur, v1, As);
    double rx[4], ry[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      rx[i] = Rs[rf + 16 * i];
      ry[i] = Rs[rg + 16 * i];
    }
    __syncthreads();                                   // Y
    if (tid < kSlots && rr + 1 < kSweepRounds) cs[(rr + 1) & 1][tid] = rotation();
    {
      const double2 r = cur[rslot];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        Rs[wf + 16 * i] = r.x * rx[i] - r.y * ry[i];
        Rs[wg + 16 * i] = r.y * rx[i] + r.x * ry[i];
      }
    }
  }
  __syncthreads();
  if (tid < 32) {
    for (int o = 16; o > 0; o >>= 1) applied += __shfl_xor_sync(0xffffffffu, applied, o);
    applied = __shfl_sync(0xffffffffu, applied, 0);
    if (tid == 0) {
      flags[pair] = applied;
      if (applied) atomicAdd(rotations, applied);
    }
    if (tid == 0) cs[0][0].x = (double)applied;
  }
  __syncthreads();
  if (cs[0][0].x != 0.0) {   // all rows are back at their own positions after the 63 rounds
    const double* Rf = Rs;
    double* out = rot_out + (int64_t)pair * (kPairRows * kPairRows);
    for (int idx = tid; idx < kPairRows * kPairRows; idx += kSweepThreads) out[idx] = Rf[(idx >> 6) * kALd + (idx & 63)];
  }
}

// rows(pair)[:, cols] <- Rot rows(pair)[:, cols]  for X (blockIdx.z = 0) and, if present, Vt (blockIdx.z = 1)
// A CTA owns 128 columns and takes them in two halves of 64: while the first half is multiplied the second
// is already on its way from global memory into registers, and with one half in shared memory three CTAs
// fit on an SM.  Warp (wy, wx) forms rows 32 wy .. + 32, columns 16 wx .. + 16 of a half.
__global__ void __launch_bounds__(256) jb_apply_kernel(double* __restrict__ X, double* __restrict__ Vt, int b, int nblk, int round,
                                                       const double* __restrict__ rot, const int* __restrict__ flags,
                                                       const SlotList slots, int matrices) {
  extern __shared__ __align__(16) double jb_smem[];
  double(*Rs)[kRotLd] = reinterpret_cast<double(*)[kRotLd]>(jb_smem);
  double(*Xs)[kHalfLd] = reinterpret_cast<double(*)[kHalfLd]>(jb_smem + kPairRows * kRotLd);
  const int pair = blockIdx.x;
  const int which = blockIdx.z % matrices;                                  // 0: X, 1: Vt
  {
    const int64_t shift = (int64_t)slots.id[blockIdx.z / matrices] * slots.bytes;
    X = slot_ptr(X, shift);
    Vt = Vt ? slot_ptr(Vt, shift) : Vt;
    rot = slot_ptr(rot, shift);
    flags = slot_ptr(flags, shift);
  }
  if (flags[pair] == 0) return;
  const BlockPair bp = block_pair(pair, round, nblk);
  double* M = which ? Vt : X;
  const int c0 = blockIdx.y * kApplyCols;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int wy = warp >> 2, wx = warp & 3;
  const bool vec = (b & 1) == 0;
  const double* rsrc = rot + (int64_t)pair * (kPairRows * kPairRows);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int id = tid + 256 * i;
    const int l = id >> 5, m2 = (id & 31) * 2;
    *reinterpret_cast<double2*>(&Rs[l][m2]) = *reinterpret_cast<const double2*>(rsrc + l * kPairRows + m2);
  }
  double2 stage[8];
  auto fetch = [&](int half) {             // 64 rows x 64 columns: row id / 32, columns 2 (id % 32) of the half
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int id = tid + 256 * i;
      const int l = id >> 5, cl = (id & 31) * 2;
      const int row = bp.row(l), col = c0 + half * kApplyHalf + cl;
      double2 v = make_double2(0.0, 0.0);
      if (row < b) {
        const double* src = M + (int64_t)row * b + col;
        if (vec && col + 1 < b) {
          v = *reinterpret_cast<const double2*>(src);
        } else {
          if (col < b) v.x = src[0];
          if (col + 1 < b) v.y = src[1];
        }
      }
      stage[i] = v;
    }
  };
  auto stash = [&]() {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int id = tid + 256 * i;
      *reinterpret_cast<double2*>(&Xs[id >> 5][(id & 31) * 2]) = stage[i];
    }
  };
  fetch(0);
  stash();
  __syncthreads();
  const bool second = c0 + kApplyHalf < b;        // the second half holds columns of the matrix
  for (int half = 0; half < 2; ++half) {
    if (half == 0 && second) fetch(1);
    double acc[4][2][2];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 2; ++j) acc[i][j][0] = acc[i][j][1] = 0.0;
#pragma unroll 4
    for (int ks = 0; ks < kPairRows / 4; ++ks) {
      double a[4], bb[2];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = Rs[wy * 32 + i * 8 + g][ks * 4 + t];
#pragma unroll
      for (int j = 0; j < 2; ++j) bb[j] = Xs[ks * 4 + t][wx * 16 + j * 8 + g];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 2; ++j) dmma(acc[i][j], a[i], bb[j]);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int row = bp.row(wy * 32 + i * 8 + g);
      if (row >= b) continue;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int col = c0 + half * kApplyHalf + wx * 16 + j * 8 + 2 * t;
        double* dst = M + (int64_t)row * b + col;
        if (vec && col + 1 < b) {
          *reinterpret_cast<double2*>(dst) = make_double2(acc[i][j][0], acc[i][j][1]);
        } else {
          if (col < b) dst[0] = acc[i][j][0];
          if (col + 1 < b) dst[1] = acc[i][j][1];
        }
      }
    }
    if (half == 1 || !second) break;
    __syncthreads();                               // every warp has read the first half
    stash();
    __syncthreads();
  }
}

struct JacobiGeometry {
  int nblk, pairs, chunks, col_tiles;
};
JacobiGeometry jacobi_geometry(int b) {
  JacobiGeometry g;
  g.nblk = std::max(2, (int)ceil_div(b, kBlockRows));
  g.nblk += g.nblk & 1;
  g.pairs = g.nblk / 2;
  g.chunks = (int)ceil_div(b, kGramChunk);
  g.col_tiles = (int)ceil_div(b, kApplyCols);
  return g;
}

constexpr size_t kApplySmem = (size_t)(kPairRows * kRotLd + kPairRows * kHalfLd) * sizeof(double);

}  // namespace

size_t jacobi_scratch_bytes(int b) {
  const JacobiGeometry g = jacobi_geometry(b);
  const size_t tile = (size_t)kPairRows * kPairRows * sizeof(double);
  return align_up((size_t)g.pairs * g.chunks * tile, 256) + align_up((size_t)g.pairs * tile, 256) +
         align_up((size_t)g.pairs * sizeof(int), 256);
}

galore_status_t jacobi_eigh(double* X, double* Vt, int b, void* scratch, int* counter, double tol, int max_sweeps,
                            int* sweeps_out, cudaStream_t st, const SlotList* slot_list) {
  const SlotList all = slot_list ? *slot_list : single_slot();
  for (int i = 0; i < all.n; ++i)
    if (sweeps_out) sweeps_out[i] = 0;
  if (b < 2) return GALORE_OK;
  const JacobiGeometry g = jacobi_geometry(b);
  const size_t tile = (size_t)kPairRows * kPairRows * sizeof(double);
  char* p = (char*)scratch;
  double* part = (double*)p;
  p += align_up((size_t)g.pairs * g.chunks * tile, 256);
  double* rot = (double*)p;
  p += align_up((size_t)g.pairs * tile, 256);
  int* flags = (int*)p;

  // per device, so set on every call rather than once per process
  GALORE_CUDA_TRY(cudaFuncSetAttribute(jb_sweep_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSweepSmem));
  GALORE_CUDA_TRY(cudaFuncSetAttribute(jb_apply_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kApplySmem));

  // Slots leave the list as they converge (a sweep without a rotation), so every problem sees exactly
  // the sweeps it would see on its own.
  SlotList live = all;
  int where[kMaxSlots];                       // position of live.id[i] in the caller's list
  for (int i = 0; i < all.n; ++i) where[i] = i;
  const int matrices = Vt ? 2 : 1;
  int sweeps = 0;
  while (sweeps < max_sweeps && live.n > 0) {
    for (int i = 0; i < live.n; ++i)
      GALORE_CUDA_TRY(cudaMemsetAsync(slot_ptr(counter, (int64_t)live.id[i] * live.bytes), 0, sizeof(int), st));
    for (int round = 0; round < g.nblk - 1; ++round) {
      jb_gram_kernel<<<dim3(g.pairs, g.chunks, live.n), 128, 0, st>>>(X, b, g.nblk, round, g.chunks, part, live);
      GALORE_LAUNCH_CHECK();
      jb_sweep_kernel<<<dim3(g.pairs, live.n), kSweepThreads, kSweepSmem, st>>>(part, g.chunks, b, g.nblk, round, tol, rot, flags,
                                                                              counter, live);
      GALORE_LAUNCH_CHECK();
      jb_apply_kernel<<<dim3(g.pairs, g.col_tiles, matrices * live.n), 256, kApplySmem, st>>>(X, Vt, b, g.nblk, round, rot, flags,
                                                                                            live, matrices);
      GALORE_LAUNCH_CHECK();
    }
    ++sweeps;
    int rot_count[kMaxSlots] = {};
    for (int i = 0; i < live.n; ++i)
      GALORE_CUDA_TRY(cudaMemcpyAsync(&rot_count[i], slot_ptr(counter, (int64_t)live.id[i] * live.bytes), sizeof(int),
                                      cudaMemcpyDeviceToHost, st));
    GALORE_CUDA_TRY(cudaStreamSynchronize(st));
    int kept = 0;
    for (int i = 0; i < live.n; ++i) {
      if (sweeps_out) sweeps_out[where[i]] = sweeps;
      if (rot_count[i] != 0) {
        live.id[kept] = live.id[i];
        where[kept] = where[i];
        ++kept;
      }
    }
    live.n = kept;
  }
  return GALORE_OK;
}

}  // namespace galore
