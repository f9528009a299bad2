// The 8-bit state code on the device: shared-memory tables and the quantiser, used by the stand-alone
// Adam kernel and by the projection kernel whose epilogue runs Adam (Sec. 4.3 names 8-bit Adam
// states; the format is this library's).
#pragma once

#include <math.h>

#include "common.cuh"

namespace galore {

constexpr int kLutSize = 3584;                 // keys 0 .. 3456 used
constexpr uint32_t kLutBase = 0x32000000u;     // bits of 2^-27: below it every value maps to key 0

// device addresses of the tables (global memory, filled once per device by q8_ensure_tables)
struct Q8TablePtrs {
  const float *code_s, *code_u;     // the 256 code values, signed / unsigned
  const float *mid_s, *mid_u;       // 255 thresholds (midpoints of neighbouring code values), then +inf
  const uint32_t *enc_s, *enc_u;    // quantiser table, one entry per bin of |y| (see q8_encode_fast)
};

struct alignas(16) Q8Tables {
  float code_s[256], code_u[256], mid_s[256], mid_u[256];
  uint32_t enc_s[kLutSize], enc_u[kLutSize];
  float red[48];          // scratch of the CTA-wide reductions of the stand-alone kernel
};

// every thread of the CTA (or of the participating group of `nthreads` threads, numbered tid) copies its share
__device__ __forceinline__ void q8_tables_fill(Q8Tables& t, const Q8TablePtrs& g, int tid, int nthreads) {
  for (int i = tid; i < kLutSize; i += nthreads) {
    t.enc_s[i] = g.enc_s[i];
    t.enc_u[i] = g.enc_u[i];
  }
  for (int i = tid; i < 256; i += nthreads) {
    t.code_s[i] = g.code_s[i];
    t.code_u[i] = g.code_u[i];
    t.mid_s[i] = g.mid_s[i];
    t.mid_u[i] = g.mid_u[i];
  }
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

// Four values of one quantisation block -> four packed codes (byte k = value k).  The fast encoder
// decides all but about 1 value in 15 000; those take one branch for the whole group.
template <bool SIGNED>
__device__ __forceinline__ uint32_t q8_encode4(const float (&x)[4], float absmax, float inv, const uint32_t* __restrict__ enc,
                                               const float* __restrict__ mids) {
  uint32_t packed = 0u, need = 0u;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    bool ex;
    const uint32_t c = q8_encode_fast<SIGNED>(x[k], inv, enc, ex) & 0xffu;
    packed |= c << (8 * k);
    need |= (ex ? 1u : 0u) << k;
  }
  if (need != 0u) {
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (need & (1u << k)) {
        const uint32_t c = (uint32_t)q8_encode(__fdiv_rn(x[k], absmax), mids) & 0xffu;
        packed = (packed & ~(0xffu << (8 * k))) | (c << (8 * k));
      }
  }
  return packed;
}

// Eq. 15 with bias correction.  The square root and the quotient use the approximate hardware
// units (about 2 ulp each): N feeds a bf16 or fp32 GEMM operand and decides no integer.
struct AdamParams {
  float b1, b2;          // beta1, beta2
  float omb1, omb2;      // 1 - beta1, 1 - beta2
  float eps;
  float inv_bc1, inv_bc2;  // 1 / (1 - beta^t), t = completed steps + 1
  float nrm_a, nrm_b;      // Eq. 15 as m / (nrm_a sqrt(v) + nrm_b): sqrt(inv_bc2) / inv_bc1 and eps / inv_bc1
};
// fills the derived fields; beta1, beta2, eps as given by the caller, t = completed steps + 1
inline AdamParams make_adam_params(double beta1, double beta2, double eps, double t) {
  AdamParams ap;
  ap.b1 = (float)beta1;
  ap.b2 = (float)beta2;
  ap.omb1 = (float)(1.0 - beta1);
  ap.omb2 = (float)(1.0 - beta2);
  ap.eps = (float)eps;
  const double ibc1 = 1.0 / (1.0 - pow(beta1, t)), ibc2 = 1.0 / (1.0 - pow(beta2, t));
  ap.inv_bc1 = (float)ibc1;
  ap.inv_bc2 = (float)ibc2;
  ap.nrm_a = (float)(sqrt(ibc2) / ibc1);
  ap.nrm_b = (float)(eps / ibc1);
  return ap;
}

// N = [m / (1 - b1^t)] / (sqrt(v / (1 - b2^t)) + eps), with the two corrections folded into the
// constants of one multiply-add: m / (nrm_a sqrt(v) + nrm_b).
__device__ __forceinline__ float adam_normalised(float m, float v, const AdamParams& p) {
  float root, inv;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(root) : "f"(v));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(inv) : "f"(fmaf(root, p.nrm_a, p.nrm_b)));
  return m * inv;
}

// The moment updates of Algorithm 1 with the rounding order fixed (no contraction left to the
// compiler): code that evaluates them twice for the same element gets the same bits both times.
__device__ __forceinline__ float adam_m(float m_old, float r, const AdamParams& p) {
  return __fmaf_rn(p.b1, m_old, __fmul_rn(p.omb1, r));
}
__device__ __forceinline__ float adam_v(float v_old, float r, const AdamParams& p) {
  return __fmaf_rn(p.b2, v_old, __fmul_rn(p.omb2, __fmul_rn(r, r)));
}

}  // namespace galore
