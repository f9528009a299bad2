// Shared host/device helpers of the GaLore CUDA library (sm_100a).
#pragma once

#include <nvtx3/nvToolsExt.h>

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/galore.h"

namespace galore {

// ---- error plumbing ---------------------------------------------------------
void note_cuda_error(cudaError_t e, const char* where);   // stores text for galore_last_cuda_error()
void count_launch(int n = 1);

#define GALORE_CUDA_TRY(expr)                                   \
  do {                                                          \
    cudaError_t e__ = (expr);                                   \
    if (e__ != cudaSuccess) {                                   \
      ::galore::note_cuda_error(e__, #expr);                    \
      return GALORE_ERR_CUDA;                                   \
    }                                                           \
  } while (0)

#define GALORE_TRY(expr)                          \
  do {                                            \
    galore_status_t s__ = (expr);                 \
    if (s__ < 0) return s__;                      \
  } while (0)

// after a kernel launch: counts it and converts a launch failure into a status
#define GALORE_LAUNCH_CHECK()                                   \
  do {                                                          \
    ::galore::count_launch();                                   \
    cudaError_t e__ = cudaGetLastError();                       \
    if (e__ != cudaSuccess) {                                   \
      ::galore::note_cuda_error(e__, "kernel launch");          \
      return GALORE_ERR_CUDA;                                   \
    }                                                           \
  } while (0)

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline size_t dtype_size(int32_t dt) { return dt == GALORE_BF16 ? 2 : 4; }

// ---- element conversion -----------------------------------------------------
template <typename To, typename From>
__host__ __device__ __forceinline__ To cvt(From x) { return static_cast<To>(x); }
template <> __device__ __forceinline__ float cvt<float, __nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }
template <> __device__ __forceinline__ double cvt<double, __nv_bfloat16>(__nv_bfloat16 x) { return (double)__bfloat162float(x); }
template <> __device__ __forceinline__ __nv_bfloat16 cvt<__nv_bfloat16, float>(float x) { return __float2bfloat16_rn(x); }
template <> __device__ __forceinline__ __nv_bfloat16 cvt<__nv_bfloat16, double>(double x) { return __float2bfloat16_rn((float)x); }

// 1 / sqrt(x) in double precision from the single-precision hardware estimate and two Newton steps
// (the latency of the general routine matters in the serial parts of the factorisations).  x is
// first scaled by an even power of two into [1, 4); outside 1e-290 .. 1e290 the general routine runs.
__device__ __forceinline__ double rsqrt_newton(double x) {
  if (!(x > 1e-290 && x < 1e290)) return rsqrt(x);
  const int ex = ((((__double2hiint(x) >> 20) & 0x7ff) - 1023)) & ~1;
  const double xs = x * __hiloint2double((1023 - ex) << 20, 0);
  double y = (double)rsqrtf((float)xs);
  const double h = 0.5 * xs;
  y = fma(y, fma(-h * y, y, 0.5), y);
  y = fma(y, fma(-h * y, y, 0.5), y);
  return y * __hiloint2double((1023 - ex / 2) << 20, 0);
}

// Several copies ("slots") of one workspace layout, `bytes` apart: a launch that carries a slot list
// runs the same problem in every listed slot, all of its workspace pointers shifted by
// id[i] * bytes for the i-th part of the grid.  Used to run the latency-bound small kernels of the
// projector refresh for several layers of the same shape at once.
constexpr int kMaxSlots = 8;
struct SlotList {
  int n;
  int id[kMaxSlots];
  int64_t bytes;
};
inline SlotList single_slot() {
  SlotList s = {};
  s.n = 1;
  return s;
}
template <typename T>
__host__ __device__ __forceinline__ T* slot_ptr(T* p, int64_t shift) {
  return (T*)((char*)p + shift);
}

// Status word in the workspace (first 256 bytes).
struct DeviceStatus {
  int32_t flags;
  int32_t pad[63];
};

// A named range on the calling thread for timeline tools (NVTX; a few nanoseconds when no tool listens).
struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
  NvtxRange(const NvtxRange&) = delete;
  NvtxRange& operator=(const NvtxRange&) = delete;
};

}  // namespace galore
