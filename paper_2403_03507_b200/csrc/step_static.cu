// galore_step_static: one fp32 GaLore-Adam step whose scratch memory lives inside the library.
//
// The regular entry points take a caller-allocated workspace for the two intermediates of a step
// (the split-K partial sums of the projected gradient R and the normalised update N).  Some
// callers have no way of providing one: a host framework may own every byte of device memory
// through its own pool and forbid plug-ins from calling cudaMalloc; an allocation may be
// unacceptable at the call site because cudaMalloc/cudaFree synchronise the whole device; or the
// code runs on a thread that is not allowed to touch the allocator at all.  For those callers the
// intermediates are placed in one fixed array that is part of the loaded module.
//
// The array is shared by every call in the process (per device) and keeps whatever the previous
// call left in it.  Nothing in it needs to start at zero except the word that collects this call's
// status bits, which each call clears itself (a second word accumulates them across calls until
// galore_static_status() reads it); every other byte that is read has been written earlier in the
// same call.  Two
// calls whose GPU work overlaps (different streams, or different host threads) would both write
// the array and race: callers serialise them.
#include <mutex>

#include "adam.cuh"
#include "common.cuh"
#include "gemm_simt.cuh"

namespace galore {

constexpr size_t kStaticScratchBytes = GALORE_STATIC_SCRATCH_BYTES;

// Device storage.  In host code this name is only a handle for the symbol, not an address a
// kernel can use: the device address is looked up once per device with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

static std::mutex g_static_mutex;
static void* g_static_ptr[64] = {};

// Device address of the array on the current device (looked up on the first call per device).
static galore_status_t static_scratch(void** out) {
  int dev = 0;
  GALORE_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return GALORE_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (!g_static_ptr[dev]) {
    void* p = nullptr;
    GALORE_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
    g_static_ptr[dev] = p;
  }
  *out = g_static_ptr[dev];
  return GALORE_OK;
}

// the bits of this call (word 0) are added to the word that only galore_static_status() clears (word 1)
__global__ void fold_status_kernel(int32_t* words) {
  if (words[0]) atomicOr(words + 1, words[0]);
}

// the stream, if one is given, must live on the device whose array is about to be used
static galore_status_t check_stream_device(cudaStream_t st) {
  if (!st || st == cudaStreamLegacy || st == cudaStreamPerThread) return GALORE_OK;
  int cur = 0, dev = 0;
  GALORE_CUDA_TRY(cudaGetDevice(&cur));
  GALORE_CUDA_TRY(cudaStreamGetDevice(st, &dev));
  return dev == cur ? GALORE_OK : GALORE_ERR_INVALID_ARG;
}

}  // namespace galore

using namespace galore;

extern "C" galore_status_t galore_static_status(int32_t* flags, void* stream) {
  if (!flags) return GALORE_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  GALORE_TRY(check_stream_device(st));
  void* base = nullptr;
  GALORE_TRY(static_scratch(&base));
  int32_t f = 0;
  GALORE_CUDA_TRY(cudaMemcpyAsync(&f, (int32_t*)base + 1, sizeof(f), cudaMemcpyDeviceToHost, st));
  GALORE_CUDA_TRY(cudaMemsetAsync((int32_t*)base + 1, 0, sizeof(f), st));
  GALORE_CUDA_TRY(cudaStreamSynchronize(st));
  *flags = f;
  return GALORE_OK;
}

extern "C" galore_status_t galore_step_static(int64_t m, int64_t n, int32_t rank, int32_t side, float alpha,
                                               double beta1, double beta2, double eps, int64_t completed_steps,
                                               const float* P, float* M, float* V, float* W, int64_t ldw,
                                               const float* G, int64_t ldg, float lr, int32_t* device_flags,
                                               void* stream) {
  if (!P || !M || !V || !W || !G) return GALORE_ERR_INVALID_ARG;
  if (m <= 0 || n <= 0 || m > 0x7fffffff || n > 0x7fffffff) return GALORE_ERR_SHAPE;
  if (rank < 1 || rank > (m < n ? m : n)) return GALORE_ERR_SHAPE;
  if (ldw < n || ldg < n || completed_steps < 0) return GALORE_ERR_INVALID_ARG;
  if (side < GALORE_SIDE_AUTO || side > GALORE_SIDE_RIGHT) return GALORE_ERR_INVALID_ARG;
  if (!(beta1 >= 0.0 && beta1 < 1.0) || !(beta2 >= 0.0 && beta2 < 1.0) || !(eps >= 0.0)) return GALORE_ERR_INVALID_ARG;
  const bool left = side == GALORE_SIDE_AUTO ? (m <= n) : (side == GALORE_SIDE_LEFT);
  const int r = rank;
  const int64_t d = left ? m : n;
  const int64_t srows = left ? r : m, scols = left ? n : r;
  const int64_t nel = srows * scols;

  // same choice of K slices as the regular fp32 path, so that results agree bit for bit
  const bool small = nel < (int64_t)128 * 128 * 96;
  const int64_t tile = small ? 64 : 128;
  const int64_t tiles = ceil_div(srows, tile) * ceil_div(scols, tile);
  int want = (int)std::min<int64_t>(16, std::max<int64_t>(1, ceil_div(2 * 148, tiles)));
  want = (int)std::min<int64_t>(want, std::max<int64_t>(1, d / 64));
  const int splits = simt_effective_splits((int)d, want);

  // layout inside the array: [status word 256 B][R partials][N]
  const size_t need = 256 + align_up((size_t)splits * nel * 4, 256) + align_up((size_t)nel * 4, 256);
  if (need > kStaticScratchBytes) return GALORE_ERR_BUFFER_TOO_SMALL;   // layer too large for the built-in scratch

  cudaStream_t st = (cudaStream_t)stream;
  GALORE_TRY(check_stream_device(st));
  void* base = nullptr;
  GALORE_TRY(static_scratch(&base));
  int32_t* status = (int32_t*)base;
  float* Rpart = (float*)((char*)base + 256);
  float* Nbuf = (float*)((char*)base + 256 + align_up((size_t)splits * nel * 4, 256));
  GALORE_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(int32_t), st));   // this call's bits: the one part that must start at zero

  EpiStore<float, float> epi{Rpart, scols, nel, 1.f, 0.f};
  if (left)
    GALORE_TRY((launch_gemm_simt<float, float, float>(r, (int)n, (int)m, P, 1, r, G, ldg, 1, splits, epi, st)));
  else
    GALORE_TRY((launch_gemm_simt<float, float, float>((int)m, r, (int)n, G, ldg, 1, P, r, 1, splits, epi, st)));

  const AdamParams ap = make_adam_params(beta1, beta2, eps, (double)(completed_steps + 1));
  AdamItem item = {};
  item.Rpart = Rpart; item.splits = splits; item.split_stride = nel;
  item.rows = (int)srows; item.cols = (int)scols;
  item.r_ld = item.n_ld = item.s_ld = scols;       // everything packed
  item.M = M; item.V = V; item.Nout = Nbuf;
  item.p = ap; item.status = status;
  GALORE_TRY(launch_adam(item, GALORE_STATE_F32, 2048, GALORE_F32, st));

  EpiApplyW<float> apply{W, ldw, lr * alpha};
  if (left)
    GALORE_TRY((launch_gemm_simt<float, float, float>((int)m, (int)n, r, P, r, 1, Nbuf, n, 1, 1, apply, st)));
  else
    GALORE_TRY((launch_gemm_simt<float, float, float>((int)m, (int)n, r, Nbuf, r, 1, P, 1, r, 1, apply, st)));

  fold_status_kernel<<<1, 1, 0, st>>>(status);
  GALORE_LAUNCH_CHECK();

  if (device_flags) {   // optional: wait for the step and report what the kernels latched
    int32_t f = 0;
    GALORE_CUDA_TRY(cudaMemcpyAsync(&f, status, sizeof(f), cudaMemcpyDeviceToHost, st));
    GALORE_CUDA_TRY(cudaStreamSynchronize(st));
    *device_flags = f;
  }
  return GALORE_OK;
}
