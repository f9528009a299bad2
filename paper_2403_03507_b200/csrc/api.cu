// C ABI of the GaLore-Adam step library: handle, buffer layout, argument
// checks and the launch sequence of one iteration of Algorithm 1.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <atomic>
#include <memory>
#include <mutex>
#include <new>
#include <vector>
#include <string>

#include "adafactor.cuh"
#include "adam.cuh"
#include "common.cuh"
#include "gemm_simt.cuh"
#include "gemm_tc.cuh"
#include "refresh.cuh"

namespace galore {

static thread_local std::string t_last_error;
static std::atomic<int64_t> g_launches{0};

void note_cuda_error(cudaError_t e, const char* where) {
  t_last_error = std::string(cudaGetErrorName(e)) + ": " + cudaGetErrorString(e) + " at " + where;
}
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

// ---- optional phase timing (benchmarks) ------------------------------------------
struct PhaseEvent { int phase; cudaEvent_t a, b; };
static std::atomic<int> g_profile{0};
static std::mutex g_profile_mutex;
static std::vector<PhaseEvent> g_phase_events;

static const char* const kPhaseNames[3] = {"galore.project", "galore.adam", "galore.back_project"};
struct PhaseTimer {
  NvtxRange range;      // the phase on the host timeline (launches are asynchronous: the kernels follow on the stream)
  bool on;
  PhaseEvent ev;
  cudaStream_t st;
  PhaseTimer(int phase, cudaStream_t s) : range(kPhaseNames[phase]), on(g_profile.load(std::memory_order_relaxed) != 0), st(s) {
    if (!on) return;
    ev.phase = phase;
    if (cudaEventCreate(&ev.a) != cudaSuccess || cudaEventCreate(&ev.b) != cudaSuccess) { on = false; return; }
    cudaEventRecord(ev.a, st);
  }
  ~PhaseTimer() {
    if (!on) return;
    cudaEventRecord(ev.b, st);
    std::lock_guard<std::mutex> lock(g_profile_mutex);
    g_phase_events.push_back(ev);
  }
};

template <typename TS, typename TD>
__global__ void convert_copy_kernel(const TS* __restrict__ src, TD* __restrict__ dst, int64_t count) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x)
    dst[i] = cvt<TD>(src[i]);
}

}  // namespace galore

using namespace galore;

struct galore_layer {
  galore_config_t cfg;
  bool left;
  bool tensor_path;
  bool has_projector;
  int64_t d;             // rows of the projector (m left, n right)
  int64_t L;             // the other dimension of G
  int64_t srows, scols;  // shape of R, M, V
  int64_t nel;
  int q_block;
  int64_t nblk;
  int block;             // columns of the refresh block
  int proj_splits;       // K slices of the projection on the fp32 path
  int tc_splits;         // K slices of the projection on the tensor-core path
  int64_t ld_part, ld_n; // padded row pitches of the R partials and of N on the tensor-core path
  int64_t ld_s;          // row pitch of the state arrays (fp32 moments: floats, 8-bit codes: bytes)
  int32_t n_dtype;       // dtype of the normalised update handed to the back-projection
  int64_t k;             // completed steps
  // device memory (all inside the caller's two buffers)
  void* P;
  float *M, *V;
  float *v_row, *v_col;  // Adafactor: running means of R^2 along rows and columns (V is unused then)
  float* af_scratch;
  uint8_t *Mc, *Vc;
  float *Mam, *Vam;
  int32_t* status;
  float* Rpart;
  void* Nbuf;
  void* refresh_ws;
  size_t state_bytes;    // size of the caller's state buffer as laid out here (it starts at P)
  bool refreshed_here = false;   // the last refresh ran in refresh_ws (its unrounded projector is still there)
  TensorPlan tc;         // tensor-map state of the tcgen05 path (unused on the fp32 path)
};

namespace {

struct Sizes {
  bool left;
  int64_t d, L, srows, scols, nel, nblk;
  int q_block, block, proj_splits, tc_splits;
  int64_t ld_part, ld_n, ld_s;
  bool tensor_path;
  size_t off_P, off_M, off_V, off_Mam, off_Vam, state_bytes;
  size_t off_vrow, off_vcol;
  size_t off_status, off_R, off_N, off_af, off_refresh, ws_bytes;
};

galore_status_t resolve(const galore_config_t* c, Sizes* s) {
  if (!c || !s) return GALORE_ERR_INVALID_ARG;
  if (c->m <= 0 || c->n <= 0 || c->m > 0x7fffffff || c->n > 0x7fffffff) return GALORE_ERR_SHAPE;
  if (c->rank < 1 || c->rank > std::min(c->m, c->n)) return GALORE_ERR_SHAPE;
  if (c->refresh_gap < 1) return GALORE_ERR_INVALID_ARG;
  if (!(c->beta1 >= 0.0 && c->beta1 < 1.0) || !(c->beta2 >= 0.0 && c->beta2 < 1.0) || !(c->eps >= 0.0))
    return GALORE_ERR_INVALID_ARG;
  if (!(c->weight_decay >= 0.0f) || !(c->weight_decay < 1e6f)) return GALORE_ERR_INVALID_ARG;
  if (c->side < GALORE_SIDE_AUTO || c->side > GALORE_SIDE_RIGHT) return GALORE_ERR_INVALID_ARG;
  for (int32_t dt : {c->w_dtype, c->g_dtype, c->p_dtype})
    if (dt != GALORE_F32 && dt != GALORE_BF16) return GALORE_ERR_INVALID_ARG;
  if (c->state_fmt < GALORE_STATE_F32 || c->state_fmt > GALORE_STATE_ADAFACTOR) return GALORE_ERR_INVALID_ARG;
  if (c->path < GALORE_PATH_AUTO || c->path > GALORE_PATH_TENSOR) return GALORE_ERR_INVALID_ARG;
  if (c->adam_place < GALORE_ADAM_AUTO || c->adam_place > GALORE_ADAM_OWN_KERNEL) return GALORE_ERR_INVALID_ARG;
  if (c->refresh_warm_iters < 0) return GALORE_ERR_INVALID_ARG;
  s->q_block = c->q_block == 0 ? 2048 : c->q_block;
  if (s->q_block != 256 && s->q_block != 512 && s->q_block != 1024 && s->q_block != 2048)
    return GALORE_ERR_INVALID_ARG;
  s->left = c->side == GALORE_SIDE_AUTO ? (c->m <= c->n) : (c->side == GALORE_SIDE_LEFT);
  const int r = c->rank;
  s->d = s->left ? c->m : c->n;
  s->L = s->left ? c->n : c->m;
  s->srows = s->left ? r : c->m;
  s->scols = s->left ? c->n : r;
  s->nel = s->srows * s->scols;
  s->ld_s = state_pitch(c->state_fmt, s->scols);
  s->nblk = state_tiles(s->srows, s->scols, s->q_block);
  // the kernels count tiles and address rows of one matrix with 32-bit integers
  if (s->srows * std::max<int64_t>(s->ld_s, (s->scols + 7) / 8 * 8) >= ((int64_t)1 << 31) - 4096) return GALORE_ERR_SHAPE;
  const bool eligible = tensor_path_eligible(*c);
  if (c->path == GALORE_PATH_TENSOR && !eligible) return GALORE_ERR_UNIMPLEMENTED;
  s->tensor_path = eligible && c->path != GALORE_PATH_FP32;
  // Extra columns of the refresh block.  More of them mean fewer power steps but a larger dense
  // eigenproblem (cubic in the block).  Where the steps run on the tensor cores and slow blocks are
  // finished by Chebyshev pairs they are cheap: a quarter of the rank, at least 256, balances the two
  // (LLaMA-7B shapes at rank 1024, groups of eight: 168 / 295 ms with 256 extra columns against
  // 205 / 318 ms with 512 and 165 / 308 ms with 192; a small rank needs the absolute floor to
  // converge on flat spectra at all); elsewhere the block is twice the rank.
  int over = c->refresh_oversample;
  if (over == 0) over = s->tensor_path ? std::max(256, r / 4) : r;
  over = std::max(0, over);
  s->block = (int)std::min<int64_t>(s->d, (int64_t)r + over);

  // K slices of the projection: enough CTAs to fill the machine when R is small
  {
    const bool small = s->nel < (int64_t)128 * 128 * 96;
    const int64_t t = small ? 64 : 128;
    const int64_t tiles = ceil_div(s->srows, t) * ceil_div(s->scols, t);
    int want = (int)std::min<int64_t>(16, std::max<int64_t>(1, ceil_div(2 * 148, tiles)));
    want = (int)std::min<int64_t>(want, std::max<int64_t>(1, s->d / 64));
    s->proj_splits = simt_effective_splits((int)s->d, want);
  }
  s->tc_splits = s->tensor_path ? tensor_proj_splits(*c, s->left) : 0;
  s->ld_part = (s->scols + 7) / 8 * 8;     // 32-byte rows for whole-sector vector stores
  s->ld_n = (s->scols + 15) / 16 * 16;     // 32-byte bf16 rows: TMA needs 16, the epilogue that writes N stores 32 at a time

  size_t o = 0;
  s->off_P = o; o += align_up((size_t)s->d * r * dtype_size(c->p_dtype), 256);
  s->off_vrow = s->off_vcol = 0;
  if (c->state_fmt == GALORE_STATE_F32) {
    s->off_M = o; o += align_up((size_t)s->srows * s->ld_s * 4, 256);
    s->off_V = o; o += align_up((size_t)s->srows * s->ld_s * 4, 256);
    s->off_Mam = s->off_Vam = o;
  } else if (c->state_fmt == GALORE_STATE_ADAFACTOR) {
    s->off_M = o; o += align_up((size_t)s->srows * s->ld_s * 4, 256);
    s->off_vrow = o; o += align_up((size_t)s->srows * 4, 256);
    s->off_vcol = o; o += align_up((size_t)s->scols * 4, 256);
    s->off_V = s->off_Mam = s->off_Vam = o;
  } else {
    s->off_M = o; o += align_up((size_t)s->srows * s->ld_s, 256);
    s->off_V = o; o += align_up((size_t)s->srows * s->ld_s, 256);
    s->off_Mam = o; o += align_up((size_t)s->nblk * 4, 256);
    s->off_Vam = o; o += align_up((size_t)s->nblk * 4, 256);
  }
  s->state_bytes = o;

  o = 0;
  s->off_status = o; o += 256;
  s->off_R = o; o += align_up(std::max((size_t)s->proj_splits * s->nel, (size_t)s->tc_splits * s->srows * s->ld_part) * 4, 256);
  s->off_N = o; o += align_up(std::max((size_t)s->nel * 4, (size_t)s->srows * s->ld_n * 2), 256);
  s->off_af = o;
  if (c->state_fmt == GALORE_STATE_ADAFACTOR) o += adafactor_scratch_bytes(s->srows, s->scols);
  s->off_refresh = o; o += refresh_workspace_bytes(s->d, s->L, r, s->block);
  s->ws_bytes = o;
  return GALORE_OK;
}

template <typename TS, typename TD>
galore_status_t convert_copy(const TS* src, TD* dst, int64_t count, cudaStream_t st) {
  if (count <= 0) return GALORE_OK;
  unsigned grid = (unsigned)std::min<int64_t>(ceil_div(count, 256), 148 * 8);
  convert_copy_kernel<TS, TD><<<grid, 256, 0, st>>>(src, dst, count);
  GALORE_LAUNCH_CHECK();
  return GALORE_OK;
}

// ---- the two projections on the fp32 path ------------------------------------------

template <typename TP, typename TG>
galore_status_t project_simt(galore_layer* l, const void* G, int64_t ldg, cudaStream_t st) {
  const int r = l->cfg.rank;
  EpiStore<float, float> epi{l->Rpart, l->scols, l->nel, 1.f, 0.f};
  if (l->left)   // R (r x n) = P^T G
    return launch_gemm_simt<TP, TG, float>(r, (int)l->cfg.n, (int)l->cfg.m, (const TP*)l->P, 1, r, (const TG*)G, ldg, 1,
                                           l->proj_splits, epi, st);
  // R (m x r) = G Q
  return launch_gemm_simt<TG, TP, float>((int)l->cfg.m, r, (int)l->cfg.n, (const TG*)G, ldg, 1, (const TP*)l->P, r, 1,
                                         l->proj_splits, epi, st);
}

// the layer's share of an Adam launch: R partials in `part` (pitch r_ld), N to `nbuf` (pitch n_ld)
AdamItem adam_item(const galore_layer* l, const float* part, int splits, int64_t split_stride, int64_t r_ld, void* nbuf,
                   int64_t n_ld, const AdamParams& ap) {
  AdamItem a = {};
  a.Rpart = part; a.splits = splits; a.split_stride = split_stride;
  a.rows = (int)l->srows; a.cols = (int)l->scols;
  a.r_ld = r_ld; a.n_ld = n_ld; a.s_ld = l->ld_s;
  a.M = l->M; a.V = l->V; a.Mc = l->Mc; a.Vc = l->Vc; a.Mam = l->Mam; a.Vam = l->Vam;
  a.Nout = nbuf;
  a.p = ap;
  a.status = l->status;
  return a;
}

// the layer's Adafactor step on the same buffers
AdafactorItem adafactor_item(const galore_layer* l, const AdamItem& a, float* scratch) {
  AdafactorItem f = {};
  f.Rpart = const_cast<float*>(a.Rpart); f.splits = a.splits; f.split_stride = a.split_stride;
  f.rows = a.rows; f.cols = a.cols;
  f.r_ld = a.r_ld; f.n_ld = a.n_ld; f.s_ld = a.s_ld;
  f.M = l->M; f.v_row = l->v_row; f.v_col = l->v_col;
  f.Nout = a.Nout;
  f.beta1 = (float)l->cfg.beta1;
  f.t = (double)(l->k + 1);
  f.scratch = scratch;
  return f;
}
galore_status_t launch_regulariser(const galore_layer* l, const AdamItem& a, int32_t n_dtype, cudaStream_t st) {
  if (l->cfg.state_fmt != GALORE_STATE_ADAFACTOR) return launch_adam(a, l->cfg.state_fmt, l->q_block, n_dtype, st);
  return launch_adafactor(adafactor_item(l, a, l->af_scratch), n_dtype, st);
}

// GaLore-AdamW: W is multiplied by 1 - lr * lambda in the pass that subtracts the update (exactly 1 for lambda = 0)
inline float decay_keep(const galore_layer* l, float lr) { return (float)(1.0 - (double)lr * (double)l->cfg.weight_decay); }

template <typename TP, typename TW>
galore_status_t back_project_simt(galore_layer* l, void* W, int64_t ldw, float scale, float keep, cudaStream_t st) {
  const int r = l->cfg.rank;
  const int m = (int)l->cfg.m, n = (int)l->cfg.n;
  EpiApplyW<TW> epi{(TW*)W, ldw, scale, keep};
  const float* N = (const float*)l->Nbuf;
  if (l->left)   // W -= scale * P N,  N is r x n
    return launch_gemm_simt<TP, float, float>(m, n, r, (const TP*)l->P, r, 1, N, n, 1, 1, epi, st);
  // W -= scale * N Q^T,  N is m x r
  return launch_gemm_simt<float, TP, float>(m, n, r, N, r, 1, (const TP*)l->P, 1, r, 1, epi, st);
}

galore_status_t step_simt(galore_layer* l, void* W, int64_t ldw, const void* G, int64_t ldg, float lr,
                          const AdamParams& ap, cudaStream_t st) {
  const bool pb = l->cfg.p_dtype == GALORE_BF16, gb = l->cfg.g_dtype == GALORE_BF16, wb = l->cfg.w_dtype == GALORE_BF16;
  {
    PhaseTimer pt(0, st);
    if (pb && gb) GALORE_TRY((project_simt<__nv_bfloat16, __nv_bfloat16>(l, G, ldg, st)));
    else if (pb) GALORE_TRY((project_simt<__nv_bfloat16, float>(l, G, ldg, st)));
    else if (gb) GALORE_TRY((project_simt<float, __nv_bfloat16>(l, G, ldg, st)));
    else GALORE_TRY((project_simt<float, float>(l, G, ldg, st)));
  }
  {
    PhaseTimer pt(1, st);
    GALORE_TRY(launch_regulariser(l, adam_item(l, l->Rpart, l->proj_splits, l->nel, l->scols, l->Nbuf, l->scols, ap), GALORE_F32, st));
  }
  PhaseTimer pt(2, st);
  const float scale = lr * l->cfg.alpha, keep = decay_keep(l, lr);
  if (pb && wb) return back_project_simt<__nv_bfloat16, __nv_bfloat16>(l, W, ldw, scale, keep, st);
  if (pb) return back_project_simt<__nv_bfloat16, float>(l, W, ldw, scale, keep, st);
  if (wb) return back_project_simt<float, __nv_bfloat16>(l, W, ldw, scale, keep, st);
  return back_project_simt<float, float>(l, W, ldw, scale, keep, st);
}

// projection and back-projection on tcgen05, Adam in between reading the padded partials
// GALORE_ADAM_AUTO, by state format {fp32, 8-bit}.  fp32 moments: the epilogue's work is loads, five
// multiply-adds and stores per element and hides under the MMAs of the next tile (LLaMA-1B set: 1.86 ms
// against 1.01 + 1.14 ms for projection and Adam apart).  8-bit moments: about a hundred dependent
// instructions per element with table lookups in between; the 16 epilogue warps that fit beside the
// tensor-core pipeline issue 0.3 instructions per cycle and scheduler, the stand-alone kernel with 40
// warps per SM 0.7, and the tile's epilogue then takes twice as long as its MMAs (LLaMA-7B set: 21.1 ms
// against 10.3 + 8.0 ms apart).  So 8-bit moments keep the stand-alone kernel unless asked otherwise.
constexpr bool kAutoFuses[2] = {true, false};

TcAdamArgs tc_adam_args(const galore_layer* l, void* nbuf, const AdamParams& ap) {
  TcAdamArgs a = {};
  a.state_fmt = l->cfg.state_fmt;
  a.M = l->M; a.V = l->V; a.Mc = l->Mc; a.Vc = l->Vc; a.Mam = l->Mam; a.Vam = l->Vam;
  a.ld_s = l->ld_s;
  a.q_block = l->q_block;
  a.Nout = nbuf;
  a.ld_n = l->ld_n;
  a.ap = ap;
  return a;
}

// Adam in the projection's epilogue?  Only when K is not sliced; AUTO: see the note at its definition.
bool adam_in_projection(const galore_layer* l, int splits) {
  if (splits != 1 || l->cfg.adam_place == GALORE_ADAM_OWN_KERNEL || l->cfg.state_fmt == GALORE_STATE_ADAFACTOR) return false;
  if (l->cfg.adam_place == GALORE_ADAM_IN_PROJECTION) return true;
  return kAutoFuses[l->cfg.state_fmt == GALORE_STATE_F32 ? 0 : 1];
}

galore_status_t step_tensor(galore_layer* l, void* W, int64_t ldw, const void* G, int64_t ldg, float lr,
                            const AdamParams& ap, cudaStream_t st) {
  if (adam_in_projection(l, l->tc.splits)) {
    // one K slice per tile: Adam runs in the projection's epilogue, R never reaches memory
    PhaseTimer pt(0, st);
    GALORE_TRY(tensor_project_adam(&l->tc, l->cfg, l->left, G, ldg, tc_adam_args(l, l->Nbuf, ap), l->status, st));
  } else {
   {
    PhaseTimer pt(0, st);
    GALORE_TRY(tensor_project(&l->tc, l->cfg, l->left, G, ldg, l->status, st));
  }
  {
    PhaseTimer pt(1, st);
    GALORE_TRY(launch_regulariser(l, adam_item(l, l->Rpart, l->tc.splits, l->srows * l->ld_part, l->ld_part, l->Nbuf, l->ld_n, ap),
                                  GALORE_BF16, st));
   }
  }
  PhaseTimer pt(2, st);
  return tensor_back_project(&l->tc, l->cfg, l->left, W, ldw, lr * l->cfg.alpha, decay_keep(l, lr), l->status, st);
}

RefreshProblem refresh_problem(const galore_layer* l, const void* G, int64_t ldg) {
  RefreshProblem pr;
  pr.G = G;
  pr.g_dtype = l->cfg.g_dtype;
  pr.ldg = ldg;
  pr.m = l->cfg.m;
  pr.n = l->cfg.n;
  pr.left = l->left;
  pr.rank = l->cfg.rank;
  pr.block = l->block;
  pr.P = l->P;
  pr.p_dtype = l->cfg.p_dtype;
  pr.seed = l->cfg.seed;
  pr.tol = l->cfg.refresh_tol > 0.f ? (double)l->cfg.refresh_tol : 1e-4;
  pr.max_iters = l->cfg.refresh_max_iters > 0 ? l->cfg.refresh_max_iters : 96;
  pr.first_iters = 4;
  pr.use_tensor = l->tensor_path;
  pr.warm_iters = (l->cfg.refresh_warm_iters > 0 && l->has_projector) ? l->cfg.refresh_warm_iters : 0;
  return pr;
}

galore_status_t do_refresh(galore_layer* l, const void* G, int64_t ldg, cudaStream_t st, galore_refresh_info_t* info,
                           void* workspace = nullptr) {
  const RefreshProblem pr = refresh_problem(l, G, ldg);
  galore_status_t s = refresh_projector(pr, workspace ? workspace : l->refresh_ws, l->status, info, st);
  if (s >= 0) l->has_projector = true;
  l->refreshed_here = (s >= 0 && workspace == nullptr);
  return s;
}

// layers that can be refreshed in one group: same problem geometry and the same iteration limits
bool same_refresh_shape(const galore_layer* a, const galore_layer* b) {
  return a->cfg.m == b->cfg.m && a->cfg.n == b->cfg.n && a->left == b->left && a->cfg.rank == b->cfg.rank &&
         a->block == b->block && a->cfg.g_dtype == b->cfg.g_dtype && a->tensor_path == b->tensor_path &&
         a->cfg.refresh_max_iters == b->cfg.refresh_max_iters;
}

// ---- layers on the fp32 path in a batch: the same three phases, each one grouped launch ----------------
bool fma_groupable(const galore_layer* l) { return !l->tensor_path && l->has_projector; }
bool fma_same_kind(const galore_layer* a, const galore_layer* b) {
  return a->left == b->left && a->cfg.p_dtype == b->cfg.p_dtype && a->cfg.g_dtype == b->cfg.g_dtype &&
         a->cfg.w_dtype == b->cfg.w_dtype && a->cfg.state_fmt == b->cfg.state_fmt && a->q_block == b->q_block;
}
// with eight or more such layers in flight the K dimension needs no slicing to fill the machine
int fma_splits(const galore_layer* l, int groupable) {
  return simt_effective_splits((int)l->d, groupable >= 8 ? 1 : l->proj_splits);
}
size_t fma_r_bytes(const galore_layer* l, int splits) { return align_up((size_t)splits * l->nel * 4, 256); }
size_t fma_n_bytes(const galore_layer* l) { return align_up((size_t)l->nel * 4, 256); }
size_t fma_layer_bytes(const galore_layer* l, int splits) {
  return fma_r_bytes(l, splits) + fma_n_bytes(l) +
         (l->cfg.state_fmt == GALORE_STATE_ADAFACTOR ? adafactor_scratch_bytes(l->srows, l->scols) : 0);
}

struct FmaProblem {       // one member of a group, with its operands of this call
  galore_layer* l;
  void* W;
  int64_t ldw;
  const void* G;
  int64_t ldg;
  float* part;            // R partials (fma_r_bytes), then N (fp32), then the Adafactor scratch
  int splits;
};

template <typename TP, typename TG>
galore_status_t fma_group_project(const std::vector<FmaProblem>& ps, cudaStream_t st) {
  using Epi = EpiStore<float, float>;
  std::unique_ptr<SimtGroup<Epi>> g(new SimtGroup<Epi>);
  g->count = 0;
  const bool left = ps[0].l->left;
  for (const FmaProblem& q : ps) {
    const galore_layer* l = q.l;
    const int r = l->cfg.rank, m = (int)l->cfg.m, n = (int)l->cfg.n;
    Epi epi{q.part, l->scols, l->nel, 1.f, 0.f};
    if (left)    // R (r x n) = P^T G
      GALORE_TRY(simt_group_add(*g, r, n, m, l->P, 1, r, q.G, q.ldg, 1, q.splits, epi));
    else         // R (m x r) = G Q
      GALORE_TRY(simt_group_add(*g, m, r, n, q.G, q.ldg, 1, l->P, r, 1, q.splits, epi));
  }
  if (left) return launch_gemm_simt_group<TP, TG, float>(*g, st);
  return launch_gemm_simt_group<TG, TP, float>(*g, st);
}

template <typename TP, typename TW>
galore_status_t fma_group_back(const std::vector<FmaProblem>& ps, float lr, cudaStream_t st) {
  using Epi = EpiApplyW<TW>;
  std::unique_ptr<SimtGroup<Epi>> g(new SimtGroup<Epi>);
  g->count = 0;
  const bool left = ps[0].l->left;
  for (const FmaProblem& q : ps) {
    const galore_layer* l = q.l;
    const int r = l->cfg.rank, m = (int)l->cfg.m, n = (int)l->cfg.n;
    const float* N = (const float*)((const char*)q.part + fma_r_bytes(l, q.splits));
    Epi epi{(TW*)q.W, q.ldw, lr * l->cfg.alpha, decay_keep(l, lr)};
    if (left)    // W -= scale * P N,  N is r x n
      GALORE_TRY(simt_group_add(*g, m, n, r, l->P, r, 1, N, n, 1, 1, epi));
    else         // W -= scale * N Q^T,  N is m x r
      GALORE_TRY(simt_group_add(*g, m, n, r, N, r, 1, l->P, 1, r, 1, epi));
  }
  if (left) return launch_gemm_simt_group<TP, float, float>(*g, st);
  return launch_gemm_simt_group<float, TP, float>(*g, st);
}

}  // namespace

extern "C" {

galore_status_t galore_query_bytes(const galore_config_t* cfg, size_t* state_bytes, size_t* workspace_bytes) {
  Sizes s;
  GALORE_TRY(resolve(cfg, &s));
  if (state_bytes) *state_bytes = s.state_bytes;
  if (workspace_bytes) *workspace_bytes = s.ws_bytes;
  return GALORE_OK;
}

galore_status_t galore_init_layer(const galore_config_t* cfg, void* state_buf, size_t state_bytes, void* workspace,
                                  size_t workspace_bytes, void* stream, galore_layer_t** out) {
  if (!out) return GALORE_ERR_INVALID_ARG;
  *out = nullptr;
  Sizes s;
  GALORE_TRY(resolve(cfg, &s));
  if (!state_buf || !workspace) return GALORE_ERR_INVALID_ARG;
  if (((uintptr_t)state_buf | (uintptr_t)workspace) & 255) return GALORE_ERR_ALIGNMENT;
  if (state_bytes < s.state_bytes || workspace_bytes < s.ws_bytes) return GALORE_ERR_BUFFER_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  galore_layer* l = new (std::nothrow) galore_layer();
  if (!l) return GALORE_ERR_INVALID_ARG;
  l->cfg = *cfg;
  l->left = s.left;
  l->tensor_path = s.tensor_path;
  l->has_projector = false;
  l->d = s.d; l->L = s.L; l->srows = s.srows; l->scols = s.scols; l->nel = s.nel;
  l->q_block = s.q_block; l->nblk = s.nblk; l->block = s.block; l->proj_splits = s.proj_splits;
  l->tc_splits = s.tc_splits; l->ld_part = s.ld_part; l->ld_n = s.ld_n; l->ld_s = s.ld_s;
  l->n_dtype = s.tensor_path ? GALORE_BF16 : GALORE_F32;
  l->k = 0;
  char* sb = (char*)state_buf;
  char* ws = (char*)workspace;
  l->P = sb + s.off_P;
  l->M = l->V = nullptr; l->Mc = l->Vc = nullptr; l->Mam = l->Vam = nullptr;
  l->v_row = l->v_col = nullptr; l->af_scratch = nullptr;
  if (cfg->state_fmt == GALORE_STATE_F32) {
    l->M = (float*)(sb + s.off_M);
    l->V = (float*)(sb + s.off_V);
  } else if (cfg->state_fmt == GALORE_STATE_ADAFACTOR) {
    l->M = (float*)(sb + s.off_M);
    l->v_row = (float*)(sb + s.off_vrow);
    l->v_col = (float*)(sb + s.off_vcol);
    l->af_scratch = (float*)(ws + s.off_af);
  } else {
    l->Mc = (uint8_t*)(sb + s.off_M);
    l->Vc = (uint8_t*)(sb + s.off_V);
    l->Mam = (float*)(sb + s.off_Mam);
    l->Vam = (float*)(sb + s.off_Vam);
  }
  l->status = (int32_t*)(ws + s.off_status);
  l->Rpart = (float*)(ws + s.off_R);
  l->Nbuf = ws + s.off_N;
  l->refresh_ws = ws + s.off_refresh;
  l->state_bytes = s.state_bytes;

  cudaError_t e = cudaSuccess;
  if (cfg->state_fmt == GALORE_STATE_F32) {
    e = cudaMemsetAsync(l->M, 0, (size_t)l->srows * l->ld_s * 4, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(l->V, 0, (size_t)l->srows * l->ld_s * 4, st);
  } else if (cfg->state_fmt == GALORE_STATE_ADAFACTOR) {
    e = cudaMemsetAsync(l->M, 0, (size_t)l->srows * l->ld_s * 4, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(l->v_row, 0, (size_t)l->srows * 4, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(l->v_col, 0, (size_t)l->scols * 4, st);
  } else {
    e = cudaMemsetAsync(l->Mc, 127, (size_t)l->srows * l->ld_s, st);   // 127 and 0 are the codes of the value 0
    if (e == cudaSuccess) e = cudaMemsetAsync(l->Vc, 0, (size_t)l->srows * l->ld_s, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(l->Mam, 0, (size_t)l->nblk * 4, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(l->Vam, 0, (size_t)l->nblk * 4, st);
  }
  if (e == cudaSuccess) e = cudaMemsetAsync(l->status, 0, 256, st);
  if (e != cudaSuccess) {
    note_cuda_error(e, "cudaMemsetAsync(state)");
    delete l;
    return GALORE_ERR_CUDA;
  }
  if (l->tensor_path) {
    galore_status_t ts = tensor_plan_init(&l->tc, *cfg, l->left, l->P, l->Nbuf, l->Rpart, l->tc_splits, l->ld_part, l->ld_n);
    if (ts < 0) {
      delete l;
      return ts;
    }
  }
  *out = l;
  return GALORE_OK;
}

galore_status_t galore_refresh_projector(galore_layer_t* l, const void* G, int64_t ldg, void* stream,
                                         galore_refresh_info_t* info) {
  if (!l || !G) return GALORE_ERR_INVALID_ARG;
  if (ldg < l->cfg.n) return GALORE_ERR_INVALID_ARG;
  return do_refresh(l, G, ldg, (cudaStream_t)stream, info);
}

galore_status_t galore_refresh_query_bytes(const galore_layer_t* l, size_t* bytes) {
  if (!l || !bytes) return GALORE_ERR_INVALID_ARG;
  *bytes = refresh_workspace_bytes(l->d, l->L, l->cfg.rank, l->block);
  return GALORE_OK;
}

galore_status_t galore_refresh_batch(galore_layer_t* const* layers, const void* const* G, const int64_t* ldg, int32_t count,
                                     void* workspace, size_t workspace_bytes, void* stream, galore_refresh_info_t* infos) {
  if (count < 0 || (count > 0 && (!layers || !G || !ldg || !workspace))) return GALORE_ERR_INVALID_ARG;
  if ((uintptr_t)workspace & 255) return GALORE_ERR_INVALID_ARG;
  for (int i = 0; i < count; ++i) {
    if (!layers[i] || !G[i] || ldg[i] < layers[i]->cfg.n) return GALORE_ERR_INVALID_ARG;
    if (refresh_workspace_bytes(layers[i]->d, layers[i]->L, layers[i]->cfg.rank, layers[i]->block) > workspace_bytes)
      return GALORE_ERR_BUFFER_TOO_SMALL;
  }
  // Layers of one shape that follow each other in the list are refreshed together, as many at a time
  // as the workspace has room for (at most kMaxSlots): the serial parts of the method then run for
  // all of them in one launch per kernel.
  galore_status_t warn = GALORE_OK;
  int i = 0;
  while (i < count) {
    const size_t slot = refresh_workspace_bytes(layers[i]->d, layers[i]->L, layers[i]->cfg.rank, layers[i]->block);
    const int room = (int)std::min<size_t>(kMaxSlots, workspace_bytes / slot);
    int n = 1;
    while (n < room && i + n < count && same_refresh_shape(layers[i], layers[i + n])) ++n;
    RefreshProblem prs[kMaxSlots];
    int32_t* status[kMaxSlots];
    for (int j = 0; j < n; ++j) {
      prs[j] = refresh_problem(layers[i + j], G[i + j], ldg[i + j]);
      status[j] = layers[i + j]->status;
    }
    const galore_status_t s = refresh_projector_group(prs, n, workspace, slot, status, infos ? &infos[i] : nullptr,
                                                      (cudaStream_t)stream);
    if (s < 0) return s;
    for (int j = 0; j < n; ++j) {
      layers[i + j]->has_projector = true;
      layers[i + j]->refreshed_here = false;
    }
    if (s > warn) warn = s;
    i += n;
  }
  return warn;
}

galore_status_t galore_step(galore_layer_t* l, void* W, int64_t ldw, const void* G, int64_t ldg, float lr, void* stream) {
  if (!l || !W || !G) return GALORE_ERR_INVALID_ARG;
  if (ldw < l->cfg.n || ldg < l->cfg.n) return GALORE_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  galore_status_t warn = GALORE_OK;
  if (l->cfg.auto_refresh && l->k % l->cfg.refresh_gap == 0) {
    galore_status_t s = do_refresh(l, G, ldg, st, nullptr);
    if (s < 0) return s;
    warn = s;
  }
  if (!l->has_projector) return GALORE_ERR_STATE;
  const AdamParams ap = make_adam_params(l->cfg.beta1, l->cfg.beta2, l->cfg.eps, (double)(l->k + 1));
  galore_status_t s;
  if (l->tensor_path && tensor_operands_aligned(l->cfg, W, ldw, G, ldg)) {
    s = step_tensor(l, W, ldw, G, ldg, lr, ap, st);
  } else if (l->tensor_path && l->cfg.path == GALORE_PATH_TENSOR) {
    return GALORE_ERR_ALIGNMENT;     // the caller insisted on tensor cores but these buffers cannot feed TMA
  } else {
    s = step_simt(l, W, ldw, G, ldg, lr, ap, st);
  }
  if (s < 0) return s;
  l->k += 1;
  return warn;
}

galore_status_t galore_step_host(galore_layer_t* l, void* W_host, const void* G_host, void* W_dev, void* G_dev, float lr,
                                 void* stream) {
  if (!l || !W_host || !G_host || !W_dev || !G_dev) return GALORE_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t wb = (size_t)l->cfg.m * l->cfg.n * dtype_size(l->cfg.w_dtype);
  const size_t gb = (size_t)l->cfg.m * l->cfg.n * dtype_size(l->cfg.g_dtype);
  GALORE_CUDA_TRY(cudaMemcpyAsync(W_dev, W_host, wb, cudaMemcpyHostToDevice, st));
  GALORE_CUDA_TRY(cudaMemcpyAsync(G_dev, G_host, gb, cudaMemcpyHostToDevice, st));
  galore_status_t s = galore_step(l, W_dev, l->cfg.n, G_dev, l->cfg.n, lr, stream);
  if (s < 0) return s;
  GALORE_CUDA_TRY(cudaMemcpyAsync(W_host, W_dev, wb, cudaMemcpyDeviceToHost, st));
  return s;
}

// ---- pipelined step for host-resident W and G -------------------------------------------------------
namespace {

int64_t staged_ld(const galore_layer* l) { return (l->cfg.n + 15) / 16 * 16; }   // 32-byte bf16 rows: TMA-addressable
size_t staged_w_bytes(const galore_layer* l) { return align_up((size_t)l->cfg.m * staged_ld(l) * dtype_size(l->cfg.w_dtype), 256); }
size_t staged_g_bytes(const galore_layer* l) { return align_up((size_t)l->cfg.m * staged_ld(l) * dtype_size(l->cfg.g_dtype), 256); }

struct HostPipe {
  int device = -1;
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t start = nullptr;
  std::vector<cudaEvent_t> arrived, stepped, drained;   // per layer, per layer, per slot
  void release() {    // streams and events go back when the thread ends or moves to another device
    if (device < 0) return;
    int cur = 0;
    const bool sw = cudaGetDevice(&cur) == cudaSuccess && cur != device && cudaSetDevice(device) == cudaSuccess;
    for (auto* v : {&arrived, &stepped, &drained}) {
      for (cudaEvent_t e : *v) cudaEventDestroy(e);
      v->clear();
    }
    if (start) cudaEventDestroy(start);
    if (in) cudaStreamDestroy(in);
    if (out) cudaStreamDestroy(out);
    start = nullptr; in = out = nullptr;
    if (sw) cudaSetDevice(cur);
    device = -1;
  }
  ~HostPipe() { release(); }
};

galore_status_t host_pipe_prepare(HostPipe& hp, int dev, size_t layers, size_t slots) {
  if (hp.device != dev) {
    hp.release();
    hp.device = dev;
    GALORE_CUDA_TRY(cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking));
    GALORE_CUDA_TRY(cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking));
    GALORE_CUDA_TRY(cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming));
  }
  auto grow = [](std::vector<cudaEvent_t>& v, size_t n) -> galore_status_t {
    while (v.size() < n) {
      cudaEvent_t e;
      GALORE_CUDA_TRY(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
      v.push_back(e);
    }
    return GALORE_OK;
  };
  GALORE_TRY(grow(hp.arrived, layers));
  GALORE_TRY(grow(hp.stepped, layers));
  GALORE_TRY(grow(hp.drained, slots));
  return GALORE_OK;
}

}  // namespace

galore_status_t galore_host_batch_query_bytes(galore_layer_t* const* layers, int32_t count, int32_t slots, size_t* bytes) {
  if (!layers || !bytes || count < 0 || slots < 1) return GALORE_ERR_INVALID_ARG;
  size_t one = 0;
  for (int i = 0; i < count; ++i) {
    if (!layers[i]) return GALORE_ERR_INVALID_ARG;
    one = std::max(one, staged_w_bytes(layers[i]) + staged_g_bytes(layers[i]));
  }
  *bytes = one * (size_t)slots;
  return GALORE_OK;
}

galore_status_t galore_step_host_batch(galore_layer_t* const* layers, void* const* W_host, const void* const* G_host,
                                       int32_t count, float lr, void* staging, size_t staging_bytes, int32_t slots,
                                       void* stream) {
  if (count < 0 || slots < 1 || (count > 0 && (!layers || !W_host || !G_host || !staging))) return GALORE_ERR_INVALID_ARG;
  if (count == 0) return GALORE_OK;
  if ((uintptr_t)staging & 255) return GALORE_ERR_INVALID_ARG;
  size_t need = 0;
  GALORE_TRY(galore_host_batch_query_bytes(layers, count, slots, &need));
  if (need > staging_bytes) return GALORE_ERR_BUFFER_TOO_SMALL;
  const size_t slot_bytes = need / (size_t)slots;
  for (int i = 0; i < count; ++i)
    if (!W_host[i] || !G_host[i]) return GALORE_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  int dev = 0;
  GALORE_CUDA_TRY(cudaGetDevice(&dev));
  static thread_local HostPipe hp;
  GALORE_TRY(host_pipe_prepare(hp, dev, (size_t)count, (size_t)slots));
  // Three lanes: copies in (hp.in), steps (the caller's stream), copies out (hp.out).  A slot of the
  // staging buffer is filled, stepped and drained in turn; events hand it from lane to lane, so the
  // two directions of the host link and the steps of different layers overlap.
  GALORE_CUDA_TRY(cudaEventRecord(hp.start, st));
  GALORE_CUDA_TRY(cudaStreamWaitEvent(hp.in, hp.start, 0));
  galore_status_t warn = GALORE_OK;
  for (int i = 0; i < count; ++i) {
    galore_layer* l = layers[i];
    const int slot = i % slots;
    char* dW = (char*)staging + (size_t)slot * slot_bytes;
    char* dG = dW + staged_w_bytes(l);
    const int64_t ld = staged_ld(l);
    const size_t we = dtype_size(l->cfg.w_dtype), ge = dtype_size(l->cfg.g_dtype);
    const size_t wrow = (size_t)l->cfg.n * we, grow = (size_t)l->cfg.n * ge;
    if (i >= slots) GALORE_CUDA_TRY(cudaStreamWaitEvent(hp.in, hp.drained[slot], 0));
    GALORE_CUDA_TRY(cudaMemcpy2DAsync(dW, (size_t)ld * we, W_host[i], wrow, wrow, (size_t)l->cfg.m, cudaMemcpyHostToDevice, hp.in));
    GALORE_CUDA_TRY(cudaMemcpy2DAsync(dG, (size_t)ld * ge, G_host[i], grow, grow, (size_t)l->cfg.m, cudaMemcpyHostToDevice, hp.in));
    GALORE_CUDA_TRY(cudaEventRecord(hp.arrived[i], hp.in));
    GALORE_CUDA_TRY(cudaStreamWaitEvent(st, hp.arrived[i], 0));
    const galore_status_t s = galore_step(l, dW, ld, dG, ld, lr, stream);
    if (s < 0) return s;
    if (s > warn) warn = s;
    GALORE_CUDA_TRY(cudaEventRecord(hp.stepped[i], st));
    GALORE_CUDA_TRY(cudaStreamWaitEvent(hp.out, hp.stepped[i], 0));
    GALORE_CUDA_TRY(cudaMemcpy2DAsync(W_host[i], wrow, dW, (size_t)ld * we, wrow, (size_t)l->cfg.m, cudaMemcpyDeviceToHost, hp.out));
    GALORE_CUDA_TRY(cudaEventRecord(hp.drained[slot], hp.out));
  }
  for (int j = 0; j < std::min<int>(slots, count); ++j) GALORE_CUDA_TRY(cudaStreamWaitEvent(st, hp.drained[j], 0));
  return warn;
}

// ---- batched step --------------------------------------------------------------------------------
namespace {

// bytes of group scratch one layer needs: R (one or tc_splits partial buffers) and N, each 256-aligned
// With four or more layers in flight K is not sliced, Adam runs in the projection's epilogue and R is
// never stored: the group scratch of a layer is its N alone.
bool batch_unsliced(int eligible) { return eligible >= 4; }
size_t batch_r_bytes(const galore_layer* l, int splits) {
  return adam_in_projection(l, splits) ? 0 : align_up((size_t)splits * l->srows * l->ld_part * 4, 256);
}
size_t batch_n_bytes(const galore_layer* l) { return align_up((size_t)l->srows * l->ld_n * 2, 256); }
// R partials, N and, for Adafactor, the scratch of its reductions (layers of a group run in the same launches)
size_t batch_layer_bytes(const galore_layer* l, int splits) {
  return batch_r_bytes(l, splits) + batch_n_bytes(l) +
         (l->cfg.state_fmt == GALORE_STATE_ADAFACTOR ? adafactor_scratch_bytes(l->srows, l->scols) : 0);
}

// With several layers in flight there are enough tiles to fill the machine without slicing K.
int batch_splits(const galore_layer* l, int eligible) { return batch_unsliced(eligible) ? 1 : l->tc_splits; }

bool batch_eligible(const galore_layer* l, const void* W, int64_t ldw, const void* G, int64_t ldg) {
  return l->tensor_path && l->has_projector && tensor_operands_aligned(l->cfg, W, ldw, G, ldg);
}

AdamParams adam_params(const galore_layer* l) {
  return make_adam_params(l->cfg.beta1, l->cfg.beta2, l->cfg.eps, (double)(l->k + 1));
}

struct BatchScratch {   // host-side objects reused across calls on this thread
  TensorGroup* proj = nullptr;
  TensorGroup* back = nullptr;
  AdamGroup* adam = nullptr;
  AdafactorGroup* adafactor = nullptr;
  ~BatchScratch() {
    tensor_group_free(proj);
    tensor_group_free(back);
    delete adam;
    delete adafactor;
  }
};

struct BatchMember {
  int index;            // position in the caller's arrays
  size_t offset;        // where its R partials start inside the batch workspace
  int splits;
};

}  // namespace

galore_status_t galore_batch_query_bytes(galore_layer_t* const* layers, int32_t count, size_t* bytes) {
  if (!bytes || count < 0 || (count > 0 && !layers)) return GALORE_ERR_INVALID_ARG;
  int eligible = 0;
  for (int32_t i = 0; i < count; ++i) {
    if (!layers[i]) return GALORE_ERR_INVALID_ARG;
    eligible += layers[i]->tensor_path ? 1 : 0;
  }
  // the largest sum over any run of `capacity` consecutive tensor-path layers: the groups run one after
  // another on the caller's stream and use the same region in turn
  const int cap = std::min(tensor_group_capacity(), (int)kAdamGroup);
  std::vector<size_t> need;
  for (int32_t i = 0; i < count; ++i)
    if (layers[i]->tensor_path) need.push_back(batch_layer_bytes(layers[i], batch_splits(layers[i], eligible)));
  size_t best = 0, run = 0;
  for (size_t i = 0; i < need.size(); ++i) {
    run += need[i];
    if (i >= (size_t)cap) run -= need[i - cap];
    best = std::max(best, run);
  }
  *bytes = best;
  // layers on the fp32 path are grouped the same way, after the others: the larger of the two needs
  int groupable = 0;
  for (int32_t i = 0; i < count; ++i) groupable += layers[i]->tensor_path ? 0 : 1;
  std::vector<size_t> fneed;
  for (int32_t i = 0; i < count; ++i)
    if (!layers[i]->tensor_path) fneed.push_back(fma_layer_bytes(layers[i], fma_splits(layers[i], groupable)));
  const int fcap = std::min((int)kSimtGroup, std::min((int)kAdamGroup, (int)kAdafactorGroup));
  best = run = 0;
  for (size_t i = 0; i < fneed.size(); ++i) {
    run += fneed[i];
    if (i >= (size_t)fcap) run -= fneed[i - fcap];
    best = std::max(best, run);
  }
  *bytes = std::max(*bytes, best);
  return GALORE_OK;
}

galore_status_t galore_step_batch(galore_layer_t* const* layers, void* const* W, const int64_t* ldw, const void* const* G,
                                  const int64_t* ldg, int32_t count, float lr, void* batch_ws, size_t batch_ws_bytes,
                                  void* stream) {
  if (count < 0 || (count > 0 && (!layers || !W || !ldw || !G || !ldg))) return GALORE_ERR_INVALID_ARG;
  if (batch_ws && ((uintptr_t)batch_ws & 255)) return GALORE_ERR_ALIGNMENT;
  cudaStream_t st = (cudaStream_t)stream;
  galore_status_t worst = GALORE_OK;
  // refreshes that are due come first (each synchronises the stream and uses the layer's own workspace)
  int eligible = 0, groupable = 0;
  for (int32_t i = 0; i < count; ++i) {
    galore_layer* l = layers[i];
    if (!l || !W[i] || !G[i] || ldw[i] < l->cfg.n || ldg[i] < l->cfg.n) return GALORE_ERR_INVALID_ARG;
    if (l->cfg.auto_refresh && l->k % l->cfg.refresh_gap == 0) {
      galore_status_t s = do_refresh(l, G[i], ldg[i], st, nullptr);
      if (s < 0) return s;
      worst = std::max(worst, s);
    }
    if (!l->has_projector) return GALORE_ERR_STATE;
    eligible += batch_eligible(l, W[i], ldw[i], G[i], ldg[i]) ? 1 : 0;
    groupable += fma_groupable(l) ? 1 : 0;
  }
  static thread_local BatchScratch scratch;
  if (!scratch.proj) scratch.proj = tensor_group_new();
  if (!scratch.back) scratch.back = tensor_group_new();
  if (!scratch.adam) scratch.adam = new (std::nothrow) AdamGroup;
  if (!scratch.adafactor) scratch.adafactor = new (std::nothrow) AdafactorGroup;
  if (!scratch.proj || !scratch.back || !scratch.adam || !scratch.adafactor) return GALORE_ERR_INVALID_ARG;
  const int cap = std::min(tensor_group_capacity(), std::min((int)kAdamGroup, (int)kAdafactorGroup));

  // ---- 1. partition: layers that cannot be grouped step on their own, the rest form groups ----------
  // The groups run one after another on the caller's stream, each in the whole batch workspace.
  const size_t room = batch_ws_bytes & ~(size_t)255;
  std::vector<std::vector<BatchMember>> groups, fgroups;
  const int fcap = std::min((int)kSimtGroup, std::min((int)kAdamGroup, (int)kAdafactorGroup));
  {
    size_t used = 0;
    std::vector<size_t> fused_bytes_of;
    for (int32_t i = 0; i < count; ++i) {
      galore_layer* l = layers[i];
      const bool ok = batch_ws && batch_eligible(l, W[i], ldw[i], G[i], ldg[i]);
      const int splits = batch_splits(l, eligible);
      const size_t need = ok ? batch_layer_bytes(l, splits) : 0;
      if (!ok && batch_ws && fma_groupable(l) && groupable >= 2) {
        const int fs = fma_splits(l, groupable);
        const size_t fneed = fma_layer_bytes(l, fs);
        if (fneed <= room) {
          // any open group of the same kind takes it (the layers are independent: their order in the list does
          // not matter, so a list in model order, sides alternating, still gives full groups)
          int at = -1;
          for (int gi = (int)fgroups.size() - 1; gi >= 0 && at < 0; --gi)
            if (fma_same_kind(layers[fgroups[gi][0].index], l) && (int)fgroups[gi].size() < fcap && fused_bytes_of[gi] + fneed <= room)
              at = gi;
          if (at < 0) {
            fgroups.emplace_back();
            fused_bytes_of.push_back(0);
            at = (int)fgroups.size() - 1;
          }
          fgroups[at].push_back(BatchMember{i, fused_bytes_of[at], fs});
          fused_bytes_of[at] += fneed;
          continue;
        }
      }
      if (!ok || need > room) {
        // plain step (its refresh, if due, is already done: auto_refresh off for this call)
        const int32_t saved = l->cfg.auto_refresh;
        l->cfg.auto_refresh = 0;
        galore_status_t s = galore_step(l, W[i], ldw[i], G[i], ldg[i], lr, stream);
        l->cfg.auto_refresh = saved;
        if (s < 0) return s;
        worst = std::max(worst, s);
        continue;
      }
      bool fresh = groups.empty();
      if (!fresh) {
        const galore_layer* first = layers[groups.back()[0].index];
        const bool same = first->cfg.w_dtype == l->cfg.w_dtype && first->cfg.state_fmt == l->cfg.state_fmt &&
                          first->q_block == l->q_block && first->tc.ctas == l->tc.ctas &&
                          adam_in_projection(first, groups.back()[0].splits) == adam_in_projection(l, splits);
        fresh = !same || (int)groups.back().size() >= cap || used + need > room;
      }
      if (fresh) {
        groups.emplace_back();
        used = 0;
      }
      groups.back().push_back(BatchMember{i, used, splits});
      used += need;
    }
  }
  if (groups.empty() && fgroups.empty()) return worst;

  // ---- 2. launch helpers -------------------------------------------------------------------------------
  auto scratch_of = [&](size_t gi, const BatchMember& mb, float** part, void** nbuf) {
    const galore_layer* l = layers[mb.index];
    (void)gi;
    char* base = (char*)batch_ws + mb.offset;
    *part = (float*)base;
    *nbuf = base + batch_r_bytes(l, mb.splits);
  };
  auto fused = [&](size_t gi) { return adam_in_projection(layers[groups[gi][0].index], groups[gi][0].splits); };
  auto launch_proj_adam = [&](size_t gi, cudaStream_t s) -> galore_status_t {
    tensor_group_reset(scratch.proj);
    const galore_layer* first = layers[groups[gi][0].index];
    for (const BatchMember& mb : groups[gi]) {
      galore_layer* l = layers[mb.index];
      float* part; void* nbuf;
      scratch_of(gi, mb, &part, &nbuf);
      GALORE_TRY(tensor_group_add_project_adam(scratch.proj, &l->tc, l->cfg, l->left, G[mb.index], ldg[mb.index],
                                               tc_adam_args(l, nbuf, adam_params(l)), l->status));
    }
    PhaseTimer pt(0, s);
    return tensor_group_launch_project_adam(scratch.proj, first->cfg.state_fmt, s);
  };
  auto launch_proj = [&](size_t gi, cudaStream_t s) -> galore_status_t {
    tensor_group_reset(scratch.proj);
    for (const BatchMember& mb : groups[gi]) {
      galore_layer* l = layers[mb.index];
      float* part; void* nbuf;
      scratch_of(gi, mb, &part, &nbuf);
      GALORE_TRY(tensor_group_add_project(scratch.proj, &l->tc, l->cfg, l->left, G[mb.index], ldg[mb.index], part,
                                          l->ld_part, mb.splits, l->status));
    }
    PhaseTimer pt(0, s);
    return tensor_group_launch_project(scratch.proj, s);
  };
  auto launch_adam = [&](size_t gi, cudaStream_t s) -> galore_status_t {
    scratch.adam->count = 0;
    scratch.adafactor->count = 0;
    const galore_layer* first = layers[groups[gi][0].index];
    const bool adafactor = first->cfg.state_fmt == GALORE_STATE_ADAFACTOR;
    for (const BatchMember& mb : groups[gi]) {
      galore_layer* l = layers[mb.index];
      float* part; void* nbuf;
      scratch_of(gi, mb, &part, &nbuf);
      const AdamItem a = adam_item(l, part, mb.splits, l->srows * l->ld_part, l->ld_part, nbuf, l->ld_n, adam_params(l));
      if (adafactor)
        GALORE_TRY(adafactor_group_add(*scratch.adafactor, adafactor_item(l, a, (float*)((char*)nbuf + batch_n_bytes(l)))));
      else
        GALORE_TRY(adam_group_add(*scratch.adam, a, l->cfg.state_fmt, l->q_block));
    }
    PhaseTimer pt(1, s);
    if (adafactor) return launch_adafactor_group(*scratch.adafactor, GALORE_BF16, s);
    return launch_adam_group(*scratch.adam, first->cfg.state_fmt, first->q_block, GALORE_BF16, s);
  };
  auto launch_back = [&](size_t gi, cudaStream_t s) -> galore_status_t {
    tensor_group_reset(scratch.back);
    const galore_layer* first = layers[groups[gi][0].index];
    for (const BatchMember& mb : groups[gi]) {
      galore_layer* l = layers[mb.index];
      float* part; void* nbuf;
      scratch_of(gi, mb, &part, &nbuf);
      GALORE_TRY(tensor_group_add_back(scratch.back, &l->tc, l->cfg, l->left, nbuf, l->ld_n, W[mb.index], ldw[mb.index],
                                       lr * l->cfg.alpha, decay_keep(l, lr), l->status));
    }
    PhaseTimer pt(2, s);
    GALORE_TRY(tensor_group_launch_back(scratch.back, first->cfg.w_dtype, s));
    for (const BatchMember& mb : groups[gi]) layers[mb.index]->k += 1;
    return GALORE_OK;
  };

  // ---- 3. schedule ----------------------------------------------------------------------------------------
  // One stream, the phases of a group back to back.  (Running the Adam pass of group g on a second
  // stream under the projection of group g+1 was measured and dropped: within 2 % either way, and
  // other experiments with two streams of kernels around the tensor-core kernels stalled.)
  for (size_t gi = 0; gi < groups.size(); ++gi) {
    if (fused(gi)) {
      GALORE_TRY(launch_proj_adam(gi, st));
    } else {
      GALORE_TRY(launch_proj(gi, st));
      GALORE_TRY(launch_adam(gi, st));
    }
    GALORE_TRY(launch_back(gi, st));
  }

  // ---- 4. the groups of fp32-path layers -----------------------------------------------------------------
  for (size_t gi = 0; gi < fgroups.size(); ++gi) {
    std::vector<FmaProblem> ps;
    for (const BatchMember& mb : fgroups[gi]) {
      galore_layer* l = layers[mb.index];
      ps.push_back(FmaProblem{l, W[mb.index], ldw[mb.index], G[mb.index], ldg[mb.index],
                              (float*)((char*)batch_ws + mb.offset), mb.splits});
    }
    const galore_layer* first = ps[0].l;
    const bool pb = first->cfg.p_dtype == GALORE_BF16, gb = first->cfg.g_dtype == GALORE_BF16, wb = first->cfg.w_dtype == GALORE_BF16;
    {
      PhaseTimer pt(0, st);
      if (pb && gb) GALORE_TRY((fma_group_project<__nv_bfloat16, __nv_bfloat16>(ps, st)));
      else if (pb) GALORE_TRY((fma_group_project<__nv_bfloat16, float>(ps, st)));
      else if (gb) GALORE_TRY((fma_group_project<float, __nv_bfloat16>(ps, st)));
      else GALORE_TRY((fma_group_project<float, float>(ps, st)));
    }
    {
      scratch.adam->count = 0;
      scratch.adafactor->count = 0;
      const bool adafactor = first->cfg.state_fmt == GALORE_STATE_ADAFACTOR;
      for (const FmaProblem& q : ps) {
        galore_layer* l = q.l;
        char* nbuf = (char*)q.part + fma_r_bytes(l, q.splits);
        const AdamItem a = adam_item(l, q.part, q.splits, l->nel, l->scols, nbuf, l->scols, adam_params(l));
        if (adafactor)
          GALORE_TRY(adafactor_group_add(*scratch.adafactor, adafactor_item(l, a, (float*)(nbuf + fma_n_bytes(l)))));
        else
          GALORE_TRY(adam_group_add(*scratch.adam, a, l->cfg.state_fmt, l->q_block));
      }
      PhaseTimer pt(1, st);
      if (adafactor) GALORE_TRY(launch_adafactor_group(*scratch.adafactor, GALORE_F32, st));
      else GALORE_TRY(launch_adam_group(*scratch.adam, first->cfg.state_fmt, first->q_block, GALORE_F32, st));
    }
    {
      PhaseTimer pt(2, st);
      if (pb && wb) GALORE_TRY((fma_group_back<__nv_bfloat16, __nv_bfloat16>(ps, lr, st)));
      else if (pb) GALORE_TRY((fma_group_back<__nv_bfloat16, float>(ps, lr, st)));
      else if (wb) GALORE_TRY((fma_group_back<float, __nv_bfloat16>(ps, lr, st)));
      else GALORE_TRY((fma_group_back<float, float>(ps, lr, st)));
    }
    for (const FmaProblem& q : ps) q.l->k += 1;
  }
  return worst;
}

galore_status_t galore_free(galore_layer_t* l) {
  if (!l) return GALORE_ERR_INVALID_ARG;
  delete l;
  return GALORE_OK;
}

galore_status_t galore_get_projector(galore_layer_t* l, float* dst, size_t dst_bytes, void* stream) {
  if (!l || !dst) return GALORE_ERR_INVALID_ARG;
  const int64_t count = l->d * l->cfg.rank;
  if (dst_bytes < (size_t)count * 4) return GALORE_ERR_BUFFER_TOO_SMALL;
  if (!l->has_projector) return GALORE_ERR_STATE;
  cudaStream_t st = (cudaStream_t)stream;
  if (l->cfg.p_dtype == GALORE_BF16) return convert_copy((const __nv_bfloat16*)l->P, dst, count, st);
  GALORE_CUDA_TRY(cudaMemcpyAsync(dst, l->P, (size_t)count * 4, cudaMemcpyDeviceToDevice, st));
  return GALORE_OK;
}

galore_status_t galore_get_unrounded_projector(galore_layer_t* l, double* dst, size_t dst_bytes, void* stream) {
  if (!l || !dst) return GALORE_ERR_INVALID_ARG;
  const int64_t count = l->d * l->cfg.rank;
  if (dst_bytes < (size_t)count * 8) return GALORE_ERR_BUFFER_TOO_SMALL;
  if (!l->refreshed_here) return GALORE_ERR_STATE;
  const double* src = refresh_unrounded_projector(l->refresh_ws, l->d, l->L, l->cfg.rank, l->block);
  GALORE_CUDA_TRY(cudaMemcpyAsync(dst, src, (size_t)count * 8, cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
  return GALORE_OK;
}

galore_status_t galore_set_projector(galore_layer_t* l, const float* src, size_t src_bytes, void* stream) {
  if (!l || !src) return GALORE_ERR_INVALID_ARG;
  const int64_t count = l->d * l->cfg.rank;
  if (src_bytes < (size_t)count * 4) return GALORE_ERR_BUFFER_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  if (l->cfg.p_dtype == GALORE_BF16) {
    GALORE_TRY(convert_copy(src, (__nv_bfloat16*)l->P, count, st));
  } else {
    GALORE_CUDA_TRY(cudaMemcpyAsync(l->P, src, (size_t)count * 4, cudaMemcpyDeviceToDevice, st));
  }
  l->has_projector = true;
  return GALORE_OK;
}

galore_status_t galore_get_moments(galore_layer_t* l, float* M, float* V, size_t bytes_each, void* stream) {
  if (!l || !M || !V) return GALORE_ERR_INVALID_ARG;
  if (bytes_each < (size_t)l->nel * 4) return GALORE_ERR_BUFFER_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  if (l->cfg.state_fmt == GALORE_STATE_F32) {
    const size_t row = (size_t)l->scols * 4;
    GALORE_CUDA_TRY(cudaMemcpy2DAsync(M, row, l->M, (size_t)l->ld_s * 4, row, (size_t)l->srows, cudaMemcpyDeviceToDevice, st));
    GALORE_CUDA_TRY(cudaMemcpy2DAsync(V, row, l->V, (size_t)l->ld_s * 4, row, (size_t)l->srows, cudaMemcpyDeviceToDevice, st));
    return GALORE_OK;
  }
  if (l->cfg.state_fmt != GALORE_STATE_Q8_BLOCK) return GALORE_ERR_STATE;   // Adafactor: galore_get_adafactor_state
  const int tr = l->q_block / kStateTileCols;
  GALORE_TRY(launch_q8_dequantize(l->Mc, l->ld_s, l->Mam, l->srows, l->scols, 1, tr, kStateTileCols, M, l->scols, st));
  return launch_q8_dequantize(l->Vc, l->ld_s, l->Vam, l->srows, l->scols, 0, tr, kStateTileCols, V, l->scols, st);
}

galore_status_t galore_get_adafactor_state(galore_layer_t* l, float* M, float* v_row, float* v_col, void* stream) {
  if (!l || !M || !v_row || !v_col) return GALORE_ERR_INVALID_ARG;
  if (l->cfg.state_fmt != GALORE_STATE_ADAFACTOR) return GALORE_ERR_STATE;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t row = (size_t)l->scols * 4;
  GALORE_CUDA_TRY(cudaMemcpy2DAsync(M, row, l->M, (size_t)l->ld_s * 4, row, (size_t)l->srows, cudaMemcpyDeviceToDevice, st));
  GALORE_CUDA_TRY(cudaMemcpyAsync(v_row, l->v_row, (size_t)l->srows * 4, cudaMemcpyDeviceToDevice, st));
  GALORE_CUDA_TRY(cudaMemcpyAsync(v_col, l->v_col, (size_t)l->scols * 4, cudaMemcpyDeviceToDevice, st));
  return GALORE_OK;
}

galore_status_t galore_get_q8_state(galore_layer_t* l, uint8_t* Mc, float* Mam, uint8_t* Vc, float* Vam, void* stream) {
  if (!l || !Mc || !Mam || !Vc || !Vam) return GALORE_ERR_INVALID_ARG;
  if (l->cfg.state_fmt != GALORE_STATE_Q8_BLOCK) return GALORE_ERR_STATE;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t row = (size_t)l->scols;
  GALORE_CUDA_TRY(cudaMemcpy2DAsync(Mc, row, l->Mc, (size_t)l->ld_s, row, (size_t)l->srows, cudaMemcpyDeviceToDevice, st));
  GALORE_CUDA_TRY(cudaMemcpy2DAsync(Vc, row, l->Vc, (size_t)l->ld_s, row, (size_t)l->srows, cudaMemcpyDeviceToDevice, st));
  GALORE_CUDA_TRY(cudaMemcpyAsync(Mam, l->Mam, (size_t)l->nblk * 4, cudaMemcpyDeviceToDevice, st));
  GALORE_CUDA_TRY(cudaMemcpyAsync(Vam, l->Vam, (size_t)l->nblk * 4, cudaMemcpyDeviceToDevice, st));
  return GALORE_OK;
}

galore_status_t galore_get_step_count(const galore_layer_t* l, int64_t* k) {
  if (!l || !k) return GALORE_ERR_INVALID_ARG;
  *k = l->k;
  return GALORE_OK;
}

galore_status_t galore_set_step_count(galore_layer_t* l, int64_t k) {
  if (!l || k < 0) return GALORE_ERR_INVALID_ARG;
  l->k = k;
  return GALORE_OK;
}

galore_status_t galore_layer_info(const galore_layer_t* l, int32_t* side, int32_t* uses_tensor_path, int64_t* state_rows,
                                  int64_t* state_cols) {
  if (!l) return GALORE_ERR_INVALID_ARG;
  if (side) *side = l->left ? GALORE_SIDE_LEFT : GALORE_SIDE_RIGHT;
  if (uses_tensor_path) *uses_tensor_path = l->tensor_path ? 1 : 0;
  if (state_rows) *state_rows = l->srows;
  if (state_cols) *state_cols = l->scols;
  return GALORE_OK;
}

galore_status_t galore_device_status(galore_layer_t* l, int32_t* flags, void* stream) {
  if (!l || !flags) return GALORE_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  int32_t f = 0;
  GALORE_CUDA_TRY(cudaMemcpyAsync(&f, l->status, sizeof(f), cudaMemcpyDeviceToHost, st));
  GALORE_CUDA_TRY(cudaMemsetAsync(l->status, 0, sizeof(f), st));
  GALORE_CUDA_TRY(cudaStreamSynchronize(st));
  *flags = f;
  return GALORE_OK;
}

galore_status_t galore_check_device(galore_layer_t* l, void* stream) {
  int32_t f = 0;
  GALORE_TRY(galore_device_status(l, &f, stream));
  if (f & GALORE_DEV_WAIT_EXPIRED) return GALORE_ERR_TIMEOUT;
  if (f & GALORE_DEV_NONFINITE) return GALORE_ERR_NONFINITE;
  if (f & GALORE_DEV_CHOLESKY) return GALORE_ERR_STATE;
  return GALORE_OK;
}

// ---- checkpoint: what Algorithm 1 carries from one iteration to the next (P, M, V, step count) ----
namespace {

struct ExportHeader {
  uint64_t magic;          // "GALOREST"
  uint32_t version;
  uint32_t header_bytes;
  uint64_t layout_hash;    // of everything that fixes the layout of the state buffer
  int64_t completed_steps;
  int32_t has_projector;
  int32_t reserved;
  uint64_t state_bytes;
};
constexpr uint64_t kExportMagic = 0x5453455230414c47ull;

uint64_t layout_hash(const galore_layer* l) {
  const int64_t fields[] = {l->cfg.m, l->cfg.n, l->cfg.rank, l->left ? 1 : 0, l->cfg.p_dtype, l->cfg.state_fmt,
                            l->q_block, l->ld_s, (int64_t)l->state_bytes};
  uint64_t h = 1469598103934665603ull;          // FNV-1a over the bytes of the fields
  for (int64_t f : fields)
    for (int b = 0; b < 8; ++b) {
      h ^= (uint64_t)(f >> (8 * b)) & 0xffu;
      h *= 1099511628211ull;
    }
  return h;
}

}  // namespace

galore_status_t galore_export_bytes(const galore_layer_t* l, size_t* bytes) {
  if (!l || !bytes) return GALORE_ERR_INVALID_ARG;
  *bytes = sizeof(ExportHeader) + l->state_bytes;
  return GALORE_OK;
}

galore_status_t galore_export_state(galore_layer_t* l, void* dst_host, size_t bytes, void* stream) {
  if (!l || !dst_host) return GALORE_ERR_INVALID_ARG;
  if (bytes < sizeof(ExportHeader) + l->state_bytes) return GALORE_ERR_BUFFER_TOO_SMALL;
  ExportHeader h = {};
  h.magic = kExportMagic;
  h.version = 1;
  h.header_bytes = (uint32_t)sizeof(ExportHeader);
  h.layout_hash = layout_hash(l);
  h.completed_steps = l->k;
  h.has_projector = l->has_projector ? 1 : 0;
  h.state_bytes = l->state_bytes;
  memcpy(dst_host, &h, sizeof(h));
  cudaStream_t st = (cudaStream_t)stream;
  GALORE_CUDA_TRY(cudaMemcpyAsync((char*)dst_host + sizeof(h), l->P, l->state_bytes, cudaMemcpyDeviceToHost, st));
  GALORE_CUDA_TRY(cudaStreamSynchronize(st));
  return GALORE_OK;
}

galore_status_t galore_import_state(galore_layer_t* l, const void* src_host, size_t bytes, void* stream) {
  if (!l || !src_host) return GALORE_ERR_INVALID_ARG;
  if (bytes < sizeof(ExportHeader)) return GALORE_ERR_BUFFER_TOO_SMALL;
  ExportHeader h;
  memcpy(&h, src_host, sizeof(h));
  if (h.magic != kExportMagic || h.version != 1 || h.header_bytes != sizeof(ExportHeader)) return GALORE_ERR_INVALID_ARG;
  if (h.layout_hash != layout_hash(l) || h.state_bytes != l->state_bytes) return GALORE_ERR_STATE;   // another configuration
  if (bytes < sizeof(ExportHeader) + l->state_bytes || h.completed_steps < 0) return GALORE_ERR_BUFFER_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  GALORE_CUDA_TRY(cudaMemcpyAsync(l->P, (const char*)src_host + sizeof(h), l->state_bytes, cudaMemcpyHostToDevice, st));
  GALORE_CUDA_TRY(cudaStreamSynchronize(st));
  l->k = h.completed_steps;
  l->has_projector = h.has_projector != 0;
  l->refreshed_here = false;
  return GALORE_OK;
}

galore_status_t galore_q8_codebook(int32_t is_signed, float* out256_host) {
  if (!out256_host) return GALORE_ERR_INVALID_ARG;
  q8_host_codebook(is_signed != 0, out256_host);
  return GALORE_OK;
}

galore_status_t galore_q8_quantize(const float* x, int64_t rows, int64_t cols, int32_t is_signed, int32_t tile_rows,
                                   int32_t tile_cols, uint8_t* codes, float* absmax, void* stream) {
  if (rows < 0 || cols < 0 || (rows > 0 && cols > 0 && (!x || !codes || !absmax))) return GALORE_ERR_INVALID_ARG;
  return launch_q8_quantize(x, rows, cols, cols, is_signed, tile_rows, tile_cols, codes, cols, absmax, (cudaStream_t)stream);
}

galore_status_t galore_q8_dequantize(const uint8_t* codes, const float* absmax, int64_t rows, int64_t cols,
                                     int32_t is_signed, int32_t tile_rows, int32_t tile_cols, float* out, void* stream) {
  if (rows < 0 || cols < 0 || (rows > 0 && cols > 0 && (!codes || !absmax || !out))) return GALORE_ERR_INVALID_ARG;
  return launch_q8_dequantize(codes, cols, absmax, rows, cols, is_signed, tile_rows, tile_cols, out, cols, (cudaStream_t)stream);
}

const char* galore_status_string(galore_status_t s) {
  switch (s) {
    case GALORE_OK: return "ok";
    case GALORE_WARN_NOT_CONVERGED: return "refresh reached its iteration cap before the stated convergence";
    case GALORE_ERR_INVALID_ARG: return "invalid argument";
    case GALORE_ERR_SHAPE: return "invalid shape or rank";
    case GALORE_ERR_ALIGNMENT: return "pointer or leading dimension not aligned for this path";
    case GALORE_ERR_BUFFER_TOO_SMALL: return "buffer too small";
    case GALORE_ERR_CUDA: return "CUDA call failed";
    case GALORE_ERR_STATE: return "layer state does not allow this call";
    case GALORE_ERR_NONFINITE: return "non-finite values";
    case GALORE_ERR_TIMEOUT: return "a bounded device wait ran out";
    case GALORE_ERR_UNIMPLEMENTED: return "not implemented for this configuration";
  }
  return "unknown status";
}

galore_status_t galore_abi_sizes(size_t* config_bytes, size_t* refresh_info_bytes) {
  if (config_bytes) *config_bytes = sizeof(galore_config_t);
  if (refresh_info_bytes) *refresh_info_bytes = sizeof(galore_refresh_info_t);
  return GALORE_OK;
}

const char* galore_last_cuda_error(void) { return t_last_error.c_str(); }

int64_t galore_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

galore_status_t galore_profile_enable(int32_t on) {
  g_profile.store(on ? 1 : 0);
  return GALORE_OK;
}

galore_status_t galore_profile_read(double* ms3, int64_t* count3) {
  if (!ms3 || !count3) return GALORE_ERR_INVALID_ARG;
  std::vector<PhaseEvent> evs;
  {
    std::lock_guard<std::mutex> lock(g_profile_mutex);
    evs.swap(g_phase_events);
  }
  galore_status_t rc = GALORE_OK;
  for (PhaseEvent& e : evs) {
    float ms = 0.f;
    cudaError_t err = cudaEventSynchronize(e.b);
    if (err == cudaSuccess) err = cudaEventElapsedTime(&ms, e.a, e.b);
    if (err != cudaSuccess) {
      note_cuda_error(err, "profile event");
      rc = GALORE_ERR_CUDA;
    } else if (e.phase >= 0 && e.phase < 3) {
      ms3[e.phase] += ms;
      count3[e.phase] += 1;
    }
    cudaEventDestroy(e.a);
    cudaEventDestroy(e.b);
  }
  return rc;
}

}  // extern "C"
