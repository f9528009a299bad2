/*
 * galore.h -- C ABI of the B200-native GaLore-Adam optimizer step.
 *
 * Implements, per 2-D weight W (m x n) with gradient G, one iteration of
 * "Adam with GaLore" (arXiv 2403.03507, Algorithm 1):
 *
 *   refresh (every T steps)  P <- r leading left singular vectors of G      (Eq. 12-13)
 *   project                  R <- P^T G           (m <= n, "left")          (Algorithm 1)
 *                            R <- G Q             (m >  n, "right")         (Sec. 4.2)
 *   Adam on R                M <- b1 M + (1-b1) R ; V <- b2 V + (1-b2) R*R
 *                            N <- [M/(1-b1^t)] / (sqrt(V/(1-b2^t)) + eps)   (Eq. 15)
 *   project back and apply   W <- W - lr * alpha * P N   (right: N Q^T)     (Algorithm 1)
 *
 * Conventions
 *   - All matrix arguments are DEVICE pointers to row-major storage with a
 *     leading dimension given in ELEMENTS, unless an argument says "host".
 *   - The caller passes the gradient (not its negative) and the update is
 *     subtracted.
 *   - Timeline tools see NVTX ranges named galore.project, galore.adam, galore.back_project and
 *     galore.refresh (with .steps and .rayleigh_ritz inside) on the calling thread.
 *   - The library allocates no device memory: the optimizer state and a
 *     scratch workspace are caller-allocated device buffers whose sizes come
 *     from galore_query_bytes() and which must outlive the handle.  A
 *     workspace may be shared by several layers that are never stepped
 *     concurrently.
 *   - A handle is used from one stream at a time.  Calls enqueue work on the
 *     given stream (a cudaStream_t passed as void*; NULL = default stream) and
 *     return without synchronising, except where stated.
 *   - Work of different handles is meant to be queued on ONE stream per
 *     device (the list entry points add internal streams of their own, joined
 *     by events).  Tensor-core launches given on different streams are chained
 *     by the library with events, one after another in the order of the calls:
 *     each needs a whole SM's tensor memory and shared memory, so they would
 *     not overlap anyway, and runs that kept several streams of them in flight
 *     stalled on the test machines for a reason that was not found.
 *   - Every entry point returns a galore_status_t: 0 ok, > 0 warning, < 0
 *     error.  Nothing throws or aborts across this boundary.  Conditions
 *     detected on the device (non-finite values, a bounded wait that ran out)
 *     are latched in a status word read by galore_device_status().
 */
#ifndef GALORE_H_
#define GALORE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct galore_layer galore_layer_t; /* opaque, host memory, library-owned */

typedef enum {
  GALORE_OK = 0,
  GALORE_WARN_NOT_CONVERGED = 1, /* refresh stopped at its iteration cap */
  GALORE_ERR_INVALID_ARG = -1,
  GALORE_ERR_SHAPE = -2,         /* rank outside [1, min(m, n)], non-positive sizes */
  GALORE_ERR_ALIGNMENT = -3,     /* pointer or leading dimension not usable by the requested path */
  GALORE_ERR_BUFFER_TOO_SMALL = -4,
  GALORE_ERR_CUDA = -5,          /* a CUDA runtime/driver call failed; see galore_last_cuda_error() */
  GALORE_ERR_STATE = -6,         /* e.g. a step without a projector when auto_refresh is off */
  GALORE_ERR_NONFINITE = -7,     /* galore_check_device: a non-finite projected gradient was seen */
  GALORE_ERR_TIMEOUT = -8,       /* galore_check_device: a bounded device-side wait ran out */
  GALORE_ERR_UNIMPLEMENTED = -9
} galore_status_t;

typedef enum { GALORE_SIDE_AUTO = 0, GALORE_SIDE_LEFT = 1, GALORE_SIDE_RIGHT = 2 } galore_side_t;
typedef enum { GALORE_F32 = 0, GALORE_BF16 = 1 } galore_dtype_t;
/* How the inner optimizer's statistics are kept.  F32 and Q8_BLOCK are Adam's two moments (Algorithm 1;
 * Sec. 4.3 for the 8-bit form).  ADAFACTOR swaps the inner optimizer (Sec. "GaLore with memory-efficient
 * optimizers": Adafactor with first-order statistics; the paper prints no formulas, the update is Shazeer
 * and Stern's): an fp32 first moment of R's shape plus one fp32 value per row and per column of R for the
 * factored second moment, decay 1 - t^-0.8, eps_1 = 1e-30, update clipping at 1, beta1 as the momentum,
 * the learning rate applied in the weight update as for Adam; beta2 and eps are not used. */
typedef enum { GALORE_STATE_F32 = 0, GALORE_STATE_Q8_BLOCK = 1, GALORE_STATE_ADAFACTOR = 2 } galore_state_fmt_t;
/* which kernels carry the two projections */
typedef enum {
  GALORE_PATH_AUTO = 0,   /* tensor cores when dtypes/alignment allow, else the fp32 path */
  GALORE_PATH_FP32 = 1,   /* fp32 FMA kernels: any dtype, any leading dimension */
  GALORE_PATH_TENSOR = 2  /* tcgen05 kernels; init fails with GALORE_ERR_ALIGNMENT/UNIMPLEMENTED if not eligible */
} galore_path_t;

typedef enum { GALORE_ADAM_AUTO = 0, GALORE_ADAM_IN_PROJECTION = 1, GALORE_ADAM_OWN_KERNEL = 2 } galore_adam_place_t;

/* Bits of the device status word. */
enum {
  GALORE_DEV_NONFINITE = 1,     /* a non-finite projected gradient was seen */
  GALORE_DEV_WAIT_EXPIRED = 2,  /* a bounded device-side wait ran out */
  GALORE_DEV_CHOLESKY = 8       /* a Gram matrix in the refresh was not positive definite */
};

/* Hyper-parameters of Algorithm 1 (rank r, scale alpha, refresh gap T, Adam's
 * beta1/beta2/eps; the step size is a per-call argument because it follows a
 * schedule) and the storage choices.  Zero-initialise, then fill. */
typedef struct {
  int64_t m, n;            /* W and G are m x n */
  int32_t rank;            /* r, 1 <= r <= min(m, n) */
  float alpha;             /* scale factor, not divided by r (Sec. 4.4) */
  int32_t refresh_gap;     /* T >= 1 */
  double beta1, beta2, eps; /* Adam; doubles so that 1 - beta is formed from the exact decimal the caller means */
  int32_t side;            /* galore_side_t; AUTO = left iff m <= n (Sec. 4.2) */
  int32_t w_dtype;         /* galore_dtype_t of W */
  int32_t g_dtype;         /* galore_dtype_t of G */
  int32_t p_dtype;         /* galore_dtype_t the projector is stored in */
  int32_t state_fmt;       /* galore_state_fmt_t of M, V */
  int32_t q_block;         /* elements per quantisation block: 256, 512, 1024 or 2048 (0 = 2048); a block is a
                              tile of q_block / 64 consecutive rows x 64 consecutive columns of the state matrix */
  int32_t auto_refresh;    /* 1: galore_step refreshes P when (completed steps) mod T == 0 */
  int32_t path;            /* galore_path_t */
  /* refresh: block subspace iteration on a block of rank + refresh_oversample
   * columns (clipped to min(m, n); 0 = default: max(256, rank / 4) on the
   * tensor path, rank more columns elsewhere; negative = none),
   * stopped when the predicted subspace error falls below refresh_tol or
   * after refresh_max_iters power iterations.  The prediction is
   * (theta_b / theta_r)^iterations for plain power steps; blocks that converge
   * slowly finish with pairs of steps that apply the degree-2 Chebyshev
   * polynomial of the operator over [0, theta_b], each pair counted with the
   * polynomial's value at theta_r.  0 = defaults (1e-4, 96). */
  float refresh_tol;
  int32_t refresh_max_iters;
  int32_t refresh_oversample;
  uint64_t seed;           /* start block of the subspace iteration */
  /* GaLore-AdamW: decoupled weight decay lambda >= 0 (0 = plain Adam).  The paper names AdamW as a
   * supported optimizer without equations; the reading taken is Loshchilov & Hutter's:
   * W <- W (1 - lr lambda) - lr alpha P N, the decay on the full-rank weight with the plain lr. */
  float weight_decay;
  /* Where Adam on R runs when the projection's K is not sliced (galore_adam_place_t): AUTO lets the
   * library choose per state format; IN_PROJECTION runs it in the projection kernel's epilogue (R is
   * never stored); OWN_KERNEL always uses the stand-alone Adam kernel after the projection. */
  int32_t adam_place;
  /* Warm-started refresh (the subspace of consecutive gradients changes slowly, Sec. 4.1): > 0 makes
   * every refresh of a layer that already has a projector start from that projector (plus random
   * columns for the oversampling) and run this many power steps before its Rayleigh-Ritz pass.  The
   * result is then judged by its own residual: residual over spectral gap bounds the angle to the
   * exact subspace; within 10 x refresh_tol the refresh ends there, otherwise it continues like a
   * cold one (as it does at once when the Rayleigh quotients after those steps show no gap behind
   * the block).  0 = always start from a random block. */
  int32_t refresh_warm_iters;
  int32_t reserved[5];
} galore_config_t;

/* Result of one refresh (host struct, filled after the refresh's stream work has completed). */
typedef struct {
  int32_t iterations;        /* power iterations run */
  int32_t block;             /* columns iterated (rank + oversample, clipped) */
  int32_t jacobi_sweeps;     /* sweeps of the last Rayleigh-Ritz eigen-solve */
  int32_t converged;         /* 1 when the stated criterion was met */
  double predicted_error;    /* (theta_b / theta_r)^iterations */
  double residual;           /* || (G G^T) P - P Theta ||_F / (theta_1 sqrt(r)) for the kept Ritz pairs */
  double sigma_r;            /* sqrt of the r-th Ritz value */
  double sigma_next;         /* sqrt of the (r+1)-th Ritz value, 0 if block == rank */
  double sigma_1;
  double ms_total;           /* wall time of the refresh, with its parts: */
  double ms_power;           /* power steps and their orthonormalisations */
  double ms_ritz;            /* final orthonormalisation, fp64 products, sorting, P = Y S (without the eigen-solve) */
  double ms_jacobi;          /* Jacobi eigen-solves */
  int32_t ritz_passes;       /* Rayleigh-Ritz passes (each ends a run of power steps) */
  int32_t reserved;
} galore_refresh_info_t;

/* Sizes of the two caller-allocated device buffers for one layer.
 * state_bytes covers P (rows x r, p_dtype), M and V (shape of R: r x n left,
 * m x r right; fp32, or uint8 codes plus one fp32 absmax per block) -- the
 * paper's  m r + 2 n r  elements for m <= n (Sec. 4.2), with the rows of M
 * and V padded to 32 bytes.  Both buffers must be
 * 256-byte aligned.  Host-only; touches no device. */
galore_status_t galore_query_bytes(const galore_config_t* cfg, size_t* state_bytes, size_t* workspace_bytes);

/* Creates a layer: validates cfg, lays out state_buf, zeroes M and V (stream
 * work), sets the step counter to 0.  The projector is undefined until the
 * first refresh or galore_set_projector().  *out is host memory owned by the
 * library until galore_free(). */
galore_status_t galore_init_layer(const galore_config_t* cfg, void* state_buf, size_t state_bytes,
                                  void* workspace, size_t workspace_bytes, void* stream,
                                  galore_layer_t** out);

/* One iteration of Algorithm 1 on W (read and written in place) with gradient G
 * (read only).  With auto_refresh the projector is refreshed from G first when
 * the number of completed steps is a multiple of T (so the first step
 * refreshes); a refresh synchronises the stream.  Increments the step counter. */
galore_status_t galore_step(galore_layer_t* layer, void* W, int64_t ldw, const void* G, int64_t ldg,
                            float lr, void* stream);

/* Same step with W and G in HOST memory (pinned for asynchronous copies):
 * copies both into the caller's device staging buffers (same dtype, packed,
 * leading dimension n), steps, copies W back, all on `stream`. */
galore_status_t galore_step_host(galore_layer_t* layer, void* W_host, const void* G_host,
                                 void* W_dev_staging, void* G_dev_staging, float lr, void* stream);

/* Steps `count` layers on one stream, layer i with W[i], G[i] (device pointers; host arrays of
 * pointers and leading dimensions).  Same results as calling galore_step on each layer up to the
 * order of floating-point sums (with several layers in flight the K dimension of the projection is
 * not sliced), but the layers are stepped in groups of up to 32 of one kind (tensor-core path, or
 * fp32 path with the same side and dtypes): one grouped launch for all their projections, one for
 * the inner optimizer (none when Adam runs in the projection's epilogue), one for all their
 * back-projections, so that small matrices do not each pay a kernel's ramp-up and the last wave of
 * one matrix overlaps the first of the next.  batch_ws is a caller-allocated, 256-byte aligned
 * device buffer that holds the intermediates (R and N) of the layers of one group; the groups run
 * one after another on `stream` and use it in turn.  galore_batch_query_bytes gives the size that
 * lets the groups be as large as the kernels allow.  A smaller buffer only makes the groups
 * smaller; a layer that does not fit at all is stepped by galore_step with its own workspace.  The
 * layers' own workspaces may be shared with each other. */
galore_status_t galore_batch_query_bytes(galore_layer_t* const* layers, int32_t count, size_t* batch_ws_bytes);
galore_status_t galore_step_batch(galore_layer_t* const* layers, void* const* W, const int64_t* ldw,
                                  const void* const* G, const int64_t* ldg, int32_t count, float lr,
                                  void* batch_ws, size_t batch_ws_bytes, void* stream);

/* The step for a list of layers whose W and G live in pinned host memory (an optimizer state
 * kept on the GPU for weights that are not).  (The paper has no counterpart: Algorithm 1 does not
 * say where W lives.)  Layer i's W and G (row-major, rows of n elements, no padding) are copied into one
 * of `slots` parts of `staging` (device memory, 256-byte aligned, galore_host_batch_query_bytes()),
 * stepped there, and W is copied back.  Copies in, steps and copies out run on three streams (the
 * steps on `stream`), so that both directions of the host link and the steps overlap across layers;
 * 3 slots keep all three busy.  Asynchronous: work queued on `stream` after the call runs after
 * the last copy out.  The host arrays must stay valid and untouched until then. */
galore_status_t galore_host_batch_query_bytes(galore_layer_t* const* layers, int32_t count, int32_t slots, size_t* bytes);
galore_status_t galore_step_host_batch(galore_layer_t* const* layers, void* const* W_host, const void* const* G_host,
                                       int32_t count, float lr, void* staging, size_t staging_bytes, int32_t slots,
                                       void* stream);

/* Recomputes the projector as the top-r singular subspace of G (Eq. 12-13) by
 * block subspace iteration with a final Rayleigh-Ritz rotation, so that the
 * stored columns approximate singular vectors in descending order of
 * singular value.  M, V and the step counter are left untouched.
 * Synchronises the stream.  info may be NULL.  Returns
 * GALORE_WARN_NOT_CONVERGED when the iteration cap was reached first. */
galore_status_t galore_refresh_projector(galore_layer_t* layer, const void* G, int64_t ldg, void* stream,
                                         galore_refresh_info_t* info);

/* The same refresh for `count` layers on `stream` (Algorithm 1 refreshes every layer at the same
 * steps), with `workspace` (device memory, 256-byte aligned, at least galore_refresh_query_bytes()
 * of every layer) in place of each layer's own refresh workspace, so that layers which share their
 * workspace can be refreshed through one call.  Neighbours in the list that have the same shape,
 * rank and dtypes are refreshed together, as many at a time (up to 8) as `workspace` holds copies
 * of galore_refresh_query_bytes(): the serial parts of the method (Cholesky panels, the dense
 * eigen-solver) then run for all of them at once.  Every layer receives the projector it would
 * receive from galore_refresh_projector alone.
 * infos: NULL or `count` records (phase times of layers refreshed together are the group's divided
 * by its size).  Stops at the first error; otherwise returns GALORE_WARN_NOT_CONVERGED if any layer
 * reached its iteration cap. */
galore_status_t galore_refresh_query_bytes(const galore_layer_t* layer, size_t* bytes);
galore_status_t galore_refresh_batch(galore_layer_t* const* layers, const void* const* G, const int64_t* ldg,
                                     int32_t count, void* workspace, size_t workspace_bytes, void* stream,
                                     galore_refresh_info_t* infos);

/* Releases the host handle.  Device buffers stay with the caller. */
galore_status_t galore_free(galore_layer_t* layer);

/* A step that needs no workspace from the caller and allocates nothing.  (The paper has no
 * counterpart: this is a convenience of this library.)
 *
 * For callers that cannot hand the library a scratch buffer or let it obtain one: plug-ins of a
 * host framework that owns all device memory through its own pool and bans cudaMalloc, call sites
 * where the device-wide synchronisation of cudaMalloc/cudaFree is not acceptable, threads that
 * must stay away from the allocator.  The step's intermediates (split-K partial sums of R and the
 * normalised update N) live in an array of GALORE_STATIC_SCRATCH_BYTES bytes that is part of the
 * library image; every GPU that loads the library holds that much memory until the process exits.
 *
 * One fp32 iteration of Algorithm 1 on explicit arrays, all device memory, row-major:
 *   P  projector, rows x rank packed (rows = m for the left side, n for the right), read only
 *   M, V  moments, shape of R (rank x n left, m x rank right) packed, updated in place
 *   W  m x n with leading dimension ldw, updated in place;  G  m x n with ldg, read only
 *   completed_steps  k of Algorithm 1 before this call (bias correction uses k + 1)
 *   side  galore_side_t (AUTO: left iff m <= n)
 *   device_flags  optional host pointer; when non-NULL the call waits for the stream and stores
 *                 the GALORE_DEV_* bits the kernels of THIS call latched, otherwise it returns
 *                 without waiting; either way the bits are also kept for galore_static_status()
 * No refresh is done here: the caller supplies P.
 *
 * Limits and rules
 *   - 256 + 4 * (splits + 1) * (elements of R) bytes, each part rounded up to 256, must fit in the
 *     array (splits <= 16 is chosen by the library); larger layers are refused with
 *     GALORE_ERR_BUFFER_TOO_SMALL and nothing is launched.
 *   - The first call on each device looks up the array's device address (with that device
 *     current).  Make that first call outside of any stream capture.
 *   - `stream` must belong to the current device (checked: GALORE_ERR_INVALID_ARG otherwise); the
 *     array that is used is the current device's.
 *   - All calls on a device share the array, and it keeps the previous call's contents.  The call
 *     clears the status word it needs at zero; everything else it reads it has written first.
 *     Calls whose GPU work can overlap (two streams, two threads) race on the array: serialise
 *     them.
 *   - Calls no cudaMalloc, cudaFree or other allocating routine. */
#define GALORE_STATIC_SCRATCH_BYTES (16u * 1024u * 1024u)
galore_status_t galore_step_static(int64_t m, int64_t n, int32_t rank, int32_t side, float alpha, double beta1,
                                   double beta2, double eps, int64_t completed_steps, const float* P, float* M,
                                   float* V, float* W, int64_t ldw, const float* G, int64_t ldg, float lr,
                                   int32_t* device_flags, void* stream);
/* GALORE_DEV_* bits latched by every galore_step_static call on the current device since the last
 * call of this function (they accumulate across calls, so the asynchronous form loses nothing).
 * Synchronises `stream`, returns the bits in *flags and clears them. */
galore_status_t galore_static_status(int32_t* flags, void* stream);

/* ---- accessors (tests, checkpoint/resume) -------------------------------- */

/* Projector as fp32, rows x r row-major packed (rows = m left, n right), device memory. */
galore_status_t galore_get_projector(galore_layer_t* layer, float* dst, size_t dst_bytes, void* stream);
/* Diagnostic: the projector of the last galore_refresh_projector() (or refresh inside galore_step) of
 * this layer as it was before rounding to p_dtype, rows x rank doubles (device memory).  It is read
 * from the layer's workspace: valid only until that workspace is used again (by this or by another
 * layer that shares it); GALORE_ERR_STATE if the layer has not been refreshed through its own
 * workspace.  The 1e-3 rad bound of the refresh is a statement about this matrix. */
galore_status_t galore_get_unrounded_projector(galore_layer_t* layer, double* dst, size_t dst_bytes, void* stream);
galore_status_t galore_set_projector(galore_layer_t* layer, const float* src, size_t src_bytes, void* stream);
/* Stored (uncorrected) Adam moments as fp32, shape of R row-major packed, device memory (8-bit states are
 * dequantised; GALORE_ERR_STATE for Adafactor, whose second moment is factored). */
galore_status_t galore_get_moments(galore_layer_t* layer, float* M, float* V, size_t bytes_each, void* stream);
/* Adafactor state (GALORE_STATE_ADAFACTOR, else GALORE_ERR_STATE): the first moment (fp32, shape of R, row-major
 * packed), the running row means (rows of R entries) and column means (columns of R entries) of R^2 + eps_1;
 * device memory. */
galore_status_t galore_get_adafactor_state(galore_layer_t* layer, float* M, float* v_row, float* v_col, void* stream);
/* Raw 8-bit state: codes (uint8, shape of R, packed) and per-block absmax (fp32, tile (I, J) of the
 * state at I * ceil(cols / 64) + J); device memory. */
galore_status_t galore_get_q8_state(galore_layer_t* layer, uint8_t* M_codes, float* M_absmax,
                                    uint8_t* V_codes, float* V_absmax, void* stream);
/* Completed steps k. */
galore_status_t galore_get_step_count(const galore_layer_t* layer, int64_t* k);
galore_status_t galore_set_step_count(galore_layer_t* layer, int64_t k);
/* Resolved side (galore_side_t), whether the tensor-core path is in use, and the state shape. */
galore_status_t galore_layer_info(const galore_layer_t* layer, int32_t* side, int32_t* uses_tensor_path,
                                  int64_t* state_rows, int64_t* state_cols);
/* Synchronises `stream`, returns the device status bits and clears them. */
galore_status_t galore_device_status(galore_layer_t* layer, int32_t* flags, void* stream);
/* The same read-and-clear as a status: GALORE_ERR_TIMEOUT if a bounded wait ran out, else
 * GALORE_ERR_NONFINITE for a non-finite projected gradient, else GALORE_ERR_STATE for a Cholesky
 * breakdown in the refresh, else GALORE_OK. */
galore_status_t galore_check_device(galore_layer_t* layer, void* stream);

/* Checkpoint and resume of one layer: everything Algorithm 1 carries from one iteration to the
 * next -- the projector P, the moments M and V (fp32, or codes and absmax) and the number of
 * completed steps -- as one block of HOST memory of galore_export_bytes() bytes (a small header,
 * then the state buffer as it is laid out on the device).  galore_import_state restores it into a
 * layer created with the same shape, rank, side, projector dtype, state format and block size
 * (GALORE_ERR_STATE otherwise; GALORE_ERR_INVALID_ARG if the block is not an export of this
 * library).  A run that exports, imports into a fresh layer and goes on is bit-identical to one
 * that never stopped.  Both calls synchronise `stream`. */
galore_status_t galore_export_bytes(const galore_layer_t* layer, size_t* bytes);
galore_status_t galore_export_state(galore_layer_t* layer, void* dst_host, size_t bytes, void* stream);
galore_status_t galore_import_state(galore_layer_t* layer, const void* src_host, size_t bytes, void* stream);

/* ---- 8-bit block-wise state format (Sec. 4.3 names 8-bit Adam states; the
 *      format is this library's) ------------------------------------------- */

/* The 256 fp32 code values, ascending, into host memory. is_signed != 0: the
 * first-moment code on [-1, 1]; 0: the second-moment code on [0, 1]. */
galore_status_t galore_q8_codebook(int32_t is_signed, float* out256_host);
/* x (fp32, rows x cols packed, device) -> codes (uint8, rows x cols packed) and absmax (fp32, one per
 * quantisation block).  The blocks are tiles of tile_rows x tile_cols elements of the matrix, tile
 * (I, J) at absmax[I * ceil(cols / tile_cols) + J]; tiles on the lower and right edges are cut off
 * at the border.  A flat array with blocks of b consecutive elements is rows = 1, tile 1 x b.
 * code = nearest code value to fp32(x / absmax), ties to the larger index; absmax = 0 stores the
 * code of 0.  The moments of a layer use tiles of (q_block / 64) x 64 of the state matrix. */
galore_status_t galore_q8_quantize(const float* x, int64_t rows, int64_t cols, int32_t is_signed, int32_t tile_rows,
                                   int32_t tile_cols, uint8_t* codes, float* absmax, void* stream);
galore_status_t galore_q8_dequantize(const uint8_t* codes, const float* absmax, int64_t rows, int64_t cols,
                                     int32_t is_signed, int32_t tile_rows, int32_t tile_cols, float* out, void* stream);

/* ---- diagnostics ---------------------------------------------------------- */
/* sizeof(galore_config_t) and sizeof(galore_refresh_info_t) as compiled, for bindings to check their marshalling. */
galore_status_t galore_abi_sizes(size_t* config_bytes, size_t* refresh_info_bytes);
const char* galore_status_string(galore_status_t s);
/* Text of the last CUDA error seen by this thread's calls into the library ("" if none). */
const char* galore_last_cuda_error(void);
/* Number of kernel launches issued by the library in this process (all layers). */
int64_t galore_launch_count(void);
/* Phase timing for benchmarks.  While enabled (process-wide), galore_step brackets its three
 * phases with CUDA events on the step's stream: 0 projection, 1 Adam on R, 2 back-projection + weight
 * write.  galore_profile_read synchronises on the recorded events, adds the elapsed milliseconds and
 * the number of brackets per phase into ms3 / count3 (host arrays of 3) and forgets the events. */
galore_status_t galore_profile_enable(int32_t on);
galore_status_t galore_profile_read(double* ms3, int64_t* count3);

#ifdef __cplusplus
}
#endif
#endif /* GALORE_H_ */
