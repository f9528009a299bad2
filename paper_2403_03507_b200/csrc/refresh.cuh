// Projector refresh (Eq. 12-13 by block subspace iteration): declarations.
#pragma once

#include "common.cuh"

namespace galore {

struct RefreshProblem {
  const void* G;        // m x n, row-major
  int32_t g_dtype;
  int64_t ldg;
  int64_t m, n;
  bool left;            // true: P = leading left singular vectors (m x r); false: right (n x r)
  int rank;
  int block;            // columns iterated, rank <= block <= min(m, n)
  void* P;              // output, rows x rank row-major in p_dtype
  int32_t p_dtype;
  uint64_t seed;
  double tol;
  int max_iters;
  int first_iters;      // power steps before the first Rayleigh-Ritz
  bool use_tensor;      // power steps on the tensor cores when G is bf16 and TMA-addressable
  int warm_iters;       // > 0: start from the projector already stored in P (its r columns plus random ones)
                        // and run this many power steps before the first Rayleigh-Ritz pass; 0: random start
};

// d = rows of the projector, L = the other dimension of G
size_t refresh_workspace_bytes(int64_t d, int64_t L, int r, int b);

// Where the last refresh through `workspace` left its projector before rounding to the stored
// dtype: rows x rank doubles, row-major.  Valid until the workspace is written again.
const double* refresh_unrounded_projector(void* workspace, int64_t d, int64_t L, int r, int b);

// Synchronises the stream (reads Ritz values back to decide on convergence).
galore_status_t refresh_projector(const RefreshProblem& pr, void* workspace, int32_t* status,
                                  galore_refresh_info_t* info, cudaStream_t st);

// The same refresh for `count` (<= kMaxSlots) problems of one shape, rank, block and dtype at once:
// problem i works in the i-th slot of `workspace` (slots of slot_bytes = refresh_workspace_bytes()
// each) and latches device conditions in status[i].  Each projector is what refresh_projector
// would produce for that problem alone; the serial parts of the method run for all problems in one
// launch per kernel.  infos: nullptr or `count` records (phase times are the group's, divided by
// count; the a-posteriori residual is computed only when the record is wanted).
galore_status_t refresh_projector_group(const RefreshProblem* prs, int count, void* workspace, size_t slot_bytes,
                                        int32_t* const* status, galore_refresh_info_t* infos, cudaStream_t st);

}  // namespace galore
