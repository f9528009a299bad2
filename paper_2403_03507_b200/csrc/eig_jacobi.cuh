// Symmetric eigen-decomposition by block one-sided Jacobi (the small dense problem inside the
// Rayleigh-Ritz step of the projector refresh, Eq. 12-13): declarations.
#pragma once

#include "common.cuh"

namespace galore {

// bytes of scratch jacobi_eigh needs for a b x b problem
size_t jacobi_scratch_bytes(int b);

// X: b x b row-major, on entry a symmetric positive semi-definite matrix H, on exit Theta V^T
//    (row i = eigenvalue_i x eigenvector_i^T, in no particular order).
// Vt: optional b x b matrix that receives the same row rotations (pass the identity to obtain
//    the eigenvectors as its rows; needed only when eigenvalues near zero matter).
// counter: one device int used to count rotations per sweep.
// Synchronises the stream once per sweep.  sweeps_out receives the number of sweeps run.
// slots: optional list of workspace slots; every pointer argument then names slot 0's copy and the
// same problem is solved in each listed slot, all slots in one launch per kernel (a slot drops out
// once it has converged); sweeps_out then has one entry per listed slot.
galore_status_t jacobi_eigh(double* X, double* Vt, int b, void* scratch, int* counter, double tol, int max_sweeps,
                            int* sweeps_out, cudaStream_t st, const SlotList* slots = nullptr);

}  // namespace galore
