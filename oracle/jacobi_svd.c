/*
 * TEST INFRASTRUCTURE ONLY -- part of the CPU oracle, never linked into or
 * called by the CUDA library.
 *
 * One-sided (Hestenes) Jacobi singular value decomposition in fp64, no LAPACK
 * and no BLAS.  It provides the exact "U, S, V <- SVD(G)" that Algorithm 1 of
 * the GaLore paper asks for when the projector is refreshed, and the
 * definition of Eq. 12-13 (P = the r leading left singular vectors,
 * Q = the r leading right singular vectors).
 *
 * Method.  The input A is d x L, row-major, d <= L expected (the caller passes
 * G when m <= n and G^T otherwise).  A working copy X starts as A, and a d x d
 * matrix Ut starts as the identity.  A plane rotation of rows (p, q) is chosen
 * so that the two rotated rows of X become orthogonal; the same rotation is
 * applied to rows (p, q) of Ut.  Sweeping over all pairs until no pair needs
 * rotating leaves X = Ut * A with mutually orthogonal rows, hence
 *      A = Ut^T * X,   sigma_i = ||X[i,:]||,   u_i = Ut[i,:],   v_i = X[i,:]/sigma_i.
 * Pairs are visited in round-robin ("tournament") order: each of the d-1 (d
 * even) rounds holds d/2 disjoint pairs, which touch disjoint rows and can
 * therefore run on separate threads without changing any result.
 *
 * Outputs are sorted by descending singular value.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* returns 1 when a rotation was applied */
static int rotate_pair(double *X, double *Ut, int64_t d, int64_t L, int64_t p, int64_t q, double tol) {
    double *xp = X + p * L, *xq = X + q * L;
    double app = 0.0, aqq = 0.0, apq = 0.0;
    for (int64_t j = 0; j < L; ++j) {
        app += xp[j] * xp[j];
        aqq += xq[j] * xq[j];
        apq += xp[j] * xq[j];
    }
    if (apq == 0.0) return 0;
    if (fabs(apq) <= tol * sqrt(app * aqq)) return 0;
    /* symmetric 2x2 Schur decomposition of [[app, apq], [apq, aqq]] */
    double zeta = (aqq - app) / (2.0 * apq);
    double t = (zeta >= 0.0 ? 1.0 : -1.0) / (fabs(zeta) + sqrt(1.0 + zeta * zeta));
    double c = 1.0 / sqrt(1.0 + t * t);
    double s = c * t;
    for (int64_t j = 0; j < L; ++j) {
        double a = xp[j], b = xq[j];
        xp[j] = c * a - s * b;
        xq[j] = s * a + c * b;
    }
    double *up = Ut + p * d, *uq = Ut + q * d;
    for (int64_t j = 0; j < d; ++j) {
        double a = up[j], b = uq[j];
        up[j] = c * a - s * b;
        uq[j] = s * a + c * b;
    }
    return 1;
}

typedef struct { double s; int64_t i; } sv_t;
static int cmp_desc(const void *a, const void *b) {
    double x = ((const sv_t *)a)->s, y = ((const sv_t *)b)->s;
    if (x > y) return -1;
    if (x < y) return 1;
    int64_t i = ((const sv_t *)a)->i, j = ((const sv_t *)b)->i;
    return (i > j) - (i < j);
}

/*
 * A      : d x L row-major input (not modified)
 * U      : d x d row-major output, column i = i-th left singular vector
 * S      : d singular values, descending
 * Vt     : d x L row-major output, row i = i-th right singular vector (may be NULL)
 * returns the number of sweeps used, or -1 on allocation failure,
 *         or -(2 + sweeps) when max_sweeps ran out before convergence.
 */
int jacobi_svd_rows(const double *A, int64_t d, int64_t L, double *U, double *S, double *Vt,
                    double tol, int max_sweeps, int num_threads) {
    double *X = (double *)malloc(sizeof(double) * (size_t)d * (size_t)L);
    double *Ut = (double *)calloc((size_t)d * (size_t)d, sizeof(double));
    int64_t np = d + (d & 1);                 /* players, padded to even (index d = bye) */
    int64_t *ring = (int64_t *)malloc(sizeof(int64_t) * (size_t)(np > 0 ? np : 1));
    sv_t *order = (sv_t *)malloc(sizeof(sv_t) * (size_t)(d > 0 ? d : 1));
    if (!X || !Ut || !ring || !order) { free(X); free(Ut); free(ring); free(order); return -1; }
    memcpy(X, A, sizeof(double) * (size_t)d * (size_t)L);
    for (int64_t i = 0; i < d; ++i) Ut[i * d + i] = 1.0;
#ifdef _OPENMP
    if (num_threads > 0) omp_set_num_threads(num_threads);
#else
    (void)num_threads;
#endif
    int sweeps = 0, converged = 0;
    while (sweeps < max_sweeps && !converged) {
        int64_t rotations = 0;
        for (int64_t i = 0; i < np; ++i) ring[i] = i;
        for (int64_t round = 0; round < np - 1; ++round) {
            int64_t half = np / 2;
            int64_t local = 0;
#pragma omp parallel for schedule(dynamic, 4) reduction(+ : local)
            for (int64_t k = 0; k < half; ++k) {
                int64_t p = ring[k], q = ring[np - 1 - k];
                if (p >= d || q >= d) continue;
                if (p > q) { int64_t tmp = p; p = q; q = tmp; }
                local += rotate_pair(X, Ut, d, L, p, q, tol);
            }
            rotations += local;
            /* rotate all players but the first one place round the ring */
            int64_t last = ring[np - 1];
            for (int64_t i = np - 1; i > 1; --i) ring[i] = ring[i - 1];
            if (np > 1) ring[1] = last;
        }
        ++sweeps;
        if (rotations == 0) converged = 1;
    }
    for (int64_t i = 0; i < d; ++i) {
        double nrm = 0.0;
        for (int64_t j = 0; j < L; ++j) nrm += X[i * L + j] * X[i * L + j];
        order[i].s = sqrt(nrm);
        order[i].i = i;
    }
    qsort(order, (size_t)d, sizeof(sv_t), cmp_desc);
    for (int64_t k = 0; k < d; ++k) {
        int64_t src = order[k].i;
        S[k] = order[k].s;
        for (int64_t j = 0; j < d; ++j) U[j * d + k] = Ut[src * d + j];
        if (Vt) {
            double inv = order[k].s > 0.0 ? 1.0 / order[k].s : 0.0;
            for (int64_t j = 0; j < L; ++j) Vt[k * L + j] = X[src * L + j] * inv;
        }
    }
    free(X); free(Ut); free(ring); free(order);
    return converged ? sweeps : -(2 + sweeps);
}
