"""CPU oracle for the GaLore-Adam optimizer step.  TEST INFRASTRUCTURE ONLY.

This module is the slow, plain fp64 statement of what the method computes.  It
exists so that the CUDA library can be checked against it; nothing in the
product path imports it, and it imports nothing from the CUDA package.  Only
the tests, the smoke check and the CPU-baseline leg of the benchmark use it.

What it follows (GaLore, arXiv 2403.03507):
  * Algorithm 1 ("Adam with GaLore") for the step, read as follows where the
    text leaves a choice:
      - the moments M, V have the shape of the projected gradient R;
      - the refresh test uses the number k of completed steps (k mod T == 0, so
        the first step refreshes) and the bias correction uses t = k + 1;
      - the bias-corrected moments are temporaries, the stored moments stay
        uncorrected;
      - epsilon is added outside the square root (Eq. 15);
      - the caller passes the gradient (not its negative) and the update is
        subtracted, which is the same trajectory;
      - the moments are kept unchanged across a projector refresh.
  * Sec. 4.2 ("Reducing memory usage of projection matrices") for the side:
    R = P^T G when m <= n, R = G Q otherwise.
  * Eq. 12-13 for the projector: the r leading left (right) singular vectors
    of the current gradient.
  * Sec. 4.3 ("8-bit optimizers") names block-wise 8-bit Adam states without
    giving a format.  The format used here is this project's own and is
    spelled out at `dynamic_code` (the code values) and `state_tile` (which
    elements share an absmax: tiles of q_block / 64 rows x 64 columns of the
    state matrix); it is PARITY UNPINNED against the paper
    (the paper fixes nothing to pin it to) and pinned only by its own
    invariants in the tests.
  * Sec. "GaLore with memory-efficient optimizers" names Adafactor with
    first-order statistics as another inner optimizer and prints no formulas.
    `adafactor_update` is the published Adafactor update (Shazeer & Stern) on
    the compact gradient, the reading of its options stated there; it is
    PARITY UNPINNED against the paper and pinned against an independent
    library implementation of that algorithm, a closed form and brute force.

Storage emulation: arithmetic is always fp64; values are rounded when they are
*stored* (weights to bf16 or fp32, moments to fp32 or to 8-bit codes), because
that is part of what the step computes when the paper's BF16 / 8-bit settings
are used.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SVD_SRC = os.path.join(_HERE, "jacobi_svd.c")
_SVD_LIB = os.path.join(_HERE, "libjacobi_svd.so")
_svd_handle = None


def build_native(force: bool = False) -> str:
    """Compile the Jacobi SVD (plain C, gcc) next to its source."""
    if force or not os.path.exists(_SVD_LIB) or os.path.getmtime(_SVD_LIB) < os.path.getmtime(_SVD_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", _SVD_LIB, _SVD_SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _SVD_LIB


def _svd_lib():
    global _svd_handle
    if _svd_handle is None:
        lib = ctypes.CDLL(build_native())
        lib.jacobi_svd_rows.restype = ctypes.c_int
        lib.jacobi_svd_rows.argtypes = [
            ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_void_p, ctypes.c_double, ctypes.c_int, ctypes.c_int]
        _svd_handle = lib
    return _svd_handle


# --------------------------------------------------------------------------
# Singular value decomposition and the projector (Eq. 12-13)
# --------------------------------------------------------------------------

def jacobi_svd(A, want_vt: bool = True, num_threads: int = 0):
    """Full SVD A = U diag(S) Vt by one-sided Jacobi in fp64 (no LAPACK).

    Returns U (a x k), S (k, descending), Vt (k x b) with k = min(a, b).
    The native routine wants the short dimension as rows, so a tall input is
    decomposed through its transpose (A^T = V S U^T).
    """
    A = np.ascontiguousarray(A, dtype=np.float64)
    a, b = A.shape
    if a > b:
        V, S, Ut = jacobi_svd(A.T, want_vt=True, num_threads=num_threads)
        return np.ascontiguousarray(Ut.T), S, np.ascontiguousarray(V.T)
    U = np.empty((a, a), dtype=np.float64)
    S = np.empty((a,), dtype=np.float64)
    Vt = np.empty((a, b), dtype=np.float64) if want_vt else None
    rc = _svd_lib().jacobi_svd_rows(
        A.ctypes.data, a, b, U.ctypes.data, S.ctypes.data,
        Vt.ctypes.data if want_vt else None, 1e-15, 60, num_threads)
    if rc < 0:
        raise RuntimeError(f"jacobi_svd_rows failed or did not converge (rc={rc})")
    return U, S, Vt


def top_r_projector(G, r: int, side: str, method: str = "jacobi"):
    """Eq. 12-13: P = [u_1..u_r] (side 'left', m x r) or Q = [v_1..v_r] ('right', n x r).

    method 'jacobi' is the oracle's own SVD.  method 'lapack' calls the library
    SVD as a single step; it is for matrices too large for the Jacobi code to
    finish in test time, and the tests check the two against each other.
    Returns (projector, singular values).
    """
    G = np.asarray(G, dtype=np.float64)
    if method == "jacobi":
        U, S, Vt = jacobi_svd(G, want_vt=(side == "right"))
    elif method == "lapack":
        U, S, Vt = np.linalg.svd(G, full_matrices=False)
    else:
        raise ValueError(method)
    if side == "left":
        return np.ascontiguousarray(U[:, :r]), S
    return np.ascontiguousarray(Vt[:r, :].T), S


def largest_principal_angle(P_a, P_b) -> float:
    """Largest principal angle (rad) between the column spans of two orthonormal bases.

    cos of the principal angles are the singular values of P_a^T P_b; the
    largest angle is taken from the sine, sqrt(lambda_max(I - C^T C)), so that
    small angles are resolved (the arccos of a value near 1 is not).
    """
    P_a = np.asarray(P_a, dtype=np.float64)
    P_b = np.asarray(P_b, dtype=np.float64)
    # residual of P_b outside span(P_a); its largest singular value is sin(theta_max)
    resid = P_b - P_a @ (P_a.T @ P_b)
    s = np.linalg.norm(resid, 2)
    return float(np.arcsin(min(1.0, s)))


# --------------------------------------------------------------------------
# Storage rounding
# --------------------------------------------------------------------------

def round_bf16(x):
    """Round fp64 values to the nearest bfloat16 (8 significand bits, ties to even)."""
    x = np.asarray(x, dtype=np.float64)
    mant, expo = np.frexp(x)                      # x = mant * 2**expo, 0.5 <= |mant| < 1
    mant = np.rint(mant * 256.0) / 256.0          # keep 8 significant bits; rint ties to even
    return np.ldexp(mant, expo)


def round_f32(x):
    return np.asarray(x, dtype=np.float64).astype(np.float32).astype(np.float64)


def _store(x, kind: str):
    if kind == "f64":
        return np.asarray(x, dtype=np.float64)
    if kind == "f32":
        return round_f32(x)
    if kind == "bf16":
        return round_bf16(x)
    raise ValueError(kind)


# --------------------------------------------------------------------------
# 8-bit block-wise states (Sec. 4.3 names them; the format below is ours)
# --------------------------------------------------------------------------

def dynamic_code(signed: bool) -> np.ndarray:
    """The 256 fp32 code values, ascending.

    A non-uniform "dynamic" code on [-1, 1] (signed, first moment) or [0, 1]
    (unsigned, second moment): decade e = 0, 1, 2, ... carries 2**f linearly
    spaced magnitudes in (10**-(e+1), 10**-e], with f shrinking by one per
    decade, so resolution follows magnitude.  Magnitude (e, j), j = 0..2**f-1:

        (2**f + 9 (j + 1)) / (2**f * 10**(e + 1))          [one fp64 division]

    unsigned: f = 7 - e, e = 0..7   -> 255 magnitudes, plus 0            = 256
    signed  : f = 6 - e, e = 0..6   -> 127 magnitudes, both signs, plus 0
              and one extra positive value 1e-7                          = 256
    Both contain 0 and 1 exactly (signed also -1).
    """
    top = 7 if not signed else 6
    mags = []
    for e in range(top + 1):
        f = top - e
        for j in range(2 ** f):
            mags.append((2 ** f + 9 * (j + 1)) / (2 ** f * 10 ** (e + 1)))
    mags = sorted(mags)
    if signed:
        vals = [-v for v in reversed(mags)] + [0.0, 1.0 / 10 ** 7] + mags
    else:
        vals = [0.0] + mags
    code = np.array(vals, dtype=np.float64).astype(np.float32)
    assert code.shape == (256,)
    return code


def code_midpoints(code: np.ndarray) -> np.ndarray:
    """fp32 decision thresholds between neighbouring code values."""
    c = code.astype(np.float64)
    return (0.5 * (c[:-1] + c[1:])).astype(np.float32)


def _quantize_one_block(seg, mids, zero_code):
    """One block of fp32 values (any shape) -> (codes of the same shape, fp32 absmax).

    absmax = max |x|;  y = x / absmax in fp32 (IEEE division);  the code is the
    number of thresholds <= y, i.e. the nearest code value with ties going to
    the larger index.  A block whose absmax is 0 stores the code of 0.
    """
    a = np.float32(np.max(np.abs(seg))) if seg.size else np.float32(0)
    if a == 0:
        return np.full(seg.shape, zero_code, dtype=np.uint8), a
    y = (seg / a).astype(np.float32)              # fp32 / fp32 -> IEEE fp32 quotient
    return np.searchsorted(mids, y, side="right").astype(np.uint8), a


def quantize_tiles(X, signed: bool, tile_rows: int, tile_cols: int):
    """fp32 matrix -> (uint8 codes of the same shape, fp32 absmax per tile).

    The quantisation blocks are tiles of `tile_rows` x `tile_cols` elements of
    the matrix, tile (I, J) covering rows [I tile_rows, (I+1) tile_rows) and
    columns [J tile_cols, (J+1) tile_cols); tiles on the lower and right edges
    are cut off at the matrix border.  absmax has one entry per tile, shape
    (ceil(rows / tile_rows), ceil(cols / tile_cols)).
    """
    X32 = np.asarray(X, dtype=np.float32)
    assert X32.ndim == 2
    rows, cols = X32.shape
    code = dynamic_code(signed)
    mids = code_midpoints(code)
    zero_code = int(np.nonzero(code == 0.0)[0][0])
    gr, gc = -(-rows // tile_rows), -(-cols // tile_cols)
    codes = np.empty((rows, cols), dtype=np.uint8)
    absmax = np.zeros((gr, gc), dtype=np.float32)
    for I in range(gr):
        for J in range(gc):
            sl = (slice(I * tile_rows, (I + 1) * tile_rows), slice(J * tile_cols, (J + 1) * tile_cols))
            codes[sl], absmax[I, J] = _quantize_one_block(X32[sl], mids, zero_code)
    return codes, absmax


def dequantize_tiles(codes, absmax, signed: bool, tile_rows: int, tile_cols: int):
    """(codes, absmax per tile) -> fp32 matrix: code value times the tile's absmax, in fp32."""
    codes = np.asarray(codes, dtype=np.uint8)
    rows, cols = codes.shape
    code = dynamic_code(signed)
    am = np.asarray(absmax, dtype=np.float32)
    scale = np.repeat(np.repeat(am, tile_rows, axis=0)[:rows], tile_cols, axis=1)[:, :cols]
    return (code[codes] * scale).astype(np.float32)


def quantize_blockwise(x, signed: bool, block: int = 2048):
    """Flat fp32 array -> (uint8 codes, fp32 absmax per block): blocks are runs of `block`
    consecutive elements, the last one may be shorter (a one-row matrix cut into 1 x block tiles)."""
    x32 = np.asarray(x, dtype=np.float32).reshape(1, -1)
    codes, absmax = quantize_tiles(x32, signed, 1, block)
    return codes.reshape(-1), absmax.reshape(-1)


def dequantize_blockwise(codes, absmax, signed: bool, block: int = 2048):
    """(codes, absmax) -> fp32 values: code value times the block's absmax, in fp32."""
    codes = np.asarray(codes, dtype=np.uint8).reshape(1, -1)
    am = np.asarray(absmax, dtype=np.float32).reshape(1, -1)
    return dequantize_tiles(codes, am, signed, 1, block).reshape(-1)


STATE_TILE_COLS = 64


def state_tile(q_block: int):
    """Shape of the quantisation blocks of the 8-bit moments: q_block elements as a tile of
    q_block / 64 consecutive rows x 64 consecutive columns of the state matrix (2048 -> 32 x 64)."""
    if q_block % STATE_TILE_COLS:
        raise ValueError("q_block must be a multiple of 64")
    return q_block // STATE_TILE_COLS, STATE_TILE_COLS


# --------------------------------------------------------------------------
# Algorithm 1
# --------------------------------------------------------------------------

# ---------------------------------------------------------------------------
# Adafactor as the inner regulariser (Sec. "GaLore with memory-efficient optimizers": Adafactor
# "with first-order statistics"; the paper prints no formulas, so the update is the published one
# of Shazeer & Stern, "Adafactor: Adaptive Learning Rates with Sublinear Memory Cost", Algorithm 4
# with momentum, written for the compact gradient R).  Reading taken here: external learning rate
# (no relative step size, no parameter scaling), decay beta2_t = 1 - t^-0.8, eps_1 = 1e-30, update
# clipping at d = 1, momentum beta1 on the clipped update, and the learning rate applied where
# Algorithm 1 applies it (W <- W - lr alpha P N), not inside the momentum.
# ---------------------------------------------------------------------------
ADAFACTOR_DECAY = 0.8
ADAFACTOR_EPS1 = 1e-30
ADAFACTOR_CLIP = 1.0


def adafactor_update(R, M_prev, v_row, v_col, t, beta1):
    """One Adafactor step on R (rows x cols).  v_row (rows) and v_col (cols) are the running means of
    R^2 + eps_1 along each row and each column; their outer product over the mean of v_row is the
    factored second moment.  Returns (N, v_row, v_col) with N = the new first moment."""
    R = np.asarray(R, dtype=np.float64)
    beta2t = 1.0 - float(t) ** (-ADAFACTOR_DECAY)
    sq = R * R + ADAFACTOR_EPS1
    v_row = beta2t * v_row + (1.0 - beta2t) * sq.mean(axis=1)
    v_col = beta2t * v_col + (1.0 - beta2t) * sq.mean(axis=0)
    V_hat = np.outer(v_row, v_col) / v_row.mean()
    U = R / np.sqrt(V_hat)
    rms = np.sqrt(np.mean(U * U))
    U = U / max(1.0, rms / ADAFACTOR_CLIP)
    N = beta1 * M_prev + (1.0 - beta1) * U
    return N, v_row, v_col


class GaLoreOracle:
    """One 2-D weight's GaLore-Adam state and step (Algorithm 1), in fp64.

    w_store : 'f64' | 'f32' | 'bf16'   rounding applied to W when it is written
    state   : 'f64' | 'f32' | 'q8'     how M, V are kept between steps
    n_store : 'f64' | 'f32' | 'bf16'   rounding applied to the normalised update
                                        before it is projected back (the CUDA
                                        path feeds its tensor cores bf16)
    inner   : 'adam' | 'identity' | 'adafactor'
                                        the regulariser rho_t; 'identity' is the
                                        rho_t = 1 case of Sec. 3.3 used by one pin;
                                        'adafactor' is Adafactor with first-order
                                        statistics (see adafactor_update)
    """

    def __init__(self, m, n, rank, alpha, refresh_gap, beta1=0.9, beta2=0.999, eps=1e-8,
                 side="auto", w_store="f64", state="f64", n_store="f64", q_block=2048,
                 inner="adam", svd_method="jacobi", weight_decay=0.0):
        if side == "auto":
            side = "left" if m <= n else "right"       # Sec. 4.2; m == n goes left
        if rank < 1 or rank > min(m, n):
            raise ValueError("rank must lie in [1, min(m, n)]")
        self.m, self.n, self.r = int(m), int(n), int(rank)
        self.alpha, self.T = float(alpha), int(refresh_gap)
        self.beta1, self.beta2, self.eps = float(beta1), float(beta2), float(eps)
        self.side, self.w_store, self.state, self.n_store = side, w_store, state, n_store
        self.q_block, self.inner, self.svd_method = int(q_block), inner, svd_method
        # GaLore-AdamW (Sec. "GaLore with memory-efficient optimizers" names AdamW, no equations):
        # decoupled weight decay as Loshchilov & Hutter define it, W <- W (1 - lr lambda) - lr G~,
        # applied to the full-rank weight with the plain learning rate (alpha scales only G~).
        self.weight_decay = float(weight_decay)
        self.k = 0                                      # completed steps
        self.proj = None                                # P (m x r) or Q (n x r)
        self.sigma = None
        shape = (self.r, self.n) if side == "left" else (self.m, self.r)
        self.state_shape = shape
        if state == "q8":
            self.tile = state_tile(self.q_block)
            grid = (-(-shape[0] // self.tile[0]), -(-shape[1] // self.tile[1]))
            zc_s = int(np.nonzero(dynamic_code(True) == 0.0)[0][0])
            zc_u = int(np.nonzero(dynamic_code(False) == 0.0)[0][0])
            self.M_codes = np.full(shape, zc_s, dtype=np.uint8)
            self.V_codes = np.full(shape, zc_u, dtype=np.uint8)
            self.M_absmax = np.zeros(grid, dtype=np.float32)
            self.V_absmax = np.zeros(grid, dtype=np.float32)
        else:
            self.M = np.zeros(shape, dtype=np.float64)
            self.V = np.zeros(shape, dtype=np.float64)
        if inner == "adafactor":
            if state == "q8":
                raise ValueError("the factored second moment is kept in floating point")
            self.V = None
            self.v_row = np.zeros(shape[0], dtype=np.float64)
            self.v_col = np.zeros(shape[1], dtype=np.float64)
        self.refreshes = 0

    # -- state accessors ----------------------------------------------------
    def moments(self):
        """Stored (uncorrected) M, V as fp64 arrays of the state's shape."""
        if self.state == "q8":
            M = dequantize_tiles(self.M_codes, self.M_absmax, True, *self.tile)
            V = dequantize_tiles(self.V_codes, self.V_absmax, False, *self.tile)
            return M.astype(np.float64), V.astype(np.float64)
        return self.M, self.V

    def optimizer_state_elements(self) -> int:
        """Elements held besides W: projector plus two moments (Sec. 4.2: mr + 2nr for m <= n)."""
        proj = (self.m if self.side == "left" else self.n) * self.r
        if self.inner == "adafactor":                   # first moment plus one row and one column vector
            return proj + self.state_shape[0] * self.state_shape[1] + self.state_shape[0] + self.state_shape[1]
        return proj + 2 * self.state_shape[0] * self.state_shape[1]

    def set_projector(self, proj):
        proj = np.array(proj, dtype=np.float64)
        want = (self.m if self.side == "left" else self.n, self.r)
        if proj.shape != want:
            raise ValueError(f"projector shape {proj.shape}, expected {want}")
        self.proj = proj

    # -- the refresh (Algorithm 1, the 't mod T = 0' branch; Eq. 12-13) ------
    def refresh(self, G):
        self.proj, self.sigma = top_r_projector(G, self.r, self.side, self.svd_method)
        self.refreshes += 1
        return self.proj

    # -- one iteration of Algorithm 1 ---------------------------------------
    def step(self, W, G, lr, auto_refresh=True):
        W = np.asarray(W, dtype=np.float64)
        G = np.asarray(G, dtype=np.float64)
        if auto_refresh and self.k % self.T == 0:
            self.refresh(G)
        if self.proj is None:
            raise RuntimeError("no projector: refresh or set_projector first")
        P = self.proj
        # project the gradient into the compact space
        R = P.T @ G if self.side == "left" else G @ P
        if self.inner == "identity":
            N = R
        elif self.inner == "adafactor":
            N, self.v_row, self.v_col = adafactor_update(R, self.M, self.v_row, self.v_col, self.k + 1, self.beta1)
            self.M = _store(N, self.state)
            self.v_row, self.v_col = _store(self.v_row, self.state), _store(self.v_col, self.state)
        else:
            M_prev, V_prev = self.moments()
            M = self.beta1 * M_prev + (1.0 - self.beta1) * R
            V = self.beta2 * V_prev + (1.0 - self.beta2) * (R * R)
            t = self.k + 1
            M_hat = M / (1.0 - self.beta1 ** t)
            V_hat = V / (1.0 - self.beta2 ** t)
            N = M_hat / (np.sqrt(V_hat) + self.eps)
            if self.state == "q8":
                self.M_codes, self.M_absmax = quantize_tiles(M, True, *self.tile)
                self.V_codes, self.V_absmax = quantize_tiles(V, False, *self.tile)
            else:
                self.M, self.V = _store(M, self.state), _store(V, self.state)
        N = _store(N, self.n_store)
        self.last_R, self.last_N = R, N
        # project back and apply
        G_tilde = self.alpha * (P @ N if self.side == "left" else N @ P.T)
        W_new = _store(W * (1.0 - lr * self.weight_decay) - lr * G_tilde, self.w_store)
        self.k += 1
        return W_new
