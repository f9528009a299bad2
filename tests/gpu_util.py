"""Shared helpers of the GPU parity tests: run the CUDA path and the oracle on the same arrays."""
import numpy as np
import torch

from oracle import galore_oracle as go
from paper_2403_03507_b200 import binding as gb
from paper_2403_03507_b200 import workloads as wl

TORCH_DT = {"f32": torch.float32, "bf16": torch.bfloat16}


def to_dev(x: np.ndarray, dtype: str, ld: int | None = None) -> torch.Tensor:
    """Host fp64 array (already rounded to dtype) -> device tensor, optionally with a padded leading dimension."""
    t = torch.from_numpy(np.ascontiguousarray(x)).to(TORCH_DT[dtype]).cuda()
    if ld is None or ld == x.shape[1]:
        return t
    buf = torch.full((x.shape[0], ld), float("nan"), dtype=TORCH_DT[dtype], device="cuda")
    buf[:, :x.shape[1]] = t
    return buf[:, :x.shape[1]]


def to_host(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float64).cpu().numpy()


def rel_err(a, b):
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def bf16_ulp(x):
    """Spacing of bfloat16 values at |x| (8 significand bits): 2**(floor(log2 |x|) - 7), for x != 0."""
    _mant, expo = np.frexp(np.abs(x))                  # |x| = mant * 2**expo, 0.5 <= mant < 1
    return np.ldexp(1.0, expo - 8)


def elementwise_report(W_gpu, W_orc, W0, w_dtype, peak=None):
    """Element-by-element comparison of the updated weights.

    fp32 weights: largest |dW_gpu - dW_orc| over largest |dW_orc| (dW = W - W0).
    bf16 weights: the difference in units of the bf16 spacing at the largest magnitude the element
    had on the oracle's trajectory (`peak`; the larger of start and end value when not given), and
    the share of elements that differ at all.  Both sides round the same real number up to errors
    far below one spacing (fp32 against fp64 sums), so each step can move an element that sits on a
    rounding boundary by one spacing (at the magnitude it has then) and no further; a difference
    made at a large magnitude stays when the element shrinks.
    """
    d = np.abs(W_gpu - W_orc)
    rep = {"max_abs": float(d.max()), "dw_max_rel": float(d.max() / max(np.abs(W_orc - W0).max(), 1e-300))}
    if w_dtype == "bf16":
        if peak is None:
            peak = np.maximum(np.abs(W_orc), np.abs(W0))
        ulp = bf16_ulp(np.maximum(peak, 1e-30))
        rep["max_ulp"] = float((d / ulp).max())
        rep["frac_diff"] = float(np.mean(d > 0))
    return rep


class SignWatch:
    """Marks the lines of W whose comparison is meaningless because Adam's normalised update is discontinuous
    there.  While V is dominated by the current R*R (the first steps from zero moments) N is close to
    sign(R): an element of R within rounding error of zero (fp32 against fp64 sums of K products: about
    sqrt(K) 2^-24 of R's rms) may come out with either sign, N differs by 2, and every W element that uses
    that N (column j of W for R[k, j] on the left side, row i for R[i, k] on the right) moves by
    lr alpha |P|.  Call after each oracle step; lines with such an element are excluded.
    Given the oracle's weights after each step it also keeps every element's largest magnitude so far,
    which is what sets the bf16 spacing a rounding difference can have."""

    def __init__(self, orc, rel=3e-5, W0=None):
        self.orc, self.rel = orc, rel
        rows, cols = orc.state_shape
        self.axis = 0 if orc.side == "left" else 1          # reduce over k
        self.bad = np.zeros(cols if orc.side == "left" else rows, dtype=bool)
        self.peak = None if W0 is None else np.abs(W0)

    def update(self, W_orc=None, layer=None):
        """layer: with 8-bit moments, the CUDA layer after the same step.  A moment that lands within
        rounding error of a code threshold may take the neighbouring code on one side (fp32 against fp64
        arithmetic before the fp32 quotient); in the sparse low decades of the code that changes the
        stored value, and the next N of that element, by tens of percent.  Lines of W fed by an element
        whose codes differ are excluded from then on (the codes themselves are compared by the tests)."""
        R = self.orc.last_R
        rms = np.sqrt(np.mean(R * R))
        self.bad |= (np.abs(R) < self.rel * rms).any(axis=self.axis)
        if layer is not None and self.orc.state == "q8":
            Mc, _Ma, Vc, _Va = [t.cpu().numpy() for t in layer.get_q8_state()]
            self.bad |= ((Mc != self.orc.M_codes) | (Vc != self.orc.V_codes)).any(axis=self.axis)
        if W_orc is not None:
            self.peak = np.abs(W_orc) if self.peak is None else np.maximum(self.peak, np.abs(W_orc))

    def keep(self, W):
        return W[:, ~self.bad] if self.orc.side == "left" else W[~self.bad, :]


def assert_elementwise(W_gpu, W_orc, W0, w_dtype, steps, c_f32=1e-3, frac=0.25, watch=None):
    peak = None
    if watch is not None:
        assert watch.bad.mean() < 0.2, f"{watch.bad.mean():.2f} of the lines excluded: the comparison would mean nothing"
        W_gpu, W_orc, W0 = watch.keep(W_gpu), watch.keep(W_orc), watch.keep(W0)
        peak = None if watch.peak is None else watch.keep(watch.peak)
    rep = elementwise_report(W_gpu, W_orc, W0, w_dtype, peak)
    if w_dtype == "bf16":
        # <= one bf16 spacing per step (see elementwise_report); an element that crossed a power of two on
        # the way had twice the spacing for part of it
        assert rep["max_ulp"] <= 2.0 * steps + 1e-9 and rep["frac_diff"] <= frac, rep
    else:
        assert rep["dw_max_rel"] <= c_f32, rep
    return rep


def device_gradient(m, n, seed, p, noise, dtype):
    """The workloads' gradient recipe generated on the GPU (the QR factorisations of the host generator take
    most of a long run's time at these sizes); returned as the host fp64 array both sides then read."""
    g = wl.make_gradient_torch(m, n, seed & 0x7FFFFFFF, p, noise, "cuda", TORCH_DT[dtype])
    return g.to(torch.float64).cpu().numpy()


def run_pair(m, n, r, steps, T, w_dtype="f32", g_dtype="f32", state_fmt="f32", p=1.0, noise=0.01, lr=1e-2, seed=1,
             q_block=2048, path=gb.PATH_AUTO, side=gb.SIDE_AUTO, ldw=None, ldg=None, oversample=0,
             check_angle=None, svd_method="jacobi", same_g=False, weight_decay=0.0, gen="host"):
    """Steps the CUDA path and the oracle together.

    At every refresh the oracle first computes its own top-r subspace (for the
    principal-angle check), then adopts the projector the CUDA path stored, so
    that both sides apply Adam in the same basis (singular vectors inside a
    cluster of nearly equal singular values are not unique).
    Returns a dict of per-step errors and the final arrays.
    """
    cfg = gb.make_config(m, n, r, alpha=0.25, refresh_gap=T, w_dtype=w_dtype, g_dtype=g_dtype, state_fmt=state_fmt,
                         q_block=q_block, auto_refresh=False, path=path, side=side, refresh_oversample=oversample,
                         seed=seed, weight_decay=weight_decay)
    layer = gb.Layer(cfg)
    side_name = "left" if layer.side == gb.SIDE_LEFT else "right"
    n_store = "bf16" if layer.uses_tensor_path else "f64"
    orc = go.GaLoreOracle(m, n, r, 0.25, T, side=side_name, w_store=w_dtype, n_store=n_store,
                          state={"f32": "f32", "q8": "q8", "adafactor": "f32"}[state_fmt], q_block=q_block,
                          svd_method=svd_method, weight_decay=weight_decay,
                          inner="adafactor" if state_fmt == "adafactor" else "adam")
    W0 = wl.make_weight(m, n, wl.sub_seed(seed, 999), w_dtype)
    W_orc = W0.copy()
    W_gpu = to_dev(W0, w_dtype, ldw)
    out = dict(angles=[], w_err=[], dw_err=[], infos=[], layer=layer, oracle=orc, W0=W0)
    watch = SignWatch(orc, W0=W0)
    for s in range(steps):
        if gen == "device":
            Gs = device_gradient(m, n, wl.sub_seed(seed, 0 if same_g else s), p, noise, g_dtype)
        else:
            Gs = wl.make_gradient(m, n, wl.sub_seed(seed, 0 if same_g else s), p, noise, g_dtype)
        G_gpu = to_dev(Gs, g_dtype, ldg)
        if s % T == 0:
            st, info = layer.galore_refresh_projector(G_gpu)
            out["infos"].append((st, info.as_dict()))
            P_gpu = to_host(layer.get_projector())
            if check_angle is not None:
                P_orc, sig = go.top_r_projector(Gs, r, side_name, svd_method)
                out["angles"].append(go.largest_principal_angle(P_orc, P_gpu))
                out["sigma"] = sig
            orc.set_projector(P_gpu)
        layer.galore_step(W_gpu, G_gpu, lr)
        W_orc = orc.step(W_orc, Gs, lr, auto_refresh=False)
        watch.update(W_orc)
        Wg = to_host(W_gpu)
        out["w_err"].append(rel_err(Wg, W_orc))
        out["dw_err"].append(rel_err(Wg - W0, W_orc - W0))
    torch.cuda.synchronize()
    out["W_gpu"], out["W_orc"] = to_host(W_gpu), W_orc
    out["watch"] = watch
    out["elementwise"] = elementwise_report(watch.keep(out["W_gpu"]), watch.keep(W_orc), watch.keep(W0), w_dtype,
                                            watch.keep(watch.peak))
    out["flags"] = layer.device_status()
    return out
