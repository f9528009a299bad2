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


def run_pair(m, n, r, steps, T, w_dtype="f32", g_dtype="f32", state_fmt="f32", p=1.0, noise=0.01, lr=1e-2, seed=1,
             q_block=2048, path=gb.PATH_AUTO, side=gb.SIDE_AUTO, ldw=None, ldg=None, oversample=0,
             check_angle=None, svd_method="jacobi", same_g=False, weight_decay=0.0):
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
                          state={"f32": "f32", "q8": "q8"}[state_fmt], q_block=q_block, svd_method=svd_method,
                          weight_decay=weight_decay)
    W0 = wl.make_weight(m, n, wl.sub_seed(seed, 999), w_dtype)
    W_orc = W0.copy()
    W_gpu = to_dev(W0, w_dtype, ldw)
    out = dict(angles=[], w_err=[], dw_err=[], infos=[], layer=layer, oracle=orc, W0=W0)
    for s in range(steps):
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
        Wg = to_host(W_gpu)
        out["w_err"].append(rel_err(Wg, W_orc))
        out["dw_err"].append(rel_err(Wg - W0, W_orc - W0))
    torch.cuda.synchronize()
    out["W_gpu"], out["W_orc"] = to_host(W_gpu), W_orc
    out["flags"] = layer.device_status()
    return out
