"""Parity of the refreshed projector with the oracle's top-r singular subspace."""
import numpy as np
import pytest
import torch

from oracle import galore_oracle as go
from paper_2403_03507_b200 import binding as gb
from paper_2403_03507_b200 import workloads as wl

from gpu_util import to_dev, to_host

pytestmark = pytest.mark.gpu

ANGLE_TOL = 1e-3      # largest principal angle, rad


def _refresh(G, r, g_dtype="f32", **kw):
    m, n = G.shape
    cfg = gb.make_config(m, n, r, w_dtype="f32", g_dtype=g_dtype, p_dtype="f32", auto_refresh=False, **kw)
    layer = gb.Layer(cfg)
    st, info = layer.galore_refresh_projector(to_dev(G, g_dtype))
    P = to_host(layer.get_projector())
    assert layer.device_status() == 0
    return st, info.as_dict(), P, layer


@pytest.mark.parametrize("m,n,r", [(96, 200, 8), (200, 96, 8), (128, 128, 32), (150, 310, 70)])
def test_gapped_spectrum_recovers_planted_subspace(m, n, r):
    k = min(m, n)
    spectrum = np.concatenate([np.linspace(10, 5, r), np.linspace(0.5, 0.01, k - r)])
    G, U, V = wl.make_planted(m, n, seed=5, spectrum=spectrum, dtype="f32")
    st, info, P, layer = _refresh(G, r)
    side = "left" if m <= n else "right"
    P_orc, S = go.top_r_projector(G, r, side)
    assert st == gb.OK and info["converged"] == 1
    assert np.max(np.abs(P.T @ P - np.eye(r))) < 1e-5
    assert go.largest_principal_angle(P_orc, P) < ANGLE_TOL
    assert go.largest_principal_angle((U if side == "left" else V)[:, :r], P) < ANGLE_TOL
    # columns are singular vectors in descending order (distinct singular values): |<p_i, u_i>| = 1
    assert np.allclose(np.abs(np.sum(P * P_orc, axis=0)), 1.0, atol=1e-4)
    assert abs(info["sigma_r"] - S[r - 1]) < 1e-5 * S[0] and abs(info["sigma_1"] - S[0]) < 1e-5 * S[0]
    assert info["residual"] < 1e-5


def test_exactly_low_rank_gradient():
    # rank(G) = r < block: P P^T G = G must hold although the iterated block is rank-deficient
    m, n, r = 120, 260, 10
    G, U, V = wl.make_planted(m, n, seed=3, spectrum=np.linspace(4, 1, r), dtype="f64")
    G = wl.round_to(G, "f32")
    st, info, P, _ = _refresh(G, r)
    assert np.max(np.abs(P.T @ P - np.eye(r))) < 1e-5
    assert np.linalg.norm(P @ (P.T @ G) - G) / np.linalg.norm(G) < 1e-5


def test_rank_equal_to_min_dimension_and_zero_gradient():
    G = wl.make_gradient(40, 72, 1, 1.0, 0.01, "f32")
    st, info, P, _ = _refresh(G, 40)
    assert np.max(np.abs(P.T @ P - np.eye(40))) < 1e-5 and info["block"] == 40
    assert np.linalg.norm(P @ (P.T @ G) - G) / np.linalg.norm(G) < 1e-5
    st, info, P, _ = _refresh(np.zeros((24, 40)), 6)
    assert np.all(np.isfinite(P)) and np.max(np.abs(P.T @ P - np.eye(6))) < 1e-4


@pytest.mark.parametrize("m,n,r,g_dtype", [(512, 1376, 128, "f32"), (1376, 512, 128, "f32"), (256, 704, 64, "bf16")])
def test_workload_spectrum_noise_dominated(m, n, r, g_dtype):
    # the decaying-spectrum-plus-noise recipe: sigma_{r+1}/sigma_r is about 0.999
    G = wl.make_gradient(m, n, wl.sub_seed(wl.BASE_SEED, 0), 1.0, 0.01, g_dtype)
    st, info, P, _ = _refresh(G, r, g_dtype)
    side = "left" if m <= n else "right"
    P_orc, S = go.top_r_projector(G, r, side)
    angle = go.largest_principal_angle(P_orc, P)
    print(f"{m}x{n} r={r}: angle {angle:.2e} rad, sigma_r {S[r-1]:.4f}, sigma_r+1/sigma_r {S[r]/S[r-1]:.5f}, info {info}")
    assert np.max(np.abs(P.T @ P - np.eye(r))) < 1e-5
    assert angle < ANGLE_TOL
    # Ritz basis: P^T G G^T P is diagonal with the leading sigma^2 on it
    A = G if side == "left" else G.T
    T = P.T @ A @ A.T @ P
    off = T - np.diag(np.diag(T))
    assert np.max(np.abs(off)) < 1e-4 * S[0] ** 2
    assert np.allclose(np.sqrt(np.diag(T)), S[:r], rtol=1e-4)


def test_iteration_cap_gives_a_warning_not_an_error():
    G = wl.make_gradient(128, 300, 2, 1.0, 0.01, "f32")
    st, info, P, _ = _refresh(G, 32, refresh_max_iters=1, refresh_oversample=-1)
    assert st == gb.WARN_NOT_CONVERGED and info["converged"] == 0 and info["iterations"] == 1
    assert np.max(np.abs(P.T @ P - np.eye(32))) < 1e-5


def test_same_seed_same_projector():
    G = wl.make_gradient(96, 160, 2, 1.0, 0.01, "f32")
    _, _, P1, _ = _refresh(G, 12, seed=7)
    _, _, P2, _ = _refresh(G, 12, seed=7)
    assert np.array_equal(P1, P2)


# ---- power steps on the tensor cores (bf16 gradient and projector) -----------------------------------

def _refresh_tc(G, r, **kw):
    m, n = G.shape
    cfg = gb.make_config(m, n, r, w_dtype="bf16", g_dtype="bf16", auto_refresh=False, **kw)
    layer = gb.Layer(cfg)
    assert layer.uses_tensor_path
    ld = (n + 7) // 8 * 8
    st, info = layer.galore_refresh_projector(to_dev(G, "bf16", ld))
    P = to_host(layer.get_projector())
    _refresh_tc.unrounded = layer.get_unrounded_projector().cpu().numpy()   # before rounding to bf16
    assert layer.device_status() == 0
    return st, info.as_dict(), P


@pytest.mark.parametrize("m,n,r", [(512, 1376, 128), (1376, 512, 128), (768, 2048, 256), (300, 1001, 72)])
def test_tensor_core_refresh_noise_dominated(m, n, r):
    G = wl.make_gradient(m, n, wl.sub_seed(wl.BASE_SEED, 1), 1.0, 0.01, "bf16")
    st, info, P = _refresh_tc(G, r)
    side = "left" if m <= n else "right"
    P_orc, S = go.top_r_projector(G, r, side)
    P_orc_b = wl.round_to(P_orc, "bf16")      # the stored projector is bf16: compare with the same rounding applied
    angle = go.largest_principal_angle(P_orc, P)
    floor = go.largest_principal_angle(P_orc, np.linalg.qr(P_orc_b)[0])
    print(f"{m}x{n} r={r}: angle {angle:.2e} (bf16 storage alone gives {floor:.2e}), {info}")
    assert st == gb.OK and info["converged"] == 1
    # bf16 storage of P limits the angle of the *stored* basis; the iteration itself must be far below 1e-3
    assert angle < max(ANGLE_TOL, 3 * floor)
    # ... and that is checked on the projector as it was before rounding
    assert go.largest_principal_angle(P_orc, _refresh_tc.unrounded) < ANGLE_TOL
    assert info["residual"] < 1e-4
    assert abs(info["sigma_r"] - S[r - 1]) < 1e-4 * S[0]


def test_tensor_core_refresh_gapped_and_low_rank():
    m, n, r = 384, 896, 32
    k = min(m, n)
    spectrum = np.concatenate([np.linspace(10, 5, r), np.linspace(0.5, 0.01, k - r)])
    G, U, V = wl.make_planted(m, n, seed=5, spectrum=spectrum, dtype="bf16")
    st, info, P = _refresh_tc(G, r)
    P_orc, S = go.top_r_projector(G, r, "left")
    assert st == gb.OK
    assert go.largest_principal_angle(P_orc, P) < 5e-3          # bf16 storage of P: about 2e-3
    assert abs(info["sigma_1"] - S[0]) < 1e-4 * S[0]
    # rank(G) = r (up to bf16 rounding of G): the iterated block is numerically rank-deficient
    G2, _, _ = wl.make_planted(m, n, seed=6, spectrum=np.linspace(4, 1, r), dtype="bf16")
    st, info, P = _refresh_tc(G2, r)
    assert np.linalg.norm(P @ (P.T @ G2) - G2) / np.linalg.norm(G2) < 2e-2


def test_full_size_7b_refresh_meets_the_angle_bound_before_rounding():
    """4096 x 11008 at rank 1024 through the tensor-core refresh with its default block (rank + 256).  The
    1e-3 rad bound is checked on the projector before it is rounded to bf16 (the rounding alone moves the
    stored basis by about 2e-3).  Gapped planted spectrum: the top-r subspace is well defined."""
    m, n, r = 4096, 11008, 1024
    k = min(m, n)
    spectrum = np.concatenate([np.linspace(3.0, 1.5, r), 0.6 * np.arange(1, k - r + 1, dtype=np.float64) ** -0.3])
    G, U, V = wl.make_planted(m, n, seed=21, spectrum=spectrum, dtype="bf16")
    st, info, P = _refresh_tc(G, r)
    Pu = _refresh_tc.unrounded
    assert st == gb.OK and info["converged"] == 1 and info["block"] == r + 256
    assert np.abs(Pu.T @ Pu - np.eye(r)).max() < 1e-9
    P_orc, S = go.top_r_projector(G, r, "left", method="lapack")
    assert go.largest_principal_angle(P_orc, Pu) < ANGLE_TOL
    assert go.largest_principal_angle(P_orc, P) < 5e-3
    assert abs(info["sigma_r"] - S[r - 1]) < 1e-4 * S[0]
    # columns are singular vectors in descending order: P^T G G^T P is diagonal with decreasing entries
    B = Pu.T @ G
    D = B @ B.T
    off = D - np.diag(np.diag(D))
    assert np.linalg.norm(off) < 1e-3 * np.linalg.norm(D)
    assert np.all(np.diff(np.diag(D)) <= 1e-6 * D[0, 0])


@pytest.mark.parametrize("g_dtype,m,n,r", [("bf16", 512, 1376, 128), ("bf16", 1376, 512, 128), ("f32", 256, 640, 32)])
def test_layers_refreshed_as_a_group_get_the_projectors_of_single_refreshes(g_dtype, m, n, r):
    """galore_refresh_batch runs neighbours of one shape together (one launch per serial kernel for the whole
    group, grouped tensor-core products).  Every layer keeps its own iteration count and schedule, so the
    stored projector must equal, bit for bit, the one galore_refresh_projector computes for it alone.  The
    gradients differ in spectrum (noise-dominated, gapped, low rank), hence in iterations and Jacobi sweeps;
    a layer of another shape in the middle of the list splits the groups."""
    k = min(m, n)
    grads = [wl.make_gradient(m, n, wl.sub_seed(71, 0), 1.0, 0.01, g_dtype),
             wl.make_gradient(m, n, wl.sub_seed(71, 1), 0.8, 0.05, g_dtype),
             wl.make_planted(m, n, 72, np.concatenate([np.linspace(3, 2, r), 0.3 * np.arange(1, k - r + 1) ** -0.5]), g_dtype)[0],
             wl.make_gradient(m, n, wl.sub_seed(71, 3), 1.0, 0.01, g_dtype),
             wl.make_planted(m, n, 73, np.linspace(4, 1, r), g_dtype)[0],          # rank r: the block is rank-deficient
             wl.make_gradient(m, n, wl.sub_seed(71, 5), 1.0, 0.02, g_dtype)]
    other = wl.make_gradient(m // 2, n, wl.sub_seed(71, 9), 1.0, 0.01, g_dtype)
    ld = (n + 15) // 16 * 16
    Gd = [to_dev(g, g_dtype, ld) for g in grads]
    Gd.insert(3, to_dev(other, g_dtype, ld))

    def layers():
        out = []
        for i, g in enumerate(Gd):
            mm = g.shape[0]
            out.append(gb.Layer(gb.make_config(mm, n, min(r, mm, n), w_dtype="bf16", g_dtype=g_dtype, p_dtype="f32",
                                               auto_refresh=False, seed=100 + i)))
        return out
    single, grouped = layers(), layers()
    infos_single = []
    for layer, g in zip(single, Gd):
        st, info = layer.galore_refresh_projector(g)
        assert st in (gb.OK, gb.WARN_NOT_CONVERGED)
        infos_single.append(info.as_dict())
    need = max(gb.galore_refresh_query_bytes(l) for l in grouped)
    ws = torch.empty(4 * need, dtype=torch.uint8, device="cuda")          # room for groups of four
    st, infos = gb.galore_refresh_batch(grouped, Gd, workspace=ws)
    assert st in (gb.OK, gb.WARN_NOT_CONVERGED)
    for a, b_, ia, ib in zip(single, grouped, infos_single, infos):
        assert a.device_status() == b_.device_status()
        assert torch.equal(a.get_projector(), b_.get_projector())
        assert ia["iterations"] == ib.iterations and ia["jacobi_sweeps"] == ib.jacobi_sweeps
        assert ia["converged"] == ib.converged and ia["sigma_r"] == ib.sigma_r
    # and without a record (no phase clock, no residual) the projectors are the same again
    again = layers()
    lib_st = gb.lib().galore_refresh_batch((gb.C.c_void_p * len(again))(*[l.handle.value for l in again]),
                                           (gb.C.c_void_p * len(again))(*[g.data_ptr() for g in Gd]),
                                           (gb.C.c_int64 * len(again))(*[g.stride(0) for g in Gd]), len(again),
                                           ws.data_ptr(), ws.numel(), None, None)
    assert lib_st in (gb.OK, gb.WARN_NOT_CONVERGED)
    torch.cuda.synchronize()
    for a, c in zip(single, again):
        assert torch.equal(a.get_projector(), c.get_projector())


@pytest.mark.parametrize("g_dtype,m,n,r", [("bf16", 512, 1376, 64), ("bf16", 1376, 512, 64), ("f32", 256, 640, 32)])
def test_warm_started_refresh_reaches_the_cold_subspace_in_fewer_steps(g_dtype, m, n, r):
    """Gradients whose singular subspaces turn slowly (a gapped spectrum, 0.02 rad between consecutive steps):
    a refresh that starts from the stored projector and runs three power steps is accepted by its own
    residual-over-gap bound, lands in the oracle's subspace, and needs a fraction of the cold refresh's steps.
    On the workloads' noise-dominated spectrum (no gap behind the block) the look at the Rayleigh quotients
    after those three steps sends the refresh on to the full iteration of a cold one, from its warm block."""
    k = min(m, n)
    spectrum = np.concatenate([np.linspace(3.0, 2.0, r), 0.3 * np.arange(1, k - r + 1, dtype=np.float64) ** -0.5])
    side = "left" if m <= n else "right"
    drift = 0.02 / np.sqrt(max(m, n))
    G0 = wl.make_rotating(m, n, 91, spectrum, drift, 0, dtype=g_dtype)
    G1 = wl.make_rotating(m, n, 91, spectrum, drift, 1, dtype=g_dtype)
    ld = (n + 15) // 16 * 16
    P0_orc, _ = go.top_r_projector(G0, r, side, method="lapack")
    P1_orc, _ = go.top_r_projector(G1, r, side, method="lapack")
    moved = go.largest_principal_angle(P0_orc, P1_orc)
    assert 5e-3 < moved < 0.2                                  # the subspace did move, by a small angle

    def layer(warm):
        return gb.Layer(gb.make_config(m, n, r, w_dtype="bf16", g_dtype=g_dtype, p_dtype="f32", auto_refresh=False, seed=3,
                                       refresh_warm_iters=warm))
    cold, warm = layer(0), layer(3)
    for l in (cold, warm):                                     # the first refresh of a layer has nothing to start from
        st, info0 = l.galore_refresh_projector(to_dev(G0, g_dtype, ld))
        assert st == gb.OK and go.largest_principal_angle(P0_orc, to_host(l.get_projector())) < 1e-3
    st_c, info_c = cold.galore_refresh_projector(to_dev(G1, g_dtype, ld))
    st_w, info_w = warm.galore_refresh_projector(to_dev(G1, g_dtype, ld))
    Pc, Pw = to_host(cold.get_projector()), to_host(warm.get_projector())
    print(f"{g_dtype} {m}x{n} r={r}: subspace moved {moved:.3f} rad; cold {info_c.iterations} steps, warm {info_w.iterations} steps, "
          f"bound {info_w.predicted_error:.2e}, angles cold {go.largest_principal_angle(P1_orc, Pc):.2e} warm {go.largest_principal_angle(P1_orc, Pw):.2e}")
    assert st_c == gb.OK and st_w == gb.OK and info_w.converged == 1
    assert go.largest_principal_angle(P1_orc, Pw) < 1e-3
    assert go.largest_principal_angle(Pc, Pw) < 1e-3           # the same subspace as the cold refresh
    assert info_w.iterations <= 6 and info_w.iterations < info_c.iterations
    assert np.abs(Pw.T @ Pw - np.eye(r)).max() < 1e-5
    # noise-dominated spectrum: the warm start falls back to the full iteration and still converges
    N0 = wl.make_gradient(m, n, wl.sub_seed(92, 0), 1.0, 0.01, g_dtype)
    N1 = wl.make_gradient(m, n, wl.sub_seed(92, 1), 1.0, 0.01, g_dtype)
    hard = layer(3)
    hard.galore_refresh_projector(to_dev(N0, g_dtype, ld))
    st_h, info_h = hard.galore_refresh_projector(to_dev(N1, g_dtype, ld))
    Ph_orc, _ = go.top_r_projector(N1, r, side, method="lapack")
    assert st_h == gb.OK and info_h.converged == 1 and info_h.iterations > 6
    assert go.largest_principal_angle(Ph_orc, to_host(hard.get_projector())) < 1e-3
