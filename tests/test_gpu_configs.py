"""Parity at the sizes the workload list names: the LLaMA-130M set (bf16 weights, fp32 gradients, fp32 states,
r = 256, T = 200, refreshes at steps 0 and 200), the rank sweep on one 4096 x 11008 matrix, and the refresh on
the workloads' own noise-dominated spectra at full size.  Protocol: at each refresh the oracle computes its own
top-r subspace (largest principal angle <= 1e-3 rad on the projector before rounding), then adopts the stored
projector, and both sides step."""
import numpy as np
import pytest
import torch

from oracle import galore_oracle as go
from paper_2403_03507_b200 import binding as gb
from paper_2403_03507_b200 import workloads as wl

from gpu_util import SignWatch, assert_elementwise, device_gradient, elementwise_report, rel_err, run_pair, to_dev, to_host

pytestmark = pytest.mark.gpu
ANGLE_TOL = 1e-3


# ---- the 130M layer set -------------------------------------------------------------------------------

@pytest.mark.parametrize("m,n", [(768, 768), (768, 2048), (2048, 768)])
def test_130m_shapes_through_both_refreshes(m, n):
    """Steps 0 .. 201 (refreshes at k = 0 and k = 200) of one matrix of each distinct shape of the 130M set.
    Oracle steps cost ~10 ms each at these sizes; the refresh oracle is the library SVD (pinned against the
    Jacobi code in the CPU tests)."""
    w = wl.WORKLOADS["llama_130m"]
    res = run_pair(m, n, w.rank, 202, w.refresh_gap, w.w_dtype, w.g_dtype, w.state_fmt, w.spectrum_p, w.noise, w.lr,
                   seed=wl.sub_seed(w.seed, m, n) & 0x7FFFFFFF, check_angle=True, svd_method="lapack", gen="device")
    assert res["flags"] == 0 and len(res["infos"]) == 2
    assert all(st == gb.OK and info["converged"] == 1 for st, info in res["infos"]), res["infos"]
    assert max(res["angles"]) <= ANGLE_TOL, (res["angles"], res["infos"])
    assert not res["layer"].uses_tensor_path                      # fp32 gradients: the fp32 kernels
    assert max(res["w_err"]) <= 2e-2, max(res["w_err"])
    assert max(res["dw_err"]) <= 0.1, max(res["dw_err"])
    rep = res["elementwise"]
    print(f"130M {m}x{n}: 202 steps, W err {max(res['w_err']):.2e}, update err {max(res['dw_err']):.2e}, {rep}")
    # bf16 weights: one spacing per step at most in principle; measured is a few spacings after 202 steps
    assert rep["max_ulp"] <= 16 and rep["frac_diff"] <= 0.5, rep


def test_130m_400_steps_on_one_shape():
    w = wl.WORKLOADS["llama_130m"]
    m, n = 768, 768
    res = run_pair(m, n, w.rank, 400, w.refresh_gap, w.w_dtype, w.g_dtype, w.state_fmt, w.spectrum_p, w.noise, w.lr,
                   seed=77, check_angle=True, svd_method="lapack", gen="device")
    assert res["flags"] == 0 and len(res["infos"]) == 2 and res["layer"].step_count == 400
    assert max(res["angles"]) <= ANGLE_TOL
    assert max(res["w_err"]) <= 2e-2 and max(res["dw_err"]) <= 0.1, (max(res["w_err"]), max(res["dw_err"]))


def test_130m_batched_step_equals_the_oracle():
    """All seven matrices of one 130M layer through galore_step_batch (they are not on the tensor path, so the
    batch steps them one by one): three steps against the oracle."""
    w = wl.WORKLOADS["llama_130m"]
    shapes = [(768, 768)] * 4 + [(768, 2048)] * 2 + [(2048, 768)]
    layers, orcs, Wd, W0s = [], [], [], []
    for i, (m, n) in enumerate(shapes):
        cfg = gb.make_config(m, n, w.rank, alpha=w.alpha, refresh_gap=w.refresh_gap, w_dtype=w.w_dtype, g_dtype=w.g_dtype,
                             state_fmt=w.state_fmt, auto_refresh=False)
        layer = gb.Layer(cfg)
        d = min(m, n)
        P = wl.round_to(wl.random_orthonormal(d, w.rank, np.random.default_rng(i)), "f32")
        layer.set_projector(torch.from_numpy(P))
        o = go.GaLoreOracle(m, n, w.rank, w.alpha, w.refresh_gap, w_store=w.w_dtype, state="f32")
        o.set_projector(P)
        W0 = wl.make_weight(m, n, 500 + i, w.w_dtype)
        layers.append(layer); orcs.append(o); W0s.append(W0); Wd.append(to_dev(W0, w.w_dtype))
    Wo = list(W0s)
    watches = [SignWatch(o, W0=w0) for o, w0 in zip(orcs, W0s)]
    for s in range(3):
        Gh = [wl.make_gradient(m, n, wl.sub_seed(w.seed, i, s), w.spectrum_p, w.noise, w.g_dtype) for i, (m, n) in enumerate(shapes)]
        gb.Batch(layers, Wd, [to_dev(g, w.g_dtype) for g in Gh]).galore_step_batch(w.lr)
        Wo = [o.step(x, g, w.lr, auto_refresh=False) for o, x, g in zip(orcs, Wo, Gh)]
        for wt, wo in zip(watches, Wo):
            wt.update(wo)
    for layer, wd, wo, w0, wt in zip(layers, Wd, Wo, W0s, watches):
        assert layer.device_status() == 0
        assert_elementwise(to_host(wd), wo, w0, "bf16", 3, watch=wt)


# ---- rank sweep on 4096 x 11008 and full-size refreshes on the workloads' own spectra ----------------------

def _refresh_and_angles(G, r, seed=3, oversample=0):
    m, n = G.shape
    cfg = gb.make_config(m, n, r, w_dtype="bf16", g_dtype="bf16", auto_refresh=False, seed=seed,
                         refresh_oversample=oversample)
    layer = gb.Layer(cfg)
    assert layer.uses_tensor_path
    ld = (n + 15) // 16 * 16
    st, info = layer.galore_refresh_projector(to_dev(G, "bf16", ld))
    Pu = layer.get_unrounded_projector().cpu().numpy()
    P = to_host(layer.get_projector())
    assert layer.device_status() == 0
    return layer, st, info.as_dict(), Pu, P


def _ritz_diagonality(Pu, G, left):
    B = Pu.T @ G if left else G @ Pu        # r x n resp. m x r
    D = B @ B.T if left else B.T @ B
    off = D - np.diag(np.diag(D))
    return np.linalg.norm(off) / np.linalg.norm(D), np.diag(D)


def test_rank_sweep_matrix_refresh_and_steps():
    """One 4096 x 11008 bf16 matrix of the sweep workload (s_i = 1/i, noise 0.01): one SVD serves all ranks (the
    top-r subspaces are nested).  Ranks 64, 256 and 2048: angle of the refreshed projector before rounding, then
    two steps against the oracle with the stored projector, with fp32 moments (every element compared) and with
    8-bit moments (norms, codes and a loose element-wise bound: at this size every column of W is fed by some
    moment whose code differs by one step between fp32 and fp64 arithmetic)."""
    w = wl.WORKLOADS["sweep_4096x11008"]
    m, n, _ = w.shapes[0]
    G0 = device_gradient(m, n, wl.sub_seed(w.seed, 0), w.spectrum_p, w.noise, "bf16")
    U, S, _Vt = np.linalg.svd(G0, full_matrices=False)
    W0 = wl.make_weight(m, n, 8, "bf16")
    G1 = device_gradient(m, n, wl.sub_seed(w.seed, 1), w.spectrum_p, w.noise, "bf16")
    ld = (n + 15) // 16 * 16
    cs, cu = go.dynamic_code(True).astype(np.float64), go.dynamic_code(False).astype(np.float64)
    for r in (64, 256, 2048):
        layer, st, info, Pu, P = _refresh_and_angles(G0, r)
        angle = go.largest_principal_angle(U[:, :r], Pu)
        offd, diag = _ritz_diagonality(Pu, G0, True)
        print(f"sweep r={r}: angle {angle:.2e} rad, off-diagonal {offd:.2e}, sigma_r {S[r-1]:.4f} sigma_r+1 {S[r]:.4f}, {info}")
        assert st == gb.OK and info["converged"] == 1, info
        assert angle <= ANGLE_TOL
        assert np.abs(Pu.T @ Pu - np.eye(r)).max() < 1e-9
        assert abs(info["sigma_r"] - S[r - 1]) < 1e-4 * S[0]
        del layer
        for fmt in ("f32", "q8"):
            cfg = gb.make_config(m, n, r, alpha=w.alpha, state_fmt=fmt, auto_refresh=False)
            step_layer = gb.Layer(cfg)
            step_layer.set_projector(torch.from_numpy(P))
            o = go.GaLoreOracle(m, n, r, w.alpha, w.refresh_gap, w_store="bf16", state=fmt, n_store="bf16")
            o.set_projector(P)
            Wd, Wo = to_dev(W0, "bf16", ld), W0
            wt = SignWatch(o, W0=W0)
            for G in (G0, G1):
                step_layer.galore_step(Wd, to_dev(G, "bf16", ld), w.lr)
                Wo = o.step(Wo, G, w.lr, auto_refresh=False)
                wt.update(Wo)
            assert step_layer.device_status() == 0
            Wg = to_host(Wd)
            assert rel_err(Wg, Wo) <= 2e-2 and rel_err(Wg - W0, Wo - W0) <= 5e-2
            if fmt == "f32":
                rep = assert_elementwise(Wg, Wo, W0, "bf16", 2, watch=wt)
            else:
                Mc, _Ma, Vc, _Va = [t.cpu().numpy() for t in step_layer.get_q8_state()]
                assert np.mean(Mc != o.M_codes) < 5e-3 and np.max(np.abs(cs[Mc] - cs[o.M_codes])) <= 2 * 0.9 / 64 + 1e-6
                assert np.mean(Vc != o.V_codes) < 5e-3 and np.max(np.abs(cu[Vc] - cu[o.V_codes])) <= 2 * 0.9 / 128 + 1e-6
                rep = elementwise_report(Wg, Wo, W0, "bf16", wt.peak)
                # one differing code changes one N element by O(1) and with it a column of W by lr alpha |P|:
                # a small share of the largest update, on a small share of the elements
                assert rep["dw_max_rel"] <= 0.25 and np.mean(np.abs(Wg - Wo) > 4 * 2.0 ** -8 * wt.peak) <= 0.02, rep
            print(f"   r={r} {fmt}: {rep}")
            del step_layer


@pytest.mark.parametrize("name,m,n", [("llama_1b_q8", 2048, 5461), ("llama_1b_q8", 5461, 2048), ("llama_7b_q8", 4096, 11008)])
def test_full_size_refresh_on_the_workloads_own_spectrum(name, m, n):
    """The refresh as bench.py runs it (default block, default tolerance) on the noise-dominated recipe of the
    1B and 7B workloads: sigma_{r+1} / sigma_r is about 0.9998, so the top-r subspace is the hard case."""
    w = wl.WORKLOADS[name]
    r = w.rank
    G = device_gradient(m, n, wl.sub_seed(w.seed, m, n), w.spectrum_p, w.noise, "bf16")
    left = m <= n
    layer, st, info, Pu, P = _refresh_and_angles(G, r)
    P_orc, S = go.top_r_projector(G, r, "left" if left else "right", method="lapack")
    angle = go.largest_principal_angle(P_orc, Pu)
    offd, diag = _ritz_diagonality(Pu, G, left)
    print(f"{name} {m}x{n} r={r}: angle {angle:.2e} rad before rounding, stored {go.largest_principal_angle(P_orc, P):.2e}, "
          f"off-diagonal {offd:.2e}, sigma_r {S[r-1]:.5f} sigma_r+1 {S[r]:.5f} ratio {S[r]/S[r-1]:.5f}, {info}")
    assert st == gb.OK and info["converged"] == 1, info
    assert angle <= ANGLE_TOL
    assert offd < 1e-3 and np.all(np.diff(diag) <= 1e-6 * diag[0])
    assert abs(info["sigma_r"] - S[r - 1]) < 1e-4 * S[0] and abs(info["sigma_next"] - S[r]) < 1e-3 * S[0]


# ---- checkpoint through the listed calls ------------------------------------------------------------------

@pytest.mark.parametrize("state_fmt,g_dtype,w_dtype", [("f32", "f32", "f32"), ("q8", "bf16", "bf16"), ("f32", "bf16", "bf16")])
def test_export_import_resume_is_bit_identical(state_fmt, g_dtype, w_dtype):
    """10 steps = 5 steps, export, import into a fresh layer, 5 steps; with a refresh inside each half (T = 4)."""
    m, n, r, T = 256, 520, 32, 4
    ld = (n + 15) // 16 * 16
    grads = [to_dev(wl.make_gradient(m, n, wl.sub_seed(4, s), 1.0, 0.01, g_dtype), g_dtype, ld) for s in range(10)]
    W0 = wl.make_weight(m, n, 9, w_dtype)

    def fresh():
        return gb.Layer(gb.make_config(m, n, r, refresh_gap=T, w_dtype=w_dtype, g_dtype=g_dtype, state_fmt=state_fmt,
                                       auto_refresh=True, seed=5, q_block=512))
    a, Wa = fresh(), to_dev(W0, w_dtype, ld)
    for g in grads:
        a.galore_step(Wa, g, 1e-2)
    b, Wb = fresh(), to_dev(W0, w_dtype, ld)
    for g in grads[:5]:
        b.galore_step(Wb, g, 1e-2)
    blob = b.export_state()
    assert b.step_count == 5
    c = fresh()
    c.import_state(blob)
    assert c.step_count == 5
    assert torch.equal(c.get_projector(), b.get_projector())
    Wc = Wb.clone()
    for g in grads[5:]:
        c.galore_step(Wc, g, 1e-2)
    torch.cuda.synchronize()
    assert torch.equal(Wc, Wa)
    # the states themselves (the raw buffers also hold alignment padding that nothing writes)
    assert torch.equal(c.get_projector(), a.get_projector())
    if state_fmt == "q8":
        assert all(torch.equal(x, y) for x, y in zip(c.get_q8_state(), a.get_q8_state()))
    else:
        assert all(torch.equal(x, y) for x, y in zip(c.get_moments(), a.get_moments()))
    # a blob of another configuration is refused, a truncated or foreign one too
    other = gb.Layer(gb.make_config(m, n, r + 8, refresh_gap=T, w_dtype=w_dtype, g_dtype=g_dtype, state_fmt=state_fmt))
    with pytest.raises(gb.GaloreError) as e:
        other.import_state(blob)
    assert e.value.status == gb.ERR_STATE
    with pytest.raises(gb.GaloreError) as e:
        c.import_state(blob[:40].clone())
    assert e.value.status == gb.ERR_BUFFER_TOO_SMALL
    junk = blob.clone()
    junk[0] ^= 0xFF
    with pytest.raises(gb.GaloreError) as e:
        c.import_state(junk)
    assert e.value.status == gb.ERR_INVALID_ARG


def test_check_device_maps_latched_bits_to_status_codes():
    cfg = gb.make_config(32, 48, 4, w_dtype="f32", g_dtype="f32", auto_refresh=False)
    layer = gb.Layer(cfg)
    layer.set_projector(torch.eye(32)[:, :4])
    W = torch.zeros(32, 48, device="cuda")
    G = torch.ones(32, 48, device="cuda")
    layer.galore_step(W, G, 1e-2)
    assert layer.check_device() == gb.OK
    G[3, 5] = float("nan")
    layer.galore_step(W, G, 1e-2)
    assert layer.check_device() == gb.ERR_NONFINITE
    assert layer.check_device() == gb.OK           # reading clears the bits
