"""Parity of the Adafactor inner optimizer (state format GALORE_STATE_ADAFACTOR) with the oracle."""
import numpy as np
import pytest
import torch

from oracle import galore_oracle as go
from paper_2403_03507_b200 import binding as gb
from paper_2403_03507_b200 import workloads as wl

from gpu_util import assert_elementwise, rel_err, run_pair, to_dev, to_host

pytestmark = pytest.mark.gpu


def _state_close(layer, orc, tol):
    M, v_row, v_col = [to_host(t) for t in layer.get_adafactor_state()]
    assert rel_err(M, orc.M) < tol, rel_err(M, orc.M)
    assert np.abs(v_row / orc.v_row - 1.0).max() < tol and np.abs(v_col / orc.v_col - 1.0).max() < tol


@pytest.mark.parametrize("m,n,r", [(256, 704, 64), (704, 256, 64), (130, 301, 17), (301, 130, 17), (64, 64, 64)])
def test_fp32_path_matches_the_oracle(m, n, r):
    """fp32 W, G and projector on the FMA kernels; gradients of growing size so that some steps are clipped
    (rms of the unscaled update above 1 after the second moment lags behind) and some are not."""
    out = run_pair(m, n, r, steps=7, T=3, state_fmt="adafactor", noise=0.05, seed=3)
    assert out["flags"] == 0
    assert max(out["w_err"]) < 1e-4 and max(out["dw_err"]) < 2e-3, (out["w_err"], out["dw_err"])
    _state_close(out["layer"], out["oracle"], 1e-4)
    assert_elementwise(out["W_gpu"], out["W_orc"], out["W0"], "f32", 7, watch=out["watch"])


@pytest.mark.parametrize("m,n,r", [(512, 1376, 128), (1376, 512, 128), (300, 1000, 256), (2048, 2048, 512)])
def test_tensor_path_matches_the_oracle(m, n, r):
    ld = (n + 7) // 8 * 8
    out = run_pair(m, n, r, steps=5, T=4, w_dtype="bf16", g_dtype="bf16", state_fmt="adafactor", p=0.8, noise=0.05,
                   ldw=ld, ldg=ld, svd_method="lapack", seed=5)
    assert out["layer"].uses_tensor_path and out["flags"] == 0
    assert max(out["w_err"]) < 2e-2 and max(out["dw_err"]) < 3e-2, (out["w_err"], out["dw_err"])
    _state_close(out["layer"], out["oracle"], 2e-3)      # R itself comes from bf16 operands on the tensor cores


def test_clipping_takes_effect_and_matches():
    """A gradient a hundred times larger than the ones the second moment has seen: the unclipped update has an
    rms far above 1 and is scaled back to rms 1 before it enters the momentum."""
    m, n, r = 192, 640, 48
    cfg = gb.make_config(m, n, r, w_dtype="f32", g_dtype="f32", state_fmt="adafactor", auto_refresh=False, beta1=0.0)
    layer = gb.Layer(cfg)
    P = wl.random_orthonormal(m, r, np.random.default_rng(1))
    layer.set_projector(torch.from_numpy(P.astype(np.float32)))
    orc = go.GaLoreOracle(m, n, r, 0.25, 1000, beta1=0.0, w_store="f32", state="f32", inner="adafactor")
    orc.set_projector(P.astype(np.float32).astype(np.float64))
    W = wl.make_weight(m, n, 2, "f32")
    Wg = to_dev(W, "f32")
    for s, scale in enumerate([1.0, 1.0, 1.0, 100.0, 1.0]):
        G = wl.make_gradient(m, n, wl.sub_seed(7, s), 1.0, 0.05, "f32") * scale
        layer.galore_step(Wg, to_dev(G, "f32"), 1e-2)
        W = orc.step(W, G, 1e-2, auto_refresh=False)
        M, _, _ = layer.get_adafactor_state()
        rms = float(M.double().pow(2).mean().sqrt())
        assert rms <= 1.0 + 1e-5
        if scale > 1.0:
            assert rms > 0.999                                  # beta1 = 0: M is the clipped update itself
        assert rel_err(to_host(Wg), W) < 1e-5
    _state_close(layer, orc, 1e-4)


def test_state_size_getters_and_batched_call():
    m, n, r = 512, 1024, 128
    cfg = gb.make_config(m, n, r, state_fmt="adafactor", auto_refresh=False)
    sb, _ = gb.galore_query_bytes(cfg)
    pad = lambda b: (b + 255) // 256 * 256
    assert sb == pad(2 * m * r) + pad(4 * r * n) + pad(4 * r) + pad(4 * n)      # bf16 P, fp32 M, one value per row and column
    a, b = gb.Layer(cfg), gb.Layer(gb.make_config(m, n, r, state_fmt="f32", auto_refresh=False))
    with pytest.raises(gb.GaloreError) as e:
        a.get_moments()
    assert e.value.status == gb.ERR_STATE
    # a batch that mixes the two inner optimizers: the Adafactor layer steps on its own, results as for single calls
    P = wl.round_to(wl.random_orthonormal(m, r, np.random.default_rng(3)), "bf16")
    ref = gb.Layer(cfg)
    for l in (a, b, ref):
        l.set_projector(torch.from_numpy(P))
    W0 = wl.make_weight(m, n, 4, "bf16")
    G = wl.make_gradient(m, n, 9, 0.8, 0.05, "bf16")
    Wa, Wb, Wr = to_dev(W0, "bf16"), to_dev(W0, "bf16"), to_dev(W0, "bf16")
    Gd = to_dev(G, "bf16")
    batch = gb.Batch([a, b], [Wa, Wb], [Gd, Gd])
    batch.galore_step_batch(1e-2)
    ref.galore_step(Wr, Gd, 1e-2)
    torch.cuda.synchronize()
    assert torch.equal(Wa, Wr)
    for x, y in zip(a.get_adafactor_state(), ref.get_adafactor_state()):
        assert torch.equal(x, y)


def test_export_import_resumes_bit_identically():
    m, n, r = 384, 1000, 128
    cfg = gb.make_config(m, n, r, state_fmt="adafactor", refresh_gap=3, seed=2)
    ld = (n + 7) // 8 * 8
    Gs = [to_dev(wl.make_gradient(m, n, wl.sub_seed(4, s), 0.8, 0.05, "bf16"), "bf16", ld) for s in range(6)]
    W0 = wl.make_weight(m, n, 1, "bf16")
    a = gb.Layer(cfg)
    Wa = to_dev(W0, "bf16", ld)
    for s in range(4):
        a.galore_step(Wa, Gs[s], 1e-2)
    blob = a.export_state()
    b = gb.Layer(cfg)
    b.import_state(blob)
    Wb = Wa.clone()
    for s in range(4, 6):
        a.galore_step(Wa, Gs[s], 1e-2)
        b.galore_step(Wb, Gs[s], 1e-2)
    torch.cuda.synchronize()
    assert a.step_count == b.step_count == 6 and torch.equal(Wa, Wb)
    for x, y in zip(a.get_adafactor_state(), b.get_adafactor_state()):
        assert torch.equal(x, y)


@pytest.mark.parametrize("state_fmt", ["adafactor", "f32"])
def test_fp32_path_layers_in_a_batch_match_the_oracle(state_fmt):
    """Nine fp32 layers (not on the tensor path) in one batched call: grouped launches of the FMA kernels for
    the two projections, one grouped launch for the inner optimizer; K is not sliced with this many in flight."""
    shapes = [(192, 640, 48), (640, 192, 48), (256, 333, 32), (130, 301, 17), (192, 640, 48), (512, 256, 64),
              (200, 304, 16), (384, 1000, 128), (333, 256, 32)]          # both sides, in no particular order
    inner = "adafactor" if state_fmt == "adafactor" else "adam"
    layers, orcs, Wg, Wo = [], [], [], []
    for i, (m, n, r) in enumerate(shapes):
        layer = gb.Layer(gb.make_config(m, n, r, w_dtype="f32", g_dtype="f32", state_fmt=state_fmt, auto_refresh=False))
        P = wl.random_orthonormal(min(m, n), r, np.random.default_rng(i)).astype(np.float32)
        layer.set_projector(torch.from_numpy(P))
        o = go.GaLoreOracle(m, n, r, 0.25, 1000, w_store="f32", state="f32", inner=inner)
        o.set_projector(P.astype(np.float64))
        W0 = wl.make_weight(m, n, 50 + i, "f32")
        layers.append(layer); orcs.append(o); Wg.append(to_dev(W0, "f32")); Wo.append(W0)
    before = gb.galore_launch_count()
    for s in range(3):
        Gh = [wl.make_gradient(m, n, wl.sub_seed(21, i, s), 1.0, 0.05, "f32") for i, (m, n, r) in enumerate(shapes)]
        Gd = [to_dev(g, "f32") for g in Gh]
        gb.Batch(layers, Wg, Gd).galore_step_batch(1e-2)
        Wo = [o.step(w, g, 1e-2, auto_refresh=False) for o, w, g in zip(orcs, Wo, Gh)]
    torch.cuda.synchronize()
    launches = gb.galore_launch_count() - before
    assert launches <= 2 * 3 * (3 + (5 if state_fmt == "adafactor" else 2))      # one group per side, phase and step
    for i, (wg, wo) in enumerate(zip(Wg, Wo)):
        assert rel_err(to_host(wg), wo) < 1e-5, i
    assert all(l.step_count == 3 and l.device_status() == 0 for l in layers)
    if state_fmt == "adafactor":
        for l, o in zip(layers, orcs):
            _state_close(l, o, 1e-4)
