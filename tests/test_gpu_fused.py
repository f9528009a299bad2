"""The projection kernel with Adam in its epilogue (one K slice per tile: galore_step_batch with four or more
layers, or a single layer whose projection is not sliced) against the oracle, element by element; and the
8-bit codes of every Adam kernel bit for bit on inputs whose fp32 arithmetic is exact."""
import numpy as np
import pytest
import torch

from oracle import galore_oracle as go
from paper_2403_03507_b200 import binding as gb
from paper_2403_03507_b200 import workloads as wl

from gpu_util import SignWatch, assert_elementwise, rel_err, to_dev, to_host

pytestmark = pytest.mark.gpu

# (m, n, r): left and right sides, single CTAs (r < 256) and CTA pairs, ragged last tile column (n % 128 != 0),
# ragged last tile row (rows of the state no multiple of the tile height), several 256-column tiles
SHAPES = [(256, 512, 64), (512, 256, 64), (384, 1000, 128), (1000, 384, 128), (200, 304, 16), (130, 2056, 8),
          (512, 1096, 256), (1096, 512, 256), (300, 1365, 264), (1365, 300, 264)]


def _ld(n):
    return (n + 15) // 16 * 16


def _build(state_fmt, w_dtype, q_block, shapes=SHAPES, weight_decay=0.0, adam_place=gb.ADAM_IN_PROJECTION):
    layers, orcs, Wd, W0s = [], [], [], []
    for i, (m, n, r) in enumerate(shapes):
        cfg = gb.make_config(m, n, r, refresh_gap=1000, w_dtype=w_dtype, g_dtype="bf16", state_fmt=state_fmt,
                             auto_refresh=False, q_block=q_block, weight_decay=weight_decay, adam_place=adam_place)
        layer = gb.Layer(cfg)
        assert layer.uses_tensor_path
        d = m if layer.side == gb.SIDE_LEFT else n
        P = wl.round_to(wl.random_orthonormal(d, r, np.random.default_rng(i)), "bf16")
        layer.set_projector(torch.from_numpy(P))
        o = go.GaLoreOracle(m, n, r, 0.25, 1000, w_store=w_dtype, state=state_fmt, q_block=q_block, n_store="bf16",
                            weight_decay=weight_decay)
        o.set_projector(P)
        W0 = wl.make_weight(m, n, 300 + i, w_dtype)
        layers.append(layer); orcs.append(o); W0s.append(W0); Wd.append(to_dev(W0, w_dtype, _ld(n)))
    return layers, orcs, Wd, W0s


@pytest.mark.parametrize("state_fmt,w_dtype,q_block", [("f32", "bf16", 2048), ("f32", "f32", 2048), ("q8", "bf16", 2048),
                                                       ("q8", "bf16", 256), ("q8", "f32", 512), ("q8", "bf16", 1024)])
def test_fused_batch_matches_the_oracle_element_by_element(state_fmt, w_dtype, q_block):
    layers, orcs, Wd, W0s = _build(state_fmt, w_dtype, q_block)
    launches0 = gb.galore_launch_count()
    Wo = list(W0s)
    watches = [SignWatch(o, W0=w0) for o, w0 in zip(orcs, W0s)]
    batch = None
    steps = 3
    for s in range(steps):
        Gh = [wl.make_gradient(m, n, wl.sub_seed(23, i, s), 0.8, 0.05, "bf16") for i, (m, n, r) in enumerate(SHAPES)]
        Gd = [to_dev(g, "bf16", _ld(g.shape[1])) for g in Gh]
        if batch is None:
            batch = gb.Batch(layers, Wd, Gd)
        else:
            batch.rebind(Wd, Gd)
        batch.galore_step_batch(1e-2)
        Wo = [o.step(w, g, 1e-2, auto_refresh=False) for o, w, g in zip(orcs, Wo, Gh)]
        for wt, wo, layer in zip(watches, Wo, layers):
            wt.update(wo, layer)
    torch.cuda.synchronize()
    # two launches per group and step (projection with Adam, back-projection); single CTAs and CTA pairs are
    # separate groups, and the workspace holds two groups at a time
    launches = gb.galore_launch_count() - launches0
    assert launches % (2 * steps) == 0 and 2 <= launches // (2 * steps) <= 5, launches
    cs, cu = go.dynamic_code(True).astype(np.float64), go.dynamic_code(False).astype(np.float64)
    for layer, o, wd, w0, wo, wt in zip(layers, orcs, Wd, W0s, Wo, watches):
        assert layer.device_status() == 0 and layer.step_count == steps
        Wg = to_host(wd)
        assert rel_err(Wg, wo) <= (2e-2 if w_dtype == "bf16" else 1e-4)
        assert_elementwise(Wg, wo, w0, w_dtype, steps, c_f32=2e-2 if state_fmt == "q8" else 5e-3, watch=wt)
        M, V = [to_host(t) for t in layer.get_moments()]
        Mo, Vo = o.moments()
        if state_fmt == "f32":
            assert np.abs(M - Mo).max() <= 1e-5 * np.abs(Mo).max() and np.abs(V - Vo).max() <= 1e-5 * np.abs(Vo).max()
        else:
            Mc, Ma, Vc, Va = [t.cpu().numpy() for t in layer.get_q8_state()]
            assert np.allclose(Ma, o.M_absmax, rtol=1e-5, atol=0) and np.allclose(Va, o.V_absmax, rtol=1e-5, atol=0)
            # fp32 against fp64 arithmetic may move a value on a threshold to the neighbouring code; such a code is an
            # input difference of the next step, so over a few steps two coarse steps bound the distance
            assert np.mean(Mc != o.M_codes) < 5e-3 and np.max(np.abs(cs[Mc] - cs[o.M_codes])) <= 2 * 0.9 / 64 + 1e-6
            assert np.mean(Vc != o.V_codes) < 5e-3 and np.max(np.abs(cu[Vc] - cu[o.V_codes])) <= 2 * 0.9 / 128 + 1e-6


def test_single_layer_step_without_k_slices_runs_adam_in_the_projection():
    # 1024 x 8192, r = 512: 2 x 32 tiles of 256 x 256 fill the machine without slicing K: two launches per step
    m, n, r = 1024, 8192, 512
    cfg = gb.make_config(m, n, r, state_fmt="q8", auto_refresh=False, adam_place=gb.ADAM_IN_PROJECTION)
    layer = gb.Layer(cfg)
    P = wl.round_to(wl.random_orthonormal(m, r, np.random.default_rng(0)), "bf16")
    layer.set_projector(torch.from_numpy(P))
    o = go.GaLoreOracle(m, n, r, 0.25, 1000, w_store="bf16", state="q8", n_store="bf16")
    o.set_projector(P)
    W0 = wl.make_weight(m, n, 5, "bf16")
    Wd, Wo = to_dev(W0, "bf16"), W0
    wt = SignWatch(o, W0=W0)
    l0 = gb.galore_launch_count()
    for s in range(2):
        G = wl.make_gradient(m, n, wl.sub_seed(31, s), 0.8, 0.05, "bf16")
        layer.galore_step(Wd, to_dev(G, "bf16"), 1e-2)
        Wo = o.step(Wo, G, 1e-2, auto_refresh=False)
        wt.update(Wo, layer)
    launches = gb.galore_launch_count() - l0
    assert launches in (4, 6)            # 4 when the projection is not sliced
    assert layer.device_status() == 0
    assert_elementwise(to_host(Wd), Wo, W0, "bf16", 2, watch=wt)
    Mc, Ma, Vc, Va = [t.cpu().numpy() for t in layer.get_q8_state()]
    assert np.mean(Mc != o.M_codes) < 5e-3 and np.mean(Vc != o.V_codes) < 5e-3


def _signed_permutation(d, r, rng):
    P = np.zeros((d, r))
    rows = rng.permutation(d)[:r]
    P[rows, np.arange(r)] = rng.choice([-1.0, 1.0], r)
    return P


@pytest.mark.parametrize("mode", ["fused", "tensor_standalone", "tensor_standalone_batch", "fp32_path"])
@pytest.mark.parametrize("q_block", [256, 1024, 2048])
def test_codes_are_bit_exact_when_fp32_arithmetic_is_exact(mode, q_block):
    """beta1 = 0.5, beta2 = 0.75, P = columns of a signed permutation matrix and bf16 gradients: R is a signed
    copy of rows of G, the moment updates are exact in fp32 (products of at most 8 x 8 or 2 x 24 bits, one
    rounding in the final sum on both sides), so the stored codes and absmax must equal the oracle's bit for
    bit, on every kernel that writes them: the projection epilogue, the stand-alone tile kernel on the
    tensor path (batches of fewer and of more than four layers) and on the fp32 path (interior and edge tiles)."""
    shapes = [(256, 512, 64), (512, 256, 64), (200, 304, 16), (300, 1365, 264), (1365, 300, 264)]
    if mode == "tensor_standalone":
        shapes = shapes[:3]                      # fewer than four layers per batch: K may be sliced, Adam in its own kernel
    rng = np.random.default_rng(q_block)
    layers, orcs, Wd = [], [], []
    for i, (m, n, r) in enumerate(shapes):
        g_dtype = "f32" if mode == "fp32_path" else "bf16"
        cfg = gb.make_config(m, n, r, refresh_gap=1000, beta1=0.5, beta2=0.75, w_dtype="bf16", g_dtype=g_dtype,
                             state_fmt="q8", auto_refresh=False, q_block=q_block,
                             path=gb.PATH_FP32 if mode == "fp32_path" else gb.PATH_TENSOR,
                             adam_place=gb.ADAM_IN_PROJECTION if mode == "fused" else gb.ADAM_OWN_KERNEL)
        layer = gb.Layer(cfg)
        d = m if layer.side == gb.SIDE_LEFT else n
        P = _signed_permutation(d, r, rng)
        layer.set_projector(torch.from_numpy(P))
        o = go.GaLoreOracle(m, n, r, 0.25, 1000, beta1=0.5, beta2=0.75, w_store="bf16", state="q8", q_block=q_block)
        o.set_projector(P)
        layers.append(layer); orcs.append(o)
        Wd.append(to_dev(wl.make_weight(m, n, i, "bf16"), "bf16", _ld(n)))
    for s in range(3):
        # gradients on the bf16 grid (8 significant bits) whatever the storage type
        Gh = [wl.make_gradient(m, n, wl.sub_seed(41, i, s), 0.8, 0.05, "bf16") for i, (m, n, r) in enumerate(shapes)]
        Gd = [to_dev(g, "f32" if mode == "fp32_path" else "bf16", _ld(g.shape[1])) for g in Gh]
        if mode == "fp32_path":
            for l, w, g in zip(layers, Wd, Gd):
                l.galore_step(w, g, 1e-2)
        else:
            gb.Batch(layers, Wd, Gd).galore_step_batch(1e-2)
        for o, g in zip(orcs, Gh):
            o.step(np.zeros(g.shape), g, 1e-2, auto_refresh=False)
        for layer, o in zip(layers, orcs):
            assert layer.device_status() == 0
            Mc, Ma, Vc, Va = [t.cpu().numpy() for t in layer.get_q8_state()]
            assert np.array_equal(Ma, o.M_absmax) and np.array_equal(Va, o.V_absmax), (mode, s)
            assert np.array_equal(Mc, o.M_codes) and np.array_equal(Vc, o.V_codes), (mode, s)
