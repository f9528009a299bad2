"""galore_step_batch must give the same result as stepping each layer with galore_step."""
import numpy as np
import pytest
import torch

from oracle import galore_oracle as go
from paper_2403_03507_b200 import binding as gb
from paper_2403_03507_b200 import workloads as wl

from gpu_util import rel_err, to_dev, to_host

pytestmark = pytest.mark.gpu

SHAPES = [(256, 512, 64), (512, 256, 64), (384, 1000, 128), (1000, 384, 128), (640, 640, 64), (200, 304, 16),
          (256, 1096, 64), (130, 2056, 8)]


def _make(state_fmt, w_dtype, path=gb.PATH_AUTO, g_dtype="bf16"):
    layers, Ws, Gs, Ps, W0s, Gh = [], [], [], [], [], []
    for i, (m, n, r) in enumerate(SHAPES):
        cfg = gb.make_config(m, n, r, refresh_gap=1000, w_dtype=w_dtype, g_dtype=g_dtype, state_fmt=state_fmt,
                             auto_refresh=False, path=path, q_block=256)
        layer = gb.Layer(cfg)
        d = m if layer.side == gb.SIDE_LEFT else n
        P = wl.round_to(wl.random_orthonormal(d, r, np.random.default_rng(i)), g_dtype)
        layer.set_projector(torch.from_numpy(P))
        ld = (n + 7) // 8 * 8
        W0 = wl.make_weight(m, n, 100 + i, w_dtype)
        layers.append(layer)
        Ps.append(P)
        W0s.append(W0)
        Ws.append(to_dev(W0, w_dtype, ld))
    return layers, Ws, Ps, W0s


def _grads(step, g_dtype="bf16"):
    host = [wl.make_gradient(m, n, wl.sub_seed(7, i, step), 0.8, 0.05, g_dtype) for i, (m, n, r) in enumerate(SHAPES)]
    dev = [to_dev(g, g_dtype, (g.shape[1] + 7) // 8 * 8) for g in host]
    return host, dev


@pytest.mark.parametrize("state_fmt,w_dtype", [("f32", "bf16"), ("q8", "bf16"), ("f32", "f32")])
def test_batch_equals_per_layer_steps(state_fmt, w_dtype):
    # The two modes slice K differently, so fp32 sums differ in the last bits; a bf16 rounding of N or
    # of W that sits on a boundary may then flip (one bf16 ulp = 4e-3 of that element, on few elements).
    tol = 5e-4 if w_dtype == "bf16" else 1e-5
    la, Wa, _, _ = _make(state_fmt, w_dtype)
    lb, Wb, _, _ = _make(state_fmt, w_dtype)
    assert all(l.uses_tensor_path for l in la)
    batch = None
    for s in range(3):
        _, G = _grads(s)
        for l, w, g in zip(la, Wa, G):
            l.galore_step(w, g, 1e-2)
        if batch is None:
            batch = gb.Batch(lb, Wb, G)
        else:
            batch.rebind(Wb, G)
        batch.galore_step_batch(1e-2)
    torch.cuda.synchronize()
    for l1, l2, w1, w2 in zip(la, lb, Wa, Wb):
        assert l2.step_count == 3 and l2.device_status() == 0
        assert rel_err(to_host(w2), to_host(w1)) < tol
        M1, V1 = l1.get_moments()
        M2, V2 = l2.get_moments()
        if state_fmt == "q8":   # a state on a threshold may land one code step apart
            assert rel_err(to_host(M2), to_host(M1)) < 5e-3 and rel_err(to_host(V2), to_host(V1)) < 5e-3
        else:
            assert torch.allclose(M1, M2, rtol=1e-3, atol=1e-6) and torch.allclose(V1, V2, rtol=1e-3, atol=1e-9)


def test_batch_matches_the_oracle():
    layers, Ws, Ps, W0s = _make("q8", "bf16")
    orcs = []
    for (m, n, r), P in zip(SHAPES, Ps):
        o = go.GaLoreOracle(m, n, r, 0.25, 1000, w_store="bf16", state="q8", q_block=256, n_store="bf16")
        o.set_projector(P)
        orcs.append(o)
    Wo = list(W0s)
    batch = None
    for s in range(3):
        Gh, Gd = _grads(s)
        if batch is None:
            batch = gb.Batch(layers, Ws, Gd)
        else:
            batch.rebind(Ws, Gd)
        batch.galore_step_batch(1e-2)
        Wo = [o.step(w, g, 1e-2, auto_refresh=False) for o, w, g in zip(orcs, Wo, Gh)]
    for w_gpu, w_orc, w0 in zip(Ws, Wo, W0s):
        assert rel_err(to_host(w_gpu), w_orc) <= 2e-2
        assert rel_err(to_host(w_gpu) - w0, w_orc - w0) <= 5e-2


def test_small_workspace_only_makes_groups_smaller_and_mixed_paths_work():
    la, Wa, _, _ = _make("f32", "bf16")
    lb, Wb, _, _ = _make("f32", "bf16")
    _, G = _grads(0)
    full = gb.galore_batch_query_bytes(la)
    gb.Batch(la, Wa, G).galore_step_batch(1e-2)
    gb.Batch(lb, Wb, G, workspace_bytes=full // 5).galore_step_batch(1e-2)      # several groups, maybe single steps
    for w1, w2 in zip(Wa, Wb):
        assert rel_err(to_host(w2), to_host(w1)) < 5e-4
    # fp32 layers (not on the tensor path) inside a batch run the same three phases as grouped launches of the
    # FMA kernels; with many layers in flight K is not sliced, so sums differ from single steps in their order only
    lc, Wc, _, _ = _make("f32", "f32", path=gb.PATH_FP32, g_dtype="f32")
    ld_, Wd, _, _ = _make("f32", "f32", path=gb.PATH_FP32, g_dtype="f32")
    _, G32 = _grads(0, "f32")
    before = gb.galore_launch_count()
    gb.Batch(lc, Wc, G32).galore_step_batch(1e-2)
    grouped = gb.galore_launch_count() - before
    for l, w, g in zip(ld_, Wd, G32):
        l.galore_step(w, g, 1e-2)
    assert grouped < gb.galore_launch_count() - before - grouped          # fewer launches than one step per layer
    for w1, w2 in zip(Wc, Wd):
        assert rel_err(to_host(w1), to_host(w2)) < 2e-5      # first step: N is close to sign(R), and R near zero may change sign with the order of the sum
    assert all(l.step_count == 1 for l in lc)


def test_auto_refresh_inside_a_batch():
    m, n, r = 256, 512, 32
    cfgs = [gb.make_config(m, n, r, refresh_gap=2, auto_refresh=True, seed=3) for _ in range(4)]
    la = [gb.Layer(c) for c in cfgs]
    lb = [gb.Layer(c) for c in cfgs]
    W0 = wl.make_weight(m, n, 1, "bf16")
    Wa = [to_dev(W0, "bf16") for _ in la]
    Wb = [to_dev(W0, "bf16") for _ in lb]
    for s in range(3):
        G = [to_dev(wl.make_gradient(m, n, wl.sub_seed(5, i, s), 0.8, 0.05, "bf16"), "bf16") for i in range(4)]
        for l, w, g in zip(la, Wa, G):
            l.galore_step(w, g, 1e-2)
        gb.Batch(lb, Wb, G).galore_step_batch(1e-2)
    for w1, w2 in zip(Wa, Wb):
        assert rel_err(to_host(w2), to_host(w1)) < 5e-4


def test_refresh_batch_matches_single_refreshes():
    """galore_refresh_batch over a shared workspace gives the projectors of one-by-one refreshes.

    The refresh is deterministic for a given seed, so the two agree to rounding of the stored dtype;
    both are also checked against the oracle's subspace for a gapped spectrum.
    """
    shapes = [(256, 512, 32), (512, 256, 32), (384, 1000, 64), (640, 640, 64), (256, 1096, 64), (200, 304, 16)]
    single, batched, Gs = [], [], []
    for i, (m, n, r) in enumerate(shapes):
        k = min(m, n)
        spectrum = np.concatenate([np.linspace(2.0, 1.0, r), 0.2 * np.arange(1, k - r + 1, dtype=np.float64) ** -0.5])
        G, U, V = wl.make_planted(m, n, 50 + i, spectrum, "bf16")
        Gs.append(to_dev(G, "bf16", (n + 7) // 8 * 8))
        for dst in (single, batched):
            cfg = gb.make_config(m, n, r, auto_refresh=False, p_dtype="f32", seed=11 + i)
            dst.append(gb.Layer(cfg))
    for layer, G in zip(single, Gs):
        st, _info = layer.galore_refresh_projector(G)
        assert st == 0
    st, infos = gb.galore_refresh_batch(batched, Gs)
    assert st == 0 and len(infos) == len(shapes)
    for (m, n, r), a, b_, G, info in zip(shapes, single, batched, Gs, infos):
        Pa, Pb = a.get_projector().double().cpu().numpy(), b_.get_projector().double().cpu().numpy()
        assert info.converged == 1
        assert np.abs(Pa - Pb).max() < 1e-6
        Gh = to_host(G)[:, :n]
        side = "left" if m <= n else "right"
        Po, _sv = go.top_r_projector(Gh, r, side, method="lapack")
        assert go.largest_principal_angle(Po, Pb) < 1e-3


def test_full_size_7b_matrices_in_the_benched_configuration():
    """Two 4096 x 11008 matrices (and their transposed shape) at rank 1024 with 8-bit states, stepped by
    galore_step_batch exactly as bench.py does (CTA-pair GEMMs, grouped launches), against the oracle."""
    w = wl.WORKLOADS["llama_7b_q8"]
    r = w.rank
    shapes = [(4096, 11008), (11008, 4096)]
    layers, Ws, Gd, orcs, W0s, Gh = [], [], [], [], [], []
    for i, (m, n) in enumerate(shapes):
        G = wl.make_gradient(m, n, wl.sub_seed(w.seed, i), w.spectrum_p, w.noise, "bf16")
        W0 = wl.make_weight(m, n, 40 + i, "bf16")
        d = min(m, n)
        P = wl.round_to(wl.random_orthonormal(d, r, np.random.default_rng(i)), "bf16")
        cfg = gb.make_config(m, n, r, alpha=w.alpha, refresh_gap=w.refresh_gap, state_fmt="q8", q_block=w.q_block,
                             auto_refresh=False)
        layer = gb.Layer(cfg)
        assert layer.uses_tensor_path
        layer.set_projector(torch.from_numpy(P))
        o = go.GaLoreOracle(m, n, r, w.alpha, w.refresh_gap, w_store="bf16", state="q8", q_block=w.q_block, n_store="bf16")
        o.set_projector(P)
        ld = (n + 15) // 16 * 16
        layers.append(layer); orcs.append(o); W0s.append(W0); Gh.append(G)
        Ws.append(to_dev(W0, "bf16", ld)); Gd.append(to_dev(G, "bf16", ld))
    batch = gb.Batch(layers, Ws, Gd)
    Wo = list(W0s)
    for s in range(2):
        batch.galore_step_batch(w.lr)
        Wo = [o.step(x, g, w.lr, auto_refresh=False) for o, x, g in zip(orcs, Wo, Gh)]
    for layer, w_gpu, w_orc, w0, o in zip(layers, Ws, Wo, W0s, orcs):
        assert layer.device_status() == 0 and layer.step_count == 2
        assert rel_err(to_host(w_gpu), w_orc) <= 2e-2
        assert rel_err(to_host(w_gpu) - w0, w_orc - w0) <= 5e-2
        M, V = layer.get_moments()
        Mo, Vo = o.moments()
        assert rel_err(to_host(M), Mo) < 2e-2 and rel_err(to_host(V), Vo) < 2e-2
        # the stored codes themselves: fp32 against fp64 arithmetic may move a value on a threshold to
        # the neighbouring code, never further
        Mc, _Ma, Vc, _Va = [t.cpu().numpy() for t in layer.get_q8_state()]
        cs, cu = go.dynamic_code(True).astype(np.float64), go.dynamic_code(False).astype(np.float64)
        assert np.mean(Mc != o.M_codes) < 2e-3 and np.max(np.abs(cs[Mc] - cs[o.M_codes])) <= 2 * 0.9 / 64 + 1e-6
        assert np.mean(Vc != o.V_codes) < 2e-3 and np.max(np.abs(cu[Vc] - cu[o.V_codes])) <= 2 * 0.9 / 128 + 1e-6


@pytest.mark.parametrize("slots", [1, 3])
def test_host_resident_batch_equals_device_steps(slots):
    """galore_step_host_batch (W and G in pinned host memory, staged through `slots` device buffers) leaves
    the same W as galore_step on device tensors with the same row pitch."""
    layers_h, Wh, _, W0s = _make("q8", "bf16")
    layers_d, Wd, _, _ = _make("q8", "bf16")
    Wd = [to_dev(w0, "bf16", (w0.shape[1] + 15) // 16 * 16) for w0 in W0s]
    W_host = [torch.from_numpy(np.ascontiguousarray(w0)).to(torch.bfloat16).pin_memory() for w0 in W0s]
    hb = None
    for s in range(3):
        Gh, _ = _grads(s)
        G_host = [torch.from_numpy(np.ascontiguousarray(g)).to(torch.bfloat16).pin_memory() for g in Gh]
        if hb is None:
            hb = gb.HostBatch(layers_h, W_host, G_host, slots=slots)
        else:
            hb.rebind(W_host, G_host)
        hb.galore_step_host_batch(1e-2)
        torch.cuda.synchronize()
        for l, w, g in zip(layers_d, Wd, Gh):
            l.galore_step(w, to_dev(g, "bf16", (g.shape[1] + 15) // 16 * 16), 1e-2)
    torch.cuda.synchronize()
    for l, wh, wd in zip(layers_h, W_host, Wd):
        assert l.step_count == 3 and l.device_status() == 0
        assert torch.equal(wh, wd.cpu())


def test_batch_with_weight_decay_equals_per_layer_steps_and_the_oracle():
    shapes = [(256, 512, 64), (512, 256, 64), (384, 1000, 128)]
    la, lb, Wa, Wb, orcs, Wo, W0s = [], [], [], [], [], [], []
    for i, (m, n, r) in enumerate(shapes):
        P = wl.round_to(wl.random_orthonormal(min(m, n), r, np.random.default_rng(i)), "bf16")
        W0 = wl.make_weight(m, n, 60 + i, "bf16")
        for ls, Ws in ((la, Wa), (lb, Wb)):
            cfg = gb.make_config(m, n, r, state_fmt="q8", q_block=256, auto_refresh=False, weight_decay=0.05)
            layer = gb.Layer(cfg)
            layer.set_projector(torch.from_numpy(P))
            ls.append(layer)
            Ws.append(to_dev(W0, "bf16", (n + 7) // 8 * 8))
        o = go.GaLoreOracle(m, n, r, 0.25, 1000, w_store="bf16", state="q8", q_block=256, n_store="bf16", weight_decay=0.05)
        o.set_projector(P)
        orcs.append(o); Wo.append(W0); W0s.append(W0)
    batch = None
    for s in range(3):
        Gh = [wl.make_gradient(m, n, wl.sub_seed(17, i, s), 0.8, 0.05, "bf16") for i, (m, n, r) in enumerate(shapes)]
        Gd = [to_dev(g, "bf16", (g.shape[1] + 7) // 8 * 8) for g in Gh]
        for l, w, g in zip(la, Wa, Gd):
            l.galore_step(w, g, 2e-2)
        if batch is None:
            batch = gb.Batch(lb, Wb, Gd)
        else:
            batch.rebind(Wb, Gd)
        batch.galore_step_batch(2e-2)
        Wo = [o.step(w, g, 2e-2, auto_refresh=False) for o, w, g in zip(orcs, Wo, Gh)]
    for w1, w2, wo, w0 in zip(Wa, Wb, Wo, W0s):
        assert rel_err(to_host(w2), to_host(w1)) < 5e-4
        assert rel_err(to_host(w2), wo) <= 2e-2
        assert rel_err(to_host(w2) - w0, wo - w0) <= 5e-2
