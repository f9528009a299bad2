"""Parity of the CUDA step (through the C ABI) with the oracle, element by element."""
import numpy as np
import pytest
import torch

from oracle import galore_oracle as go
from paper_2403_03507_b200 import binding as gb
from paper_2403_03507_b200 import workloads as wl

from gpu_util import rel_err, run_pair, to_dev, to_host

pytestmark = pytest.mark.gpu

# tolerances: updated W relative to the oracle's W, Frobenius norm, per matrix
TOL_W_F32 = 1e-4
TOL_W_BF16 = 2e-2
# on the cumulative update W_t - W_0 (W itself is dominated by W_0, so this is the informative one)
TOL_DW_F32 = 2e-3
TOL_DW_BF16_W = 0.1


def test_single_matrix_fp32_ten_steps_two_refreshes():
    # 512 x 1376 fp32, r = 128, T = 5, 10 steps: the LLaMA-60M MLP shape of the smallest workload
    w = wl.WORKLOADS["single_60m_mlp"]
    m, n, _ = w.shapes[0]
    res = run_pair(m, n, w.rank, 10, w.refresh_gap, "f32", "f32", "f32", w.spectrum_p, w.noise, w.lr, seed=w.seed,
                   check_angle=True)
    assert res["flags"] == 0
    assert len(res["infos"]) == 2
    assert max(res["w_err"]) <= TOL_W_F32, res["w_err"]
    assert max(res["dw_err"]) <= TOL_DW_F32, res["dw_err"]
    assert max(res["angles"]) <= 1e-3, (res["angles"], res["infos"])


def test_free_running_oracle_on_the_smallest_workload_is_reported():
    """Both sides refresh by themselves (the library inside galore_step, the oracle with its own SVD) and
    never exchange a projector.  Adam is element-wise, so the update depends on the basis inside the
    subspace; singular vectors inside the noise bulk are not unique, and every singular vector is
    defined up to its sign while the moments are carried across a refresh in the old coordinates.
    Up to the second refresh the two runs agree closely; after it they part (a flipped column flips
    the momentum of that component).  That difference is reported, not bounded."""
    w = wl.WORKLOADS["single_60m_mlp"]
    m, n, _ = w.shapes[0]
    cfg = gb.make_config(m, n, w.rank, alpha=w.alpha, refresh_gap=w.refresh_gap, w_dtype="f32", g_dtype="f32",
                         state_fmt="f32", auto_refresh=True, seed=w.seed)
    layer = gb.Layer(cfg)
    orc = go.GaLoreOracle(m, n, w.rank, w.alpha, w.refresh_gap, w_store="f32", state="f32")
    W0 = wl.make_weight(m, n, wl.sub_seed(w.seed, 999), "f32")
    W_orc, W_gpu = W0.copy(), to_dev(W0, "f32")
    errs = []
    for s in range(10):
        G = wl.make_gradient(m, n, wl.sub_seed(w.seed, s), w.spectrum_p, w.noise, "f32")
        layer.galore_step(W_gpu, to_dev(G, "f32"), w.lr)
        W_orc = orc.step(W_orc, G, w.lr)
        errs.append((rel_err(to_host(W_gpu), W_orc), rel_err(to_host(W_gpu) - W0, W_orc - W0)))
    print("free-running: (rel err of W, rel err of the cumulative update) per step:",
          [(f"{a:.2e}", f"{b:.2e}") for a, b in errs])
    assert layer.device_status() == 0 and layer.step_count == 10
    assert max(e[1] for e in errs[:w.refresh_gap]) < 2e-2        # same subspace, states start at zero
    assert all(np.isfinite(e[0]) and np.isfinite(e[1]) for e in errs)


@pytest.mark.parametrize("m,n,r", [(200, 333, 24), (333, 200, 24), (130, 130, 130), (64, 517, 1), (96, 96, 17)])
def test_fp32_path_ragged_shapes_both_sides(m, n, r):
    res = run_pair(m, n, r, 4, 3, "f32", "f32", "f32", seed=7)
    assert res["flags"] == 0
    assert max(res["w_err"]) <= TOL_W_F32, res["w_err"]
    assert max(res["dw_err"]) <= TOL_DW_F32, res["dw_err"]


def test_padded_leading_dimensions_and_untouched_padding():
    m, n, r = 150, 257, 16
    res = run_pair(m, n, r, 3, 5, "f32", "f32", "f32", seed=3, ldw=264, ldg=272)
    assert max(res["w_err"]) <= TOL_W_F32


@pytest.mark.parametrize("g_dtype", ["f32", "bf16"])
def test_bf16_weights(g_dtype):
    res = run_pair(256, 640, 32, 5, 4, "bf16", g_dtype, "f32", seed=5, path=gb.PATH_FP32)
    assert res["flags"] == 0
    assert max(res["w_err"]) <= TOL_W_BF16
    assert max(res["dw_err"]) <= TOL_DW_BF16_W, res["dw_err"]


@pytest.mark.parametrize("m,n,r,qb", [(128, 1100, 16, 2048), (700, 96, 8, 256), (64, 96, 8, 2048),
                                      (96, 700, 16, 512), (128, 1100, 16, 1024), (1100, 128, 16, 512)])
def test_q8_states_follow_the_oracle(m, n, r, qb):
    # several quantisation blocks plus a ragged tail block; right case included
    res = run_pair(m, n, r, 6, 10, "f32", "f32", "q8", seed=11, q_block=qb, path=gb.PATH_FP32)
    assert res["flags"] == 0
    # fp32 vs fp64 arithmetic can move a state by one code step; W stays well inside the fp32-path bar
    assert max(res["w_err"]) <= TOL_W_F32, res["w_err"]
    layer, orc = res["layer"], res["oracle"]
    Mc, Ma, Vc, Va = [t.cpu().numpy() for t in layer.get_q8_state()]
    cs, cu = go.dynamic_code(True).astype(np.float64), go.dynamic_code(False).astype(np.float64)
    assert np.mean(Mc != orc.M_codes) < 2e-3 and np.max(np.abs(cs[Mc] - cs[orc.M_codes])) <= 2 * 0.9 / 64 + 1e-6
    assert np.mean(Vc != orc.V_codes) < 2e-3 and np.max(np.abs(cu[Vc] - cu[orc.V_codes])) <= 2 * 0.9 / 128 + 1e-6
    assert np.allclose(Ma, orc.M_absmax, rtol=1e-5) and np.allclose(Va, orc.V_absmax, rtol=1e-5)
    M_gpu, V_gpu = [to_host(t) for t in layer.get_moments()]
    M_orc, V_orc = orc.moments()
    assert rel_err(M_gpu, M_orc) < 5e-3 and rel_err(V_gpu, V_orc) < 5e-3


def test_fp32_states_match_and_identity_projector_is_adam():
    # P = I injected: the CUDA path must be element-wise Adam with step lr * alpha
    m, n = 48, 80
    cfg = gb.make_config(m, n, m, refresh_gap=1000, w_dtype="f32", g_dtype="f32", auto_refresh=False)
    layer = gb.Layer(cfg)
    layer.set_projector(torch.eye(m))
    W0 = wl.make_weight(m, n, 1, "f32")
    W = to_dev(W0, "f32")
    w_ref = torch.nn.Parameter(torch.from_numpy(W0.copy()))
    opt = torch.optim.Adam([w_ref], lr=1e-2 * 0.25, betas=(0.9, 0.999), eps=1e-8)
    for s in range(5):
        G = wl.make_gradient(m, n, wl.sub_seed(2, s), 1.0, 0.01, "f32")
        layer.galore_step(W, to_dev(G, "f32"), 1e-2)
        w_ref.grad = torch.from_numpy(G)
        opt.step()
    assert rel_err(to_host(W) - W0, w_ref.detach().numpy() - W0) < 1e-5
    M, V = layer.get_moments()
    assert layer.step_count == 5 and tuple(M.shape) == (m, n)


def test_auto_refresh_equals_explicit_refresh_and_checkpoint_resume():
    m, n, r, T = 96, 160, 12, 3
    grads = [to_dev(wl.make_gradient(m, n, wl.sub_seed(4, s), 1.0, 0.01, "f32"), "f32") for s in range(7)]
    W0 = wl.make_weight(m, n, 9, "f32")

    def fresh(auto):
        return gb.Layer(gb.make_config(m, n, r, refresh_gap=T, w_dtype="f32", g_dtype="f32", auto_refresh=auto, seed=5))

    a, Wa = fresh(True), to_dev(W0, "f32")
    for g in grads:
        a.galore_step(Wa, g, 1e-2)
    b, Wb = fresh(False), to_dev(W0, "f32")
    for s, g in enumerate(grads):
        if s % T == 0:
            b.galore_refresh_projector(g)
        b.galore_step(Wb, g, 1e-2)
    assert torch.equal(Wa, Wb)
    # resume: state buffer + step counter are the whole checkpoint
    c, Wc = fresh(True), to_dev(W0, "f32")
    for g in grads[:4]:
        c.galore_step(Wc, g, 1e-2)
    torch.cuda.synchronize()
    saved_state, saved_k, saved_W = c.state.clone(), c.step_count, Wc.clone()
    d = fresh(True)
    d.state.copy_(saved_state)
    d.step_count = saved_k
    d.set_projector(c.get_projector())
    Wd = saved_W.clone()
    for g in grads[4:]:
        d.galore_step(Wd, g, 1e-2)
    assert torch.equal(Wd, Wa)


def test_step_without_projector_is_an_error_and_nonfinite_is_latched():
    cfg = gb.make_config(32, 48, 4, w_dtype="f32", g_dtype="f32", auto_refresh=False)
    layer = gb.Layer(cfg)
    W = torch.zeros(32, 48, device="cuda")
    G = torch.ones(32, 48, device="cuda")
    with pytest.raises(gb.GaloreError) as e:
        layer.galore_step(W, G, 1e-2)
    assert e.value.status == gb.ERR_STATE
    layer.set_projector(torch.eye(32)[:, :4])
    G[0, 0] = float("inf")
    layer.galore_step(W, G, 1e-2)
    assert layer.device_status() & gb.DEV_NONFINITE
    assert layer.device_status() == 0          # reading clears the word


def test_full_size_matrix_of_the_1b_workload_sampled():
    # one 2048 x 5461 matrix at r = 512, padded leading dimension, checked against the oracle's full step
    w = wl.WORKLOADS["llama_1b_q8"]
    m, n, r = 2048, 5461, w.rank
    G = wl.make_gradient(m, n, wl.sub_seed(w.seed, 0), w.spectrum_p, w.noise, "bf16")
    W0 = wl.make_weight(m, n, 3, "bf16")
    rng = np.random.default_rng(0)
    P = wl.round_to(wl.random_orthonormal(m, r, rng), "bf16")
    for state_fmt in ("f32", "q8"):
        cfg = gb.make_config(m, n, r, refresh_gap=200, state_fmt=state_fmt, auto_refresh=False)
        layer = gb.Layer(cfg)
        layer.set_projector(torch.from_numpy(P))
        orc = go.GaLoreOracle(m, n, r, 0.25, 200, w_store="bf16", state=state_fmt,
                              n_store="bf16" if layer.uses_tensor_path else "f64")
        orc.set_projector(P)
        Wg = to_dev(W0, "bf16", ld=5464)
        Gg = to_dev(G, "bf16", ld=5464)
        Wo = W0
        for s in range(2):
            layer.galore_step(Wg, Gg, 1e-2)
            Wo = orc.step(Wo, G, 1e-2, auto_refresh=False)
        assert layer.device_status() == 0
        assert rel_err(to_host(Wg), Wo) <= TOL_W_BF16
        assert rel_err(to_host(Wg) - W0, Wo - W0) <= TOL_DW_BF16_W


@pytest.mark.parametrize("w_dtype,g_dtype,state_fmt,path", [("f32", "f32", "f32", gb.PATH_FP32), ("bf16", "bf16", "q8", gb.PATH_AUTO),
                                                            ("bf16", "bf16", "f32", gb.PATH_AUTO)])
def test_decoupled_weight_decay_matches_the_oracle(w_dtype, g_dtype, state_fmt, path):
    """GaLore-AdamW: W <- W (1 - lr lambda) - lr alpha P N, the decay folded into the pass that applies the update."""
    m, n, r = (256, 640, 32) if w_dtype == "bf16" else (200, 333, 24)
    res = run_pair(m, n, r, 6, 4, w_dtype, g_dtype, state_fmt, seed=13, path=path, weight_decay=0.1, lr=2e-2,
                   ldw=(n + 7) // 8 * 8, ldg=(n + 7) // 8 * 8, q_block=256)
    assert res["flags"] == 0
    tol_w, tol_dw = (TOL_W_F32, TOL_DW_F32) if w_dtype == "f32" else (TOL_W_BF16, TOL_DW_BF16_W)
    assert max(res["w_err"]) <= tol_w, res["w_err"]
    assert max(res["dw_err"]) <= tol_dw, res["dw_err"]
    # the decay is really there: without it W would be elsewhere by about 6 steps of lr * lambda
    res0 = run_pair(m, n, r, 6, 4, w_dtype, g_dtype, state_fmt, seed=13, path=path, weight_decay=0.0, lr=2e-2,
                    ldw=(n + 7) // 8 * 8, ldg=(n + 7) // 8 * 8, q_block=256)
    assert rel_err(res["W_gpu"], res0["W_gpu"]) > 5e-3
