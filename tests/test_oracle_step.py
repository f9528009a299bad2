"""Pins for the oracle's reading of Algorithm 1 against what the paper and mathematics fix."""
import numpy as np
import pytest
import torch

from oracle import galore_oracle as go
from paper_2403_03507_b200 import workloads as wl

HP = dict(alpha=0.25, refresh_gap=5, beta1=0.9, beta2=0.999, eps=1e-8)


def _grads(m, n, steps, seed=0):
    return [wl.make_gradient(m, n, wl.sub_seed(seed, s), 1.0, 0.01, "f64") for s in range(steps)]


def _torch_adam(W0, grads, lr, beta1, beta2, eps):
    """Element-wise Adam as implemented by the library optimiser (an independent implementation)."""
    w = torch.nn.Parameter(torch.from_numpy(W0.copy()))
    opt = torch.optim.Adam([w], lr=lr, betas=(beta1, beta2), eps=eps)
    out = []
    for g in grads:
        w.grad = torch.from_numpy(np.ascontiguousarray(g))
        opt.step()
        out.append(w.detach().numpy().copy())
    return out


def test_identity_projector_with_weight_decay_is_library_adamw():
    """GaLore-AdamW with P = I and alpha = 1 is element-wise AdamW (decoupled decay, an independent implementation)."""
    m, n = 10, 16
    W = wl.make_weight(m, n, 2, "f64")
    grads = _grads(m, n, 6, seed=3)
    lr, wd = 3e-2, 0.2
    orc = go.GaLoreOracle(m, n, m, alpha=1.0, refresh_gap=100, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=wd)
    orc.set_projector(np.eye(m))
    w = torch.nn.Parameter(torch.from_numpy(W.copy()))
    opt = torch.optim.AdamW([w], lr=lr, betas=(0.9, 0.999), eps=1e-8, weight_decay=wd)
    for g in grads:
        W = orc.step(W, g, lr, auto_refresh=False)
        w.grad = torch.from_numpy(np.ascontiguousarray(g))
        opt.step()
        assert np.allclose(W, w.detach().numpy(), rtol=1e-12, atol=1e-14)
    # the decay acts on W alone: with zero gradients W shrinks geometrically and the moments stay zero
    orc2 = go.GaLoreOracle(m, n, 4, alpha=0.25, refresh_gap=100, weight_decay=wd)
    orc2.set_projector(np.linalg.qr(np.random.default_rng(0).standard_normal((m, 4)))[0])
    W2 = wl.make_weight(m, n, 5, "f64")
    W3 = orc2.step(orc2.step(W2, np.zeros((m, n)), lr, auto_refresh=False), np.zeros((m, n)), lr, auto_refresh=False)
    assert np.allclose(W3, W2 * (1 - lr * wd) ** 2, rtol=1e-14)


def test_identity_projector_is_elementwise_adam():
    m, n = 12, 20
    W = wl.make_weight(m, n, 1, "f64")
    grads = _grads(m, n, 7)
    orc = go.GaLoreOracle(m, n, m, **HP)
    orc.set_projector(np.eye(m))
    ref = _torch_adam(W, grads, 1e-2 * HP["alpha"], 0.9, 0.999, 1e-8)
    for g, w_ref in zip(grads, ref):
        W = orc.step(W, g, 1e-2, auto_refresh=False)
        assert np.allclose(W, w_ref, rtol=0, atol=1e-13)


def test_signed_permutation_projector_is_elementwise_adam():
    m, n = 10, 16
    rng = np.random.default_rng(2)
    perm = rng.permutation(m)
    P = np.zeros((m, m))
    P[perm, np.arange(m)] = rng.choice([-1.0, 1.0], size=m)
    W = wl.make_weight(m, n, 1, "f64")
    grads = _grads(m, n, 5)
    orc = go.GaLoreOracle(m, n, m, **HP)
    orc.set_projector(P)
    ref = _torch_adam(W, grads, 1e-2 * HP["alpha"], 0.9, 0.999, 1e-8)
    for g, w_ref in zip(grads, ref):
        W = orc.step(W, g, 1e-2, auto_refresh=False)
    assert np.allclose(W, ref[-1], atol=1e-13)


@pytest.mark.parametrize("m,n", [(14, 22), (22, 14)])
def test_square_orthonormal_projector_is_adam_in_rotated_coordinates(m, n):
    # P square orthonormal: P^T W_t (left) / W_t Q (right) follows element-wise Adam on the rotated gradients
    d = min(m, n)
    rng = np.random.default_rng(3)
    P = wl.random_orthonormal(d, d, rng)
    W0 = wl.make_weight(m, n, 4, "f64")
    grads = _grads(m, n, 6)
    orc = go.GaLoreOracle(m, n, d, **HP)
    orc.set_projector(P)
    left = m <= n
    rot = (lambda X: P.T @ X) if left else (lambda X: X @ P)
    ref = _torch_adam(rot(W0), [rot(g) for g in grads], 1e-2 * HP["alpha"], 0.9, 0.999, 1e-8)
    W = W0
    for g in grads:
        W = orc.step(W, g, 1e-2, auto_refresh=False)
    assert np.allclose(rot(W), ref[-1], atol=1e-12)


def test_first_step_closed_form():
    # zero-initialised moments and t = 1: N = R / (|R| + eps)
    m, n, r = 16, 28, 5
    W0 = wl.make_weight(m, n, 1, "f64")
    G = _grads(m, n, 1)[0]
    orc = go.GaLoreOracle(m, n, r, **HP)
    W1 = orc.step(W0, G, 3e-3)
    P = orc.proj
    R = P.T @ G
    expect = W0 - 3e-3 * 0.25 * P @ (R / (np.abs(R) + 1e-8))
    assert np.allclose(W1, expect, atol=1e-13)


def test_full_rank_identity_regulariser_returns_gradient():
    # r = min(m, n), rho = 1: the projected-back update equals alpha * G
    for m, n in [(9, 15), (15, 9)]:
        W0 = wl.make_weight(m, n, 1, "f64")
        G = _grads(m, n, 1)[0]
        orc = go.GaLoreOracle(m, n, min(m, n), inner="identity", **HP)
        W1 = orc.step(W0, G, 0.1)
        assert np.allclose(W1, W0 - 0.1 * 0.25 * G, atol=1e-13)


def test_update_stays_in_span_of_projector_between_refreshes():
    m, n, r = 20, 36, 4
    W = wl.make_weight(m, n, 1, "f64")
    orc = go.GaLoreOracle(m, n, r, **HP)
    for s, g in enumerate(_grads(m, n, 5)):
        W_new = orc.step(W, g, 1e-2)
        dW = W_new - W
        P = orc.proj
        assert np.linalg.norm(dW - P @ (P.T @ dW)) < 1e-13
        assert np.linalg.matrix_rank(dW, tol=1e-10) <= r
        W = W_new
    # right case: rows of dW lie in span(Q)
    orc = go.GaLoreOracle(n, m, r, **HP)
    W = wl.make_weight(n, m, 1, "f64")
    W_new = orc.step(W, _grads(n, m, 1)[0], 1e-2)
    Q = orc.proj
    dW = W_new - W
    assert np.linalg.norm(dW - (dW @ Q) @ Q.T) < 1e-13


def test_gradient_scale_invariance():
    m, n, r = 16, 24, 4
    W0 = wl.make_weight(m, n, 1, "f64")
    grads = _grads(m, n, 4)
    c = 64.0                                      # power of two: scaling is exact
    a = go.GaLoreOracle(m, n, r, **HP)
    hp = dict(HP, eps=HP["eps"] * c)
    b = go.GaLoreOracle(m, n, r, **hp)
    Wa, Wb = W0, W0
    for g in grads:
        Wa = a.step(Wa, g, 1e-2)
        Wb = b.step(Wb, c * g, 1e-2)
    assert np.allclose(Wa, Wb, atol=1e-12)


def test_projector_column_signs_are_immaterial():
    m, n, r = 16, 24, 6
    W0 = wl.make_weight(m, n, 1, "f64")
    grads = _grads(m, n, 3)
    P, _ = go.top_r_projector(grads[0], r, "left")
    flip = np.array([1, -1, -1, 1, -1, 1.0])
    a = go.GaLoreOracle(m, n, r, **HP); a.set_projector(P)
    b = go.GaLoreOracle(m, n, r, **HP); b.set_projector(P * flip)
    Wa, Wb = W0, W0
    for g in grads:
        Wa = a.step(Wa, g, 1e-2, auto_refresh=False)
        Wb = b.step(Wb, g, 1e-2, auto_refresh=False)
    assert np.allclose(Wa, Wb, atol=1e-14)


def test_right_case_is_left_case_of_the_transposed_problem():
    m, n, r = 30, 18, 5
    W0 = wl.make_weight(m, n, 1, "f64")
    grads = _grads(m, n, 6)
    a = go.GaLoreOracle(m, n, r, **HP)
    b = go.GaLoreOracle(n, m, r, **HP)
    assert a.side == "right" and b.side == "left"
    assert a.state_shape == (m, r) and b.state_shape == (r, m)
    Wa, Wb = W0, W0.T.copy()
    for g in grads:
        Wa = a.step(Wa, g, 1e-2)
        Wb = b.step(Wb, g.T.copy(), 1e-2)
        # singular vectors are unique up to sign here, and signs are immaterial
        assert np.allclose(Wa, Wb.T, atol=1e-10)


def test_refresh_schedule_and_side_choice():
    # T = 5 and 10 steps: refreshes exactly at k = 0 and k = 5; m == n goes left
    m = n = 12
    orc = go.GaLoreOracle(m, n, 3, **HP)
    assert orc.side == "left"
    W = wl.make_weight(m, n, 1, "f64")
    seen = []
    for s, g in enumerate(_grads(m, n, 10)):
        before = orc.refreshes
        W = orc.step(W, g, 1e-2)
        if orc.refreshes != before:
            seen.append(s)
    assert seen == [0, 5]
    assert go.GaLoreOracle(5, 9, 2, **HP).side == "left"
    assert go.GaLoreOracle(9, 5, 2, **HP).side == "right"


def test_moments_survive_a_refresh_unchanged():
    m, n, r = 12, 20, 3
    orc = go.GaLoreOracle(m, n, r, **HP)
    W = wl.make_weight(m, n, 1, "f64")
    grads = _grads(m, n, 6)
    for g in grads[:5]:
        W = orc.step(W, g, 1e-2)
    M5, V5 = orc.M.copy(), orc.V.copy()
    W = orc.step(W, grads[5], 1e-2)               # k = 5: refresh happens here
    assert orc.refreshes == 2
    R = orc.proj.T @ grads[5]
    assert np.allclose(orc.M, 0.9 * M5 + 0.1 * R, atol=1e-15)
    assert np.allclose(orc.V, 0.999 * V5 + 0.001 * R * R, atol=1e-15)


def test_memory_model():
    # optimizer state of GaLore: m r + 2 n r elements for m <= n (Table 1)
    m, n, r = 512, 1376, 128
    assert go.GaLoreOracle(m, n, r, **HP).optimizer_state_elements() == m * r + 2 * n * r
    assert go.GaLoreOracle(n, m, r, **HP).optimizer_state_elements() == m * r + 2 * n * r


def test_rank_bounds():
    with pytest.raises(ValueError):
        go.GaLoreOracle(8, 12, 9, **HP)
    go.GaLoreOracle(8, 12, 8, **HP)


def test_storage_rounding_helpers_match_library_conversion():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(4096) * 10.0 ** rng.integers(-6, 6, 4096),
                        [0.0, 1.0, -1.0, 1.00390625, 1.01171875, 3.0e-5]])   # includes exact ties
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(go.round_bf16(x), ref)
    assert np.array_equal(go.round_f32(x), x.astype(np.float32).astype(np.float64))


def test_bf16_weight_storage_rounds_each_write():
    m, n, r = 16, 24, 4
    W0 = wl.make_weight(m, n, 1, "bf16")
    G = _grads(m, n, 1)[0]
    a = go.GaLoreOracle(m, n, r, **HP)
    b = go.GaLoreOracle(m, n, r, w_store="bf16", **HP)
    Wa, Wb = a.step(W0, G, 1e-2), b.step(W0, G, 1e-2)
    assert np.array_equal(Wb, go.round_bf16(Wa))
