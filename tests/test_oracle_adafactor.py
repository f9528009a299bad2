"""Pins of the oracle's Adafactor regulariser (Sec. "GaLore with memory-efficient optimizers" names Adafactor
with first-order statistics and prints no formulas: the update is the published algorithm, pinned here against
an independent implementation of it, a closed form and brute force)."""
import math

import numpy as np
import pytest
import torch

from oracle import galore_oracle as go


def _hf_adafactor():
    try:
        from transformers.optimization import Adafactor
    except Exception as e:                                   # pragma: no cover
        pytest.skip(f"transformers' Adafactor not importable: {e}")
    return Adafactor


@pytest.mark.parametrize("m,n", [(6, 9), (12, 5)])
def test_identity_projector_reduces_to_the_library_adafactor(m, n):
    """P = I (rank = min(m, n), alpha = 1): GaLore-Adafactor is Adafactor on the full gradient.  The library
    routine (fp32) runs with an external constant learning rate, momentum 0.9, decay -0.8, clipping at 1."""
    Adafactor = _hf_adafactor()
    rng = np.random.default_rng(5)
    r = min(m, n)
    W0 = rng.standard_normal((m, n))
    orc = go.GaLoreOracle(m, n, r, 1.0, 1000, beta1=0.9, inner="adafactor")
    orc.set_projector(np.eye(r))
    p = torch.nn.Parameter(torch.tensor(W0, dtype=torch.float32))
    opt = Adafactor([p], lr=1e-2, eps=(1e-30, 1e-3), clip_threshold=1.0, decay_rate=-0.8, beta1=0.9, weight_decay=0.0,
                    scale_parameter=False, relative_step=False, warmup_init=False)
    W = W0.astype(np.float32).astype(np.float64)
    for s in range(6):
        G = rng.standard_normal((m, n)) * (1.0 + s)
        p.grad = torch.tensor(G, dtype=torch.float32)
        opt.step()
        W = orc.step(W, G.astype(np.float32).astype(np.float64), 1e-2, auto_refresh=False)
        assert np.abs(p.detach().numpy().astype(np.float64) - W).max() < 5e-6, s


def test_first_step_on_a_rank_one_magnitude_pattern_is_the_sign():
    """t = 1: beta2_1 = 0, so the factors are the row and column means of R^2.  If |R| = a b^T they reproduce
    R^2 exactly: U = sign(R), its rms is 1 (no clipping), and the step is lr alpha (1 - beta1) P sign(R)."""
    rng = np.random.default_rng(2)
    m, n, r = 7, 11, 4
    a, b = rng.uniform(0.5, 2.0, r), rng.uniform(0.5, 2.0, n)
    sign = rng.choice([-1.0, 1.0], (r, n))
    R = sign * np.outer(a, b)
    P, _ = np.linalg.qr(rng.standard_normal((m, r)))
    G = P @ R
    orc = go.GaLoreOracle(m, n, r, 0.25, 1000, beta1=0.9, inner="adafactor")
    orc.set_projector(P)
    W0 = rng.standard_normal((m, n))
    W1 = orc.step(W0, G, 1e-2, auto_refresh=False)
    assert np.abs(W1 - (W0 - 1e-2 * 0.25 * 0.1 * (P @ sign))).max() < 1e-12


def test_factored_second_moment_by_brute_force():
    """Two steps written with plain loops: running row / column means with beta2_t = 1 - t^-0.8, the outer
    product over the mean of the row factor, clipping by the rms, momentum."""
    rng = np.random.default_rng(9)
    rows, cols, beta1 = 3, 5, 0.8
    M = [[0.0] * cols for _ in range(rows)]
    vr, vc = [0.0] * rows, [0.0] * cols
    M_o, vr_o, vc_o = np.zeros((rows, cols)), np.zeros(rows), np.zeros(cols)
    for t in (1, 2, 3):
        R = rng.standard_normal((rows, cols)) * (3.0 if t == 2 else 0.5)     # t = 2 is clipped, the others are not all
        b2 = 1.0 - t ** -0.8
        for i in range(rows):
            vr[i] = b2 * vr[i] + (1 - b2) * sum(R[i][j] ** 2 + 1e-30 for j in range(cols)) / cols
        for j in range(cols):
            vc[j] = b2 * vc[j] + (1 - b2) * sum(R[i][j] ** 2 + 1e-30 for i in range(rows)) / rows
        mean_r = sum(vr) / rows
        U = [[R[i][j] / math.sqrt(vr[i] * vc[j] / mean_r) for j in range(cols)] for i in range(rows)]
        rms = math.sqrt(sum(u * u for row in U for u in row) / (rows * cols))
        div = max(1.0, rms)
        for i in range(rows):
            for j in range(cols):
                M[i][j] = beta1 * M[i][j] + (1 - beta1) * U[i][j] / div
        N_o, vr_o, vc_o = go.adafactor_update(R, M_o, vr_o, vc_o, t, beta1)
        M_o = N_o
        assert np.abs(np.array(M) - M_o).max() < 1e-13
        assert np.abs(np.array(vr) - vr_o).max() < 1e-14 and np.abs(np.array(vc) - vc_o).max() < 1e-14


def test_update_is_clipped_and_scale_free_at_the_first_step():
    rng = np.random.default_rng(4)
    R = rng.standard_normal((8, 20)) * np.exp(rng.standard_normal((8, 20)))       # far from a rank-one pattern
    N1, _, _ = go.adafactor_update(R, np.zeros_like(R), np.zeros(8), np.zeros(20), 1, 0.0)
    N2, _, _ = go.adafactor_update(1e3 * R, np.zeros_like(R), np.zeros(8), np.zeros(20), 1, 0.0)
    assert np.sqrt(np.mean(N1 * N1)) <= 1.0 + 1e-12
    assert np.abs(N1 - N2).max() < 1e-12


def test_state_elements_and_the_8_bit_refusal():
    orc = go.GaLoreOracle(64, 96, 16, 0.25, 10, inner="adafactor")
    assert orc.optimizer_state_elements() == 64 * 16 + 16 * 96 + 16 + 96
    with pytest.raises(ValueError):
        go.GaLoreOracle(64, 96, 16, 0.25, 10, inner="adafactor", state="q8")


def test_right_side_is_the_transposed_left_side():
    rng = np.random.default_rng(11)
    m, n, r = 9, 6, 3
    Q, _ = np.linalg.qr(rng.standard_normal((n, r)))
    a = go.GaLoreOracle(m, n, r, 0.5, 100, inner="adafactor")
    b = go.GaLoreOracle(n, m, r, 0.5, 100, inner="adafactor")
    a.set_projector(Q)
    b.set_projector(Q)
    assert a.side == "right" and b.side == "left"
    Wa = rng.standard_normal((m, n))
    Wb = Wa.T.copy()
    for s in range(3):
        G = rng.standard_normal((m, n))
        Wa = a.step(Wa, G, 1e-2, auto_refresh=False)
        Wb = b.step(Wb, G.T, 1e-2, auto_refresh=False)
    assert np.abs(Wa - Wb.T).max() < 1e-13
