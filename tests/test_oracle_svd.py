"""Pins for the oracle's SVD and projector (Eq. 12-13) against facts fixed outside it."""
import numpy as np
import pytest

from oracle import galore_oracle as go
from paper_2403_03507_b200 import workloads as wl


def test_brute_force_8x12_reconstruction_and_spectrum():
    rng = np.random.default_rng(7)
    G = rng.standard_normal((8, 12))
    U, S, Vt = go.jacobi_svd(G)
    # definition: G = U S V^T with orthonormal factors and descending non-negative S
    assert np.allclose((U * S) @ Vt, G, atol=1e-13)
    assert np.allclose(U.T @ U, np.eye(8), atol=1e-13)
    assert np.allclose(Vt @ Vt.T, np.eye(8), atol=1e-13)
    assert np.all(S[:-1] >= S[1:]) and np.all(S >= 0)
    # sigma^2 are the eigenvalues of G G^T, obtained by a different route (symmetric eigensolver)
    lam = np.sort(np.linalg.eigvalsh(G @ G.T))[::-1]
    assert np.allclose(S ** 2, lam, rtol=1e-12)
    # and the characteristic polynomial of G G^T vanishes at each sigma^2 (no library SVD involved)
    A = G @ G.T
    for s2 in S ** 2:
        sign, logdet = np.linalg.slogdet(A - s2 * np.eye(8))
        assert logdet < np.log(1e-9) + 7 * np.log(max(lam))


def test_tall_input_goes_through_transpose():
    rng = np.random.default_rng(8)
    G = rng.standard_normal((13, 5))
    U, S, Vt = go.jacobi_svd(G)
    assert U.shape == (13, 5) and Vt.shape == (5, 5)
    assert np.allclose((U * S) @ Vt, G, atol=1e-13)
    assert np.allclose(S, np.linalg.svd(G, compute_uv=False), rtol=1e-12)


@pytest.mark.parametrize("m,n,r", [(24, 40, 6), (40, 24, 6), (33, 33, 33), (17, 64, 1)])
def test_projector_is_orthonormal_and_exact_on_low_rank(m, n, r):
    # rank(G) <= r  =>  P P^T G = G  (left) or G Q Q^T = G (right)
    spectrum = np.linspace(3.0, 1.0, r)
    G, U, V = wl.make_planted(m, n, seed=11, spectrum=spectrum)
    side = "left" if m <= n else "right"
    P, S = go.top_r_projector(G, r, side)
    assert np.allclose(P.T @ P, np.eye(r), atol=1e-12)
    if side == "left":
        assert np.allclose(P @ (P.T @ G), G, atol=1e-12)
        assert go.largest_principal_angle(U, P) < 1e-7
    else:
        assert np.allclose((G @ P) @ P.T, G, atol=1e-12)
        assert go.largest_principal_angle(V, P) < 1e-7
    assert np.allclose(S[:r], spectrum, rtol=1e-12)
    assert np.all(S[r:] < 1e-12)


def test_gapped_spectrum_recovers_planted_subspace_in_order():
    m, n, r = 48, 80, 8
    k = min(m, n)
    spectrum = np.concatenate([np.linspace(10, 5, r), np.linspace(0.4, 0.01, k - r)])
    G, U, V = wl.make_planted(m, n, seed=5, spectrum=spectrum)
    P, S = go.top_r_projector(G, r, "left")
    assert np.allclose(S, spectrum, rtol=1e-11)
    # column i is +-u_i (distinct singular values): order is by descending sigma
    assert np.allclose(np.abs(np.sum(P * U[:, :r], axis=0)), 1.0, atol=1e-10)
    Q, _ = go.top_r_projector(G, r, "right")
    assert np.allclose(np.abs(np.sum(Q * V[:, :r], axis=0)), 1.0, atol=1e-10)


def test_jacobi_agrees_with_library_svd_on_workload_spectrum():
    # the noise-dominated recipe of the paper-shaped workloads, at a reduced size
    G = wl.make_gradient(96, 200, seed=3, p=1.0, noise=0.01, dtype="f32")
    for side in ("left", "right"):
        Pj, Sj = go.top_r_projector(G, 24, side, method="jacobi")
        Pl, Sl = go.top_r_projector(G, 24, side, method="lapack")
        assert np.allclose(Sj, Sl, rtol=1e-12)
        assert go.largest_principal_angle(Pj, Pl) < 1e-8


def test_library_shortcut_agrees_with_jacobi_at_the_60m_mlp_shape():
    """`method="lapack"` stands in for the Jacobi code at sizes it cannot reach in test time; here both run on
    the full 512 x 1376 matrix of the smallest workload (rank 128, the workload's own noise-dominated recipe)."""
    G = wl.make_gradient(512, 1376, seed=11, p=1.0, noise=0.01, dtype="f32")
    Pj, Sj = go.top_r_projector(G, 128, "left", method="jacobi")
    Pl, Sl = go.top_r_projector(G, 128, "left", method="lapack")
    assert np.allclose(Sj, Sl, rtol=1e-11)
    assert go.largest_principal_angle(Pj, Pl) < 1e-7
    assert np.abs(Pj.T @ Pj - np.eye(128)).max() < 1e-12


def test_principal_angle_of_known_rotation():
    # two planes in R^3 sharing e1, second axis tilted by 0.3 rad
    A = np.array([[1, 0], [0, 1], [0, 0]], float)
    B = np.array([[1, 0], [0, np.cos(0.3)], [0, np.sin(0.3)]], float)
    assert abs(go.largest_principal_angle(A, B) - 0.3) < 1e-12
    assert go.largest_principal_angle(A, A[:, ::-1]) < 1e-12


def test_thread_count_does_not_change_result():
    G = wl.make_gradient(40, 70, seed=9, p=1.0, noise=0.01, dtype="f64")
    U1, S1, V1 = go.jacobi_svd(G, num_threads=1)
    U4, S4, V4 = go.jacobi_svd(G, num_threads=4)
    assert np.array_equal(S1, S4) and np.array_equal(U1, U4) and np.array_equal(V1, V4)
