"""Pins for the oracle's 8-bit block-wise state format.

The paper names 8-bit Adam states without giving a format, so nothing printed
there can pin these; the format is pinned by its own invariants and by brute
force on small inputs.
"""
import numpy as np
import pytest

from oracle import galore_oracle as go
from paper_2403_03507_b200 import workloads as wl


@pytest.mark.parametrize("signed", [True, False])
def test_code_table_shape_and_anchor_values(signed):
    c = go.dynamic_code(signed)
    assert c.dtype == np.float32 and c.shape == (256,)
    assert np.all(np.diff(c.astype(np.float64)) > 0)              # strictly ascending, all distinct
    assert c[-1] == 1.0 and np.count_nonzero(c == 0.0) == 1
    if signed:
        assert c[0] == -1.0
        neg, pos = c[c < 0], c[c > 0]
        assert len(neg) == 127 and len(pos) == 128
        assert np.array_equal(-neg[::-1], pos[1:])                # symmetric apart from the extra smallest positive
    else:
        assert c[0] == 0.0
    # decades: the largest magnitude of decade e is exactly 10**-e
    for e in range(0, 7):
        assert np.float32(10.0 ** -e) in c


@pytest.mark.parametrize("signed", [True, False])
def test_every_code_value_round_trips(signed):
    c = go.dynamic_code(signed)
    for absmax in (1.0, 0.37, 1e-5, 123.0):
        x = (c.astype(np.float64) * absmax).astype(np.float32)
        x[-1] = np.float32(absmax)                                # make the block's absmax exact
        codes, am = go.quantize_blockwise(x, signed, block=256)
        assert am[0] == np.float32(absmax)
        back = go.dequantize_blockwise(codes, am, signed, block=256)
        # quantising a dequantised state reproduces the same codes (idempotent)
        codes2, am2 = go.quantize_blockwise(back, signed, block=256)
        assert np.array_equal(codes2, codes) and np.array_equal(am2, am)
    codes, _ = go.quantize_blockwise(c, signed, block=256)
    assert np.array_equal(codes, np.arange(256, dtype=np.uint8))


@pytest.mark.parametrize("signed", [True, False])
def test_brute_force_nearest_code(signed):
    rng = np.random.default_rng(1)
    x = (rng.standard_normal(700) * 10.0 ** rng.uniform(-6, 0, 700)).astype(np.float32)
    if not signed:
        x = np.abs(x)
    block = 256
    codes, am = go.quantize_blockwise(x, signed, block)
    c = go.dynamic_code(signed).astype(np.float64)
    assert len(am) == 3                                            # 256 + 256 + 188: ragged tail block
    for i, xi in enumerate(x):
        a = am[i // block]
        assert a == np.max(np.abs(x[(i // block) * block:(i // block + 1) * block]))
        y = np.float64(np.float32(xi) / np.float32(a))
        dist = np.abs(c - y)
        best = np.min(dist)
        # nearest code value; among equally near ones the larger index
        cand = np.nonzero(dist <= best * (1 + 1e-6) + 1e-12)[0]
        assert codes[i] in cand
        if len(cand) == 1:
            assert codes[i] == cand[0]


def test_tie_goes_to_larger_index_and_absmax_maps_to_one():
    c = go.dynamic_code(True)
    mids = go.code_midpoints(c)
    # a value exactly on a threshold (absmax 1 so that y == x)
    for k in (3, 100, 128, 200, 254):
        x = np.array([mids[k], 1.0], dtype=np.float32)
        codes, am = go.quantize_blockwise(x, True, block=2)
        assert am[0] == 1.0 and codes[0] == k + 1 and codes[1] == 255
    x = np.array([-2.5, 0.1, 2.0], dtype=np.float32)
    codes, am = go.quantize_blockwise(x, True, block=3)
    assert am[0] == 2.5 and codes[0] == 0                          # -absmax -> code of -1


def test_zero_block_and_empty_input():
    x = np.zeros(10, dtype=np.float32)
    for signed in (True, False):
        codes, am = go.quantize_blockwise(x, signed, block=4)
        zero = int(np.nonzero(go.dynamic_code(signed) == 0)[0][0])
        assert np.all(codes == zero) and np.all(am == 0) and len(am) == 3
        assert np.all(go.dequantize_blockwise(codes, am, signed, block=4) == 0)
    codes, am = go.quantize_blockwise(np.zeros(0, np.float32), True)
    assert codes.size == 0 and am.size == 0


def test_relative_error_bound_of_the_code():
    # within a decade the spacing is 0.9 * 10**-e / 2**f, so |x - dq(x)| <= half of that times absmax
    rng = np.random.default_rng(5)
    x = rng.uniform(0.1, 1.0, 5000).astype(np.float32)
    x[0] = 1.0
    codes, am = go.quantize_blockwise(x, False, block=5000)
    back = go.dequantize_blockwise(codes, am, False, block=5000)
    assert np.max(np.abs(back - x)) <= 0.5 * 0.9 / 128 + 1e-6


def test_q8_states_track_fp32_states():
    # GaLore-Adam with 8-bit moments stays close to the fp32-moment run (sanity of the wiring)
    m, n, r = 32, 160, 8
    hp = dict(alpha=0.25, refresh_gap=100, beta1=0.9, beta2=0.999, eps=1e-8)
    a = go.GaLoreOracle(m, n, r, state="f32", **hp)
    b = go.GaLoreOracle(m, n, r, state="q8", q_block=256, **hp)
    W0 = wl.make_weight(m, n, 1, "f64")
    Wa, Wb = W0, W0
    for s in range(6):
        g = wl.make_gradient(m, n, wl.sub_seed(1, s), 1.0, 0.01, "f64")
        Wa, Wb = a.step(Wa, g, 1e-2), b.step(Wb, g, 1e-2)
    Ma, Va = a.moments()
    Mb, Vb = b.moments()
    assert b.M_absmax.shape == ((r + 3) // 4, (n + 63) // 64)          # q_block 256 = tiles of 4 x 64
    assert np.linalg.norm(Mb - Ma) / np.linalg.norm(Ma) < 0.05
    assert np.linalg.norm((Wb - W0) - (Wa - W0)) / np.linalg.norm(Wa - W0) < 0.1
    # first step does not depend on the state format at all (states start at zero)
    a1 = go.GaLoreOracle(m, n, r, state="f32", **hp)
    b1 = go.GaLoreOracle(m, n, r, state="q8", q_block=256, **hp)
    g = wl.make_gradient(m, n, 3, 1.0, 0.01, "f64")
    assert np.array_equal(a1.step(W0, g, 1e-2), b1.step(W0, g, 1e-2))


@pytest.mark.parametrize("signed", [True, False])
@pytest.mark.parametrize("rows,cols,tr,tc", [(37, 300, 32, 64), (5, 128, 4, 64), (33, 65, 32, 64), (40, 90, 8, 32)])
def test_tiles_brute_force_geometry_and_codes(signed, rows, cols, tr, tc):
    """Which elements share an absmax, written out with explicit index arithmetic, and the nearest code by
    exhaustive search over the 256 values."""
    rng = np.random.default_rng(rows * 1000 + cols)
    X = (rng.standard_normal((rows, cols)) * 10.0 ** rng.uniform(-5, 0, (rows, cols))).astype(np.float32)
    if not signed:
        X = np.abs(X)
    codes, am = go.quantize_tiles(X, signed, tr, tc)
    assert codes.shape == X.shape and am.shape == ((rows + tr - 1) // tr, (cols + tc - 1) // tc)
    c = go.dynamic_code(signed).astype(np.float64)
    for i in range(rows):
        for j in range(cols):
            I, J = i // tr, j // tc
            a = np.float32(0)
            for ii in range(I * tr, min(rows, (I + 1) * tr)):
                for jj in range(J * tc, min(cols, (J + 1) * tc)):
                    a = max(a, abs(X[ii, jj]))
            assert am[I, J] == a
            y = np.float64(X[i, j] / a)                                # fp32 quotient
            dist = np.abs(c - y)
            cand = np.nonzero(dist <= dist.min() * (1 + 1e-6) + 1e-12)[0]
            assert codes[i, j] in cand
    back = go.dequantize_tiles(codes, am, signed, tr, tc)
    for i in range(0, rows, 3):
        for j in range(0, cols, 7):
            assert back[i, j] == np.float32(go.dynamic_code(signed)[codes[i, j]] * am[i // tr, j // tc])


def test_one_large_element_changes_only_its_own_tile():
    X = np.full((40, 300), 0.01, dtype=np.float32)
    base_codes, base_am = go.quantize_tiles(X, True, 16, 128)
    X[17, 130] = 5.0                                                    # tile (1, 1)
    codes, am = go.quantize_tiles(X, True, 16, 128)
    changed = np.argwhere(codes != base_codes)
    assert am[1, 1] == 5.0 and np.count_nonzero(am != base_am) == 1
    assert changed[:, 0].min() == 16 and changed[:, 0].max() == 31 and changed[:, 1].min() == 128 and changed[:, 1].max() == 255
    assert len(changed) == 16 * 128 - 1          # every other element of that tile (the large one keeps the code of 1), nothing else


def test_flat_blocks_are_tiles_of_a_one_row_matrix():
    rng = np.random.default_rng(9)
    x = rng.standard_normal(1000).astype(np.float32)
    c1, a1 = go.quantize_blockwise(x, True, 256)
    c2, a2 = go.quantize_tiles(x.reshape(1, -1), True, 1, 256)
    assert np.array_equal(c1, c2.ravel()) and np.array_equal(a1, a2.ravel()) and len(a1) == 4


def test_state_tile_shapes():
    assert go.state_tile(2048) == (32, 64) and go.state_tile(256) == (4, 64) and go.state_tile(1024) == (16, 64)
    with pytest.raises(ValueError):
        go.state_tile(1000)
    o = go.GaLoreOracle(40, 300, 40, 0.25, 10, state="q8", q_block=2048)
    assert o.M_codes.shape == (40, 300) and o.M_absmax.shape == (2, 5)
    o = go.GaLoreOracle(300, 40, 24, 0.25, 10, state="q8", q_block=512)          # right side: state is m x r
    assert o.V_codes.shape == (300, 24) and o.V_absmax.shape == (38, 1)
