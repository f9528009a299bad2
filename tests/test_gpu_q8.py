"""The 8-bit state codes must equal the oracle's bit for bit on identical fp32 inputs."""
import numpy as np
import pytest
import torch

from oracle import galore_oracle as go
from paper_2403_03507_b200 import binding as gb

pytestmark = pytest.mark.gpu


def _inputs(count, signed, seed):
    rng = np.random.default_rng(seed)
    x = (rng.standard_normal(count) * 10.0 ** rng.uniform(-7, 1, count)).astype(np.float32)
    return x if signed else np.abs(x)


@pytest.mark.parametrize("signed", [True, False])
@pytest.mark.parametrize("count,block", [(2048 * 5 + 777, 2048), (256 * 3, 256), (4096 * 2 + 1, 4096), (100, 512), (1, 1024)])
def test_codes_and_absmax_bit_exact(signed, count, block):
    x = _inputs(count, signed, seed=count + block)
    codes_o, am_o = go.quantize_blockwise(x, signed, block)
    codes_g, am_g = gb.galore_q8_quantize(torch.from_numpy(x).cuda(), signed, block)
    assert np.array_equal(codes_g.cpu().numpy(), codes_o)
    assert np.array_equal(am_g.cpu().numpy(), am_o)
    back_o = go.dequantize_blockwise(codes_o, am_o, signed, block)
    back_g = gb.galore_q8_dequantize(codes_g, am_g, signed, block)
    assert np.array_equal(back_g.cpu().numpy(), back_o)


@pytest.mark.parametrize("signed", [True, False])
def test_thresholds_ties_and_zero_blocks(signed):
    code = go.dynamic_code(signed)
    mids = go.code_midpoints(code)
    # every threshold, its neighbours in fp32, every code value; absmax forced to exactly 1
    pts = np.concatenate([mids, np.nextafter(mids, np.float32(2)), np.nextafter(mids, np.float32(-2)), code,
                          np.array([1.0], np.float32)]).astype(np.float32)
    pad = (-len(pts)) % 256
    pts = np.concatenate([pts, np.ones(pad, np.float32)])
    # one block of all zeros in the middle
    x = np.concatenate([pts[:512], np.zeros(256, np.float32), pts[512:]])
    x[::256] = 1.0
    x[512:768] = 0.0
    codes_o, am_o = go.quantize_blockwise(x, signed, 256)
    codes_g, am_g = gb.galore_q8_quantize(torch.from_numpy(x).cuda(), signed, 256)
    assert np.array_equal(codes_g.cpu().numpy(), codes_o)
    assert np.array_equal(am_g.cpu().numpy(), am_o)
    assert am_o[2] == 0 and np.all(codes_o[512:768] == (127 if signed else 0))


@pytest.mark.parametrize("signed", [True, False])
def test_quotients_next_to_thresholds_any_absmax(signed):
    """Blocks [a, x_1 .. x_255] with x_i within a few ulp of threshold_i * a for arbitrary absmax a: the
    cases where x * (1 / a) and the correctly rounded x / a can fall on different sides of a threshold."""
    mids = go.code_midpoints(go.dynamic_code(signed)).astype(np.float32)
    assert len(mids) == 255
    rng = np.random.default_rng(5)
    blocks = []
    for off in range(-3, 4):
        for _ in range(160):
            a = np.float32(rng.uniform(1.0, 2.0) * 10.0 ** rng.uniform(-6, 3))
            x = (mids.astype(np.float64) * float(a)).astype(np.float32)
            x = (x.view(np.int32) + off).view(np.float32)          # same-sign neighbours: |x| moves by `off` ulp
            blocks.append(np.concatenate([[a], x]).astype(np.float32))
    x = np.concatenate(blocks)
    assert np.all(np.abs(x.reshape(-1, 256)[:, 1:]) <= x.reshape(-1, 256)[:, :1])
    codes_o, am_o = go.quantize_blockwise(x, signed, 256)
    codes_g, am_g = gb.galore_q8_quantize(torch.from_numpy(x).cuda(), signed, 256)
    assert np.array_equal(am_g.cpu().numpy(), am_o)
    assert np.array_equal(codes_g.cpu().numpy(), codes_o)


@pytest.mark.parametrize("signed", [True, False])
@pytest.mark.parametrize("rows,cols,tile", [(37, 300, (32, 64)), (64, 256, (32, 64)), (5, 128, (4, 64)),
                                            (33, 129, (16, 64)), (40, 90, (8, 32))])
def test_tiled_blocks_bit_exact(signed, rows, cols, tile):
    """Quantisation blocks as tiles of a matrix (the layout of a layer's 8-bit moments), ragged edges included."""
    x = _inputs(rows * cols, signed, seed=rows + cols).reshape(rows, cols)
    codes_o, am_o = go.quantize_tiles(x, signed, *tile)
    codes_g, am_g = gb.galore_q8_quantize(torch.from_numpy(x).cuda(), signed, tile=tile)
    assert np.array_equal(codes_g.cpu().numpy(), codes_o)
    assert np.array_equal(am_g.cpu().numpy(), am_o)
    back_g = gb.galore_q8_dequantize(codes_g, am_g, signed, tile=tile)
    assert np.array_equal(back_g.cpu().numpy(), go.dequantize_tiles(codes_o, am_o, signed, *tile))


def test_empty_input():
    codes, am = gb.galore_q8_quantize(torch.zeros(0, device="cuda"), True, 2048)
    assert codes.numel() == 0 and am.numel() == 0
