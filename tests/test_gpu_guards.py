"""Nothing outside the caller's matrices is written: W and G live inside larger buffers whose surroundings
(rows before and after, the padding columns of every row) hold a sentinel that must survive the steps, and
G itself must come back unchanged."""
import numpy as np
import pytest
import torch

from paper_2403_03507_b200 import binding as gb
from paper_2403_03507_b200 import workloads as wl

pytestmark = pytest.mark.gpu

SENTINEL = 12345.0
GUARD_ROWS = 3


def _guarded(host, dtype, ld):
    """host (m x n) placed in a (m + 2 guard rows) x ld buffer filled with the sentinel; returns (buffer, view)."""
    m, n = host.shape
    tdt = {"f32": torch.float32, "bf16": torch.bfloat16}[dtype]
    buf = torch.full((m + 2 * GUARD_ROWS, ld), SENTINEL, dtype=tdt, device="cuda")
    view = buf[GUARD_ROWS:GUARD_ROWS + m, :n]
    view.copy_(torch.from_numpy(host).to(tdt))
    return buf, view


def _surroundings_intact(buf, m, n):
    s = torch.tensor(SENTINEL, dtype=buf.dtype, device=buf.device)
    return bool((buf[:GUARD_ROWS] == s).all() and (buf[GUARD_ROWS + m:] == s).all() and
                (buf[GUARD_ROWS:GUARD_ROWS + m, n:] == s).all())


CASES = [
    # m, n, r, dtype of W and G, state format, extra padding columns
    (300, 1000, 72, "bf16", "q8", 24),          # tensor path, ragged tiles in every dimension
    (1000, 300, 72, "bf16", "q8", 8),           # right side
    (512, 1376, 256, "bf16", "f32", 16),        # CTA pairs
    (384, 1000, 128, "bf16", "adafactor", 8),
    (130, 301, 17, "f32", "f32", 5),            # fp32 path, odd sizes and an odd pitch
    (301, 130, 17, "f32", "q8", 3),
    (200, 304, 16, "f32", "adafactor", 1),
]


@pytest.mark.parametrize("m,n,r,dt,fmt,pad", CASES)
@pytest.mark.parametrize("batched", [False, True])
def test_steps_and_refresh_stay_inside_the_matrices(m, n, r, dt, fmt, pad, batched):
    ld = n + pad
    if dt == "bf16":
        ld = (ld + 7) // 8 * 8                  # rows the tensor path can address
    count = 3 if batched else 1
    layers, Wb, Wv, Gb, Gv, G0 = [], [], [], [], [], []
    for i in range(count):
        layers.append(gb.Layer(gb.make_config(m, n, r, w_dtype=dt, g_dtype=dt, state_fmt=fmt, refresh_gap=2, seed=i)))
        b, v = _guarded(wl.make_weight(m, n, 10 + i, dt), dt, ld)
        Wb.append(b); Wv.append(v)
        b, v = _guarded(wl.make_gradient(m, n, 20 + i, 0.8, 0.05, dt), dt, ld)
        Gb.append(b); Gv.append(v); G0.append(v.clone())
    W_start = [v.clone() for v in Wv]
    for step in range(3):                        # refreshes at k = 0 and k = 2 run inside the calls
        if batched:
            gb.Batch(layers, Wv, Gv).galore_step_batch(1e-2)
        else:
            layers[0].galore_step(Wv[0], Gv[0], 1e-2)
    torch.cuda.synchronize()
    for i in range(count):
        assert _surroundings_intact(Wb[i], m, n), "W: something outside the matrix was written"
        assert _surroundings_intact(Gb[i], m, n) and torch.equal(Gv[i], G0[i]), "G was written"
        assert not torch.equal(Wv[i], W_start[i]) and bool(torch.isfinite(Wv[i].float()).all())
        assert layers[i].device_status() == 0 and layers[i].step_count == 3
