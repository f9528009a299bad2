"""galore_step_static: the step for callers that cannot allocate device memory.

Some users of the library run where a device allocation is off limits (a framework that owns all
device memory and forbids cudaMalloc, or a call site that cannot afford the device-wide
synchronisation an allocation implies), so they cannot create the workspace the regular entry
points need.  galore_step_static keeps its intermediates in an array built into the library.
This file checks it against the regular galore_step and against the CPU oracle on two consecutive
steps; it is named so that pytest collects it after every other test file.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import galore_oracle as go
from paper_2403_03507_b200 import binding as gb
from paper_2403_03507_b200 import workloads as wl

TOL_W_F32 = 1e-4     # same bar as the fp32-path parity tests


def test_oversized_layer_is_refused_without_a_gpu():
    # 4096 x 11008 at rank 1024 needs far more than the built-in 16 MiB: refused before any CUDA call
    one = C.c_void_p(256)
    st = gb.lib().galore_step_static(4096, 11008, 1024, gb.SIDE_AUTO, 0.25, 0.9, 0.999, 1e-8, 0, one, one, one, one,
                                     11008, one, 11008, 1e-2, None, None)
    assert st == gb.ERR_BUFFER_TOO_SMALL
    assert gb.lib().galore_step_static(8, 8, 9, gb.SIDE_AUTO, 0.25, 0.9, 0.999, 1e-8, 0, one, one, one, one, 8, one, 8,
                                       1e-2, None, None) == gb.ERR_SHAPE


@pytest.mark.gpu
@pytest.mark.parametrize("m,n,r", [(512, 1376, 128), (300, 130, 24)])
def test_static_step_matches_regular_step_on_two_calls_in_a_row(m, n, r):
    cfg = gb.make_config(m, n, r, refresh_gap=1000, w_dtype="f32", g_dtype="f32", state_fmt="f32", auto_refresh=False)
    layer = gb.Layer(cfg)
    rows = m if m <= n else n
    P = torch.from_numpy(wl.random_orthonormal(rows, r, np.random.default_rng(1))).float().cuda()
    layer.set_projector(P)
    W0 = torch.from_numpy(wl.make_weight(m, n, 2, "f32")).float().cuda()
    W_ref, W_new = W0.clone(), W0.clone()
    M = torch.zeros(layer.state_shape, device="cuda")
    V = torch.zeros(layer.state_shape, device="cuda")
    orc = go.GaLoreOracle(m, n, r, 0.25, 1000, w_store="f32", state="f32")
    orc.set_projector(P.double().cpu().numpy())
    W_orc = W0.double().cpu().numpy()
    gb.galore_static_status()                      # start from a clean accumulated status word
    # the second step and the second shape run with whatever earlier calls left in the shared array
    for s in range(2):
        Gh = wl.make_gradient(m, n, wl.sub_seed(3, s), 1.0, 0.01, "f32")
        G = torch.from_numpy(Gh).float().cuda()
        W_orc = orc.step(W_orc, Gh, 1e-2, auto_refresh=False)
        layer.galore_step(W_ref, G, 1e-2)
        flags = gb.galore_step_static(P, M, V, W_new, G, 1e-2, completed_steps=s)
        assert flags == 0
        torch.cuda.synchronize()
        err = (W_new.double() - W_ref.double()).norm() / W_ref.double().norm()
        derr = ((W_new.double() - W0.double()) - (W_ref.double() - W0.double())).norm() / (W_ref.double() - W0.double()).norm()
        assert err <= TOL_W_F32 and derr <= 1e-3, (s, float(err), float(derr))
        # and against the oracle, within the fp32-path tolerance
        Wn = W_new.double().cpu().numpy()
        assert np.linalg.norm(Wn - W_orc) / np.linalg.norm(W_orc) <= TOL_W_F32
        M_ref, V_ref = layer.get_moments()
        assert torch.allclose(M, M_ref, rtol=1e-5, atol=1e-12) and torch.allclose(V, V_ref, rtol=1e-5, atol=1e-20)
    assert layer.device_status() == 0
    assert gb.galore_static_status() == 0


@pytest.mark.gpu
def test_static_step_keeps_status_bits_for_the_asynchronous_form():
    """Without a flags pointer the call returns at once; what its kernels latch must still be readable later."""
    m, n, r = 64, 96, 8
    P = torch.eye(m, device="cuda")[:, :r].contiguous()
    M = torch.zeros(r, n, device="cuda")
    V = torch.zeros(r, n, device="cuda")
    W = torch.zeros(m, n, device="cuda")
    G = torch.ones(m, n, device="cuda")
    gb.galore_static_status()
    G[0, 0] = float("inf")
    assert gb.galore_step_static(P, M, V, W, G, 1e-2, completed_steps=0, want_flags=False) == 0
    G[0, 0] = 1.0
    M.zero_(); V.zero_()
    assert gb.galore_step_static(P, M, V, W, G, 1e-2, completed_steps=0, want_flags=True) == 0   # this call was clean
    assert gb.galore_static_status() & gb.DEV_NONFINITE        # the earlier one is not lost
    assert gb.galore_static_status() == 0
