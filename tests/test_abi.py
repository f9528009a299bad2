"""Host-only checks of the C ABI: the library loads, exports what the header declares, validates arguments."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import galore_oracle as go
from paper_2403_03507_b200 import binding as gb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "galore.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(galore_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared_symbols()
    assert "galore_init_layer" in names and "galore_step" in names
    assert "galore_refresh_projector" in names and "galore_free" in names
    handle = C.CDLL(gb.LIB_PATH)
    for name in names:
        assert hasattr(handle, name), f"{name} declared in galore.h but not exported"
    # and the binding marshals every one of them
    assert set(names) == set(gb._PROTOTYPES)


def test_config_struct_layout_matches_header():
    # the header's galore_config_t: field order and sizes as marshalled by the binding
    assert C.sizeof(gb.Config) == 144
    a, b = C.c_size_t(), C.c_size_t()
    assert gb.lib().galore_abi_sizes(C.byref(a), C.byref(b)) == 0
    assert (a.value, b.value) == (C.sizeof(gb.Config), C.sizeof(gb.RefreshInfo))
    assert gb.Config.seed.offset % 8 == 0
    assert C.sizeof(gb.RefreshInfo) == 96


def test_query_bytes_follows_memory_model():
    # optimizer state = m r + 2 n r elements for m <= n (Table 1), each buffer padded to 256 bytes
    m, n, r = 512, 1376, 128
    cfg = gb.make_config(m, n, r, w_dtype="f32", g_dtype="f32", state_fmt="f32")
    sb, wb = gb.galore_query_bytes(cfg)
    assert sb == 4 * (m * r + 2 * n * r)
    cfg_t = gb.make_config(n, m, r, w_dtype="f32", g_dtype="f32", state_fmt="f32")
    assert gb.galore_query_bytes(cfg_t)[0] == sb
    assert sb == 4 * go.GaLoreOracle(m, n, r, 0.25, 5).optimizer_state_elements()
    # 8-bit states: one byte per moment element plus one fp32 absmax per 2048-block, bf16 projector
    cfg8 = gb.make_config(4096, 11008, 1024, state_fmt="q8")
    sb8, _ = gb.galore_query_bytes(cfg8)
    nel = 1024 * 11008
    assert sb8 == 2 * 4096 * 1024 + 2 * nel + 2 * 4 * (nel // 2048)
    assert wb > 0
    # Adafactor: first moment plus one value per row and per column of R (fp32 everywhere here), parts padded to 256 bytes
    cfa = gb.make_config(m, n, r, w_dtype="f32", g_dtype="f32", state_fmt="adafactor")
    sba, _ = gb.galore_query_bytes(cfa)
    pad = lambda b: (b + 255) // 256 * 256
    assert sba == pad(4 * m * r) + pad(4 * r * n) + pad(4 * r) + pad(4 * n)
    assert 0 <= sba - 4 * go.GaLoreOracle(m, n, r, 0.25, 5, inner="adafactor").optimizer_state_elements() < 4 * 256


@pytest.mark.parametrize("kw,status", [
    (dict(rank=0), gb.ERR_SHAPE),
    (dict(rank=13), gb.ERR_SHAPE),
    (dict(m=0), gb.ERR_SHAPE),
    (dict(refresh_gap=0), gb.ERR_INVALID_ARG),
    (dict(beta1=1.0), gb.ERR_INVALID_ARG),
    (dict(q_block=1000), gb.ERR_INVALID_ARG),
    (dict(side=7), gb.ERR_INVALID_ARG),
    (dict(raw_state_fmt=3), gb.ERR_INVALID_ARG),
    (dict(adam_place=5), gb.ERR_INVALID_ARG),
    (dict(refresh_warm_iters=-1), gb.ERR_INVALID_ARG),
    (dict(path=gb.PATH_TENSOR, g_dtype="f32"), gb.ERR_UNIMPLEMENTED),
])
def test_invalid_configs_are_rejected(kw, status):
    base = dict(m=12, n=20, rank=4, refresh_gap=5, w_dtype="f32", g_dtype="f32")
    base.update(kw)
    raw_state_fmt = base.pop("raw_state_fmt", None)
    cfg = gb.make_config(**base)
    if raw_state_fmt is not None:
        cfg.state_fmt = raw_state_fmt                 # a value the binding's names do not reach
    sb, wb = C.c_size_t(), C.c_size_t()
    assert gb.lib().galore_query_bytes(C.byref(cfg), C.byref(sb), C.byref(wb)) == status
    with pytest.raises(gb.GaloreError):
        gb.galore_query_bytes(cfg)


def test_states_too_large_for_32_bit_row_arithmetic_are_refused():
    # 2^31 - 1 columns at rank 2: the state has 2 rows of 2^31 elements, beyond what the kernels index
    cfg = gb.make_config(4, 2 ** 31 - 1, 2, w_dtype="f32", g_dtype="f32")
    sb, wb = C.c_size_t(), C.c_size_t()
    assert gb.lib().galore_query_bytes(C.byref(cfg), C.byref(sb), C.byref(wb)) == gb.ERR_SHAPE
    out = C.c_void_p()
    assert gb.lib().galore_init_layer(C.byref(cfg), 256, 1 << 40, 256, 1 << 40, None, C.byref(out)) == gb.ERR_SHAPE
    # a large but addressable layer is accepted
    assert gb.lib().galore_query_bytes(C.byref(gb.make_config(16384, 65536, 2048)), C.byref(sb), C.byref(wb)) == 0


def test_rank_equal_to_min_dimension_is_legal():
    gb.galore_query_bytes(gb.make_config(12, 20, 12, w_dtype="f32", g_dtype="f32"))


def test_null_and_misaligned_arguments():
    L = gb.lib()
    cfg = gb.make_config(12, 20, 4, w_dtype="f32", g_dtype="f32")
    out = C.c_void_p()
    assert L.galore_init_layer(C.byref(cfg), None, 0, None, 0, None, C.byref(out)) == gb.ERR_INVALID_ARG
    assert L.galore_init_layer(C.byref(cfg), 256, 1 << 30, 128, 1 << 30, None, C.byref(out)) == gb.ERR_ALIGNMENT
    assert L.galore_init_layer(C.byref(cfg), 256, 16, 512, 16, None, C.byref(out)) == gb.ERR_BUFFER_TOO_SMALL
    assert L.galore_step(None, None, 0, None, 0, 0.0, None) == gb.ERR_INVALID_ARG
    assert L.galore_free(None) == gb.ERR_INVALID_ARG
    assert L.galore_status_string(gb.ERR_SHAPE) and L.galore_status_string(1)


def test_codebooks_match_the_oracle_bit_for_bit():
    for signed in (True, False):
        lib_code = np.array(gb.galore_q8_codebook(signed), dtype=np.float32)
        assert np.array_equal(lib_code, go.dynamic_code(signed))


def test_list_entry_points_validate_before_touching_the_device():
    lib = gb.lib()
    none = C.c_void_p(None)
    out = C.c_size_t(7)
    # empty lists are no-ops, negative counts and missing arrays are argument errors
    assert lib.galore_refresh_batch(None, None, None, 0, none, 0, none, None) == 0
    assert lib.galore_refresh_batch(None, None, None, -1, none, 0, none, None) == gb.ERR_INVALID_ARG
    assert lib.galore_refresh_batch(None, None, None, 3, none, 0, none, None) == gb.ERR_INVALID_ARG
    assert lib.galore_step_host_batch(None, None, None, 0, 1e-2, none, 0, 3, none) == 0
    assert lib.galore_step_host_batch(None, None, None, 2, 1e-2, none, 0, 3, none) == gb.ERR_INVALID_ARG
    assert lib.galore_step_host_batch(None, None, None, 0, 1e-2, none, 0, 0, none) == gb.ERR_INVALID_ARG
    assert lib.galore_host_batch_query_bytes(None, 0, 3, C.byref(out)) == gb.ERR_INVALID_ARG
    assert lib.galore_refresh_query_bytes(None, C.byref(out)) == gb.ERR_INVALID_ARG
