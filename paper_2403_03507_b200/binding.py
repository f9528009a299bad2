"""Thin ctypes binding of the C ABI in include/galore.h.

Argument marshalling only: every step of the path runs in the CUDA library.
Loading fails loudly when the library has not been built; there is no
fallback of any kind.  torch is used for device buffers and streams.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgalore.so")

OK, WARN_NOT_CONVERGED = 0, 1
ERR_INVALID_ARG, ERR_SHAPE, ERR_ALIGNMENT, ERR_BUFFER_TOO_SMALL = -1, -2, -3, -4
ERR_CUDA, ERR_STATE, ERR_NONFINITE, ERR_TIMEOUT, ERR_UNIMPLEMENTED = -5, -6, -7, -8, -9
SIDE_AUTO, SIDE_LEFT, SIDE_RIGHT = 0, 1, 2
F32, BF16 = 0, 1
STATE_F32, STATE_Q8_BLOCK, STATE_ADAFACTOR = 0, 1, 2
PATH_AUTO, PATH_FP32, PATH_TENSOR = 0, 1, 2
ADAM_AUTO, ADAM_IN_PROJECTION, ADAM_OWN_KERNEL = 0, 1, 2
DEV_NONFINITE, DEV_WAIT_EXPIRED, DEV_CHOLESKY = 1, 2, 8

_DTYPES = {"f32": F32, "bf16": BF16, torch.float32: F32, torch.bfloat16: BF16}
_TORCH = {F32: torch.float32, BF16: torch.bfloat16}


class Config(C.Structure):
    _fields_ = [
        ("m", C.c_int64), ("n", C.c_int64), ("rank", C.c_int32), ("alpha", C.c_float),
        ("refresh_gap", C.c_int32), ("beta1", C.c_double), ("beta2", C.c_double), ("eps", C.c_double),
        ("side", C.c_int32), ("w_dtype", C.c_int32), ("g_dtype", C.c_int32), ("p_dtype", C.c_int32),
        ("state_fmt", C.c_int32), ("q_block", C.c_int32), ("auto_refresh", C.c_int32), ("path", C.c_int32),
        ("refresh_tol", C.c_float), ("refresh_max_iters", C.c_int32), ("refresh_oversample", C.c_int32),
        ("seed", C.c_uint64), ("weight_decay", C.c_float), ("adam_place", C.c_int32), ("refresh_warm_iters", C.c_int32), ("reserved", C.c_int32 * 5),
    ]


class RefreshInfo(C.Structure):
    _fields_ = [
        ("iterations", C.c_int32), ("block", C.c_int32), ("jacobi_sweeps", C.c_int32), ("converged", C.c_int32),
        ("predicted_error", C.c_double), ("residual", C.c_double), ("sigma_r", C.c_double),
        ("sigma_next", C.c_double), ("sigma_1", C.c_double),
        ("ms_total", C.c_double), ("ms_power", C.c_double), ("ms_ritz", C.c_double), ("ms_jacobi", C.c_double),
        ("ritz_passes", C.c_int32), ("reserved", C.c_int32),
    ]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


class GaloreError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        msg = lib().galore_status_string(status).decode()
        cuda = lib().galore_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} ({status})" + (f" [{cuda}]" if status == ERR_CUDA and cuda else ""))


_lib = None

_PROTOTYPES = {
    "galore_query_bytes": (C.c_int, [C.POINTER(Config), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]),
    "galore_init_layer": (C.c_int, [C.POINTER(Config), C.c_void_p, C.c_size_t, C.c_void_p, C.c_size_t, C.c_void_p,
                                    C.POINTER(C.c_void_p)]),
    "galore_step": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_float, C.c_void_p]),
    "galore_step_host": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_float, C.c_void_p]),
    "galore_batch_query_bytes": (C.c_int, [C.POINTER(C.c_void_p), C.c_int32, C.POINTER(C.c_size_t)]),
    "galore_step_batch": (C.c_int, [C.POINTER(C.c_void_p), C.POINTER(C.c_void_p), C.POINTER(C.c_int64),
                                    C.POINTER(C.c_void_p), C.POINTER(C.c_int64), C.c_int32, C.c_float, C.c_void_p,
                                    C.c_size_t, C.c_void_p]),
    "galore_refresh_projector": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.POINTER(RefreshInfo)]),
    "galore_host_batch_query_bytes": (C.c_int, [C.POINTER(C.c_void_p), C.c_int32, C.c_int32, C.POINTER(C.c_size_t)]),
    "galore_step_host_batch": (C.c_int, [C.POINTER(C.c_void_p), C.POINTER(C.c_void_p), C.POINTER(C.c_void_p), C.c_int32,
                                         C.c_float, C.c_void_p, C.c_size_t, C.c_int32, C.c_void_p]),
    "galore_refresh_query_bytes": (C.c_int, [C.c_void_p, C.POINTER(C.c_size_t)]),
    "galore_refresh_batch": (C.c_int, [C.POINTER(C.c_void_p), C.POINTER(C.c_void_p), C.POINTER(C.c_int64), C.c_int32,
                                       C.c_void_p, C.c_size_t, C.c_void_p, C.POINTER(RefreshInfo)]),
    "galore_free": (C.c_int, [C.c_void_p]),
    "galore_step_static": (C.c_int, [C.c_int64, C.c_int64, C.c_int32, C.c_int32, C.c_float, C.c_double, C.c_double,
                                     C.c_double, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64,
                                     C.c_void_p, C.c_int64, C.c_float, C.POINTER(C.c_int32), C.c_void_p]),
    "galore_get_projector": (C.c_int, [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "galore_get_unrounded_projector": (C.c_int, [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "galore_set_projector": (C.c_int, [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "galore_get_moments": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "galore_get_adafactor_state": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "galore_get_q8_state": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "galore_get_step_count": (C.c_int, [C.c_void_p, C.POINTER(C.c_int64)]),
    "galore_set_step_count": (C.c_int, [C.c_void_p, C.c_int64]),
    "galore_layer_info": (C.c_int, [C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.POINTER(C.c_int64),
                                    C.POINTER(C.c_int64)]),
    "galore_device_status": (C.c_int, [C.c_void_p, C.POINTER(C.c_int32), C.c_void_p]),
    "galore_check_device": (C.c_int, [C.c_void_p, C.c_void_p]),
    "galore_export_bytes": (C.c_int, [C.c_void_p, C.POINTER(C.c_size_t)]),
    "galore_export_state": (C.c_int, [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "galore_import_state": (C.c_int, [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "galore_static_status": (C.c_int, [C.POINTER(C.c_int32), C.c_void_p]),
    "galore_q8_codebook": (C.c_int, [C.c_int32, C.POINTER(C.c_float)]),
    "galore_q8_quantize": (C.c_int, [C.c_void_p, C.c_int64, C.c_int64, C.c_int32, C.c_int32, C.c_int32, C.c_void_p,
                                     C.c_void_p, C.c_void_p]),
    "galore_q8_dequantize": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int32, C.c_int32, C.c_int32,
                                       C.c_void_p, C.c_void_p]),
    "galore_abi_sizes": (C.c_int, [C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]),
    "galore_status_string": (C.c_char_p, [C.c_int]),
    "galore_last_cuda_error": (C.c_char_p, []),
    "galore_launch_count": (C.c_int64, []),
    "galore_profile_enable": (C.c_int, [C.c_int32]),
    "galore_profile_read": (C.c_int, [C.POINTER(C.c_double), C.POINTER(C.c_int64)]),
}


def lib():
    """The loaded C library.  Raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2403_03507_b200.build`")
        handle = C.CDLL(LIB_PATH)
        for name, (res, args) in _PROTOTYPES.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        a, b = C.c_size_t(), C.c_size_t()
        handle.galore_abi_sizes(C.byref(a), C.byref(b))
        if (a.value, b.value) != (C.sizeof(Config), C.sizeof(RefreshInfo)):
            raise ImportError("libgalore.so and binding.py disagree on the struct layout: rebuild the library")
        _lib = handle
    return _lib


def _check(status, where):
    if status < 0:
        raise GaloreError(status, where)
    return status


def _stream_ptr(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def make_config(m, n, rank, alpha=0.25, refresh_gap=200, beta1=0.9, beta2=0.999, eps=1e-8, side=SIDE_AUTO,
                w_dtype="bf16", g_dtype="bf16", p_dtype=None, state_fmt="f32", q_block=2048, auto_refresh=True,
                path=PATH_AUTO, refresh_tol=0.0, refresh_max_iters=0, refresh_oversample=0, seed=0,
                weight_decay=0.0, adam_place=ADAM_AUTO, refresh_warm_iters=0) -> Config:
    c = Config()
    c.m, c.n, c.rank, c.alpha, c.refresh_gap = m, n, rank, alpha, refresh_gap
    c.beta1, c.beta2, c.eps = beta1, beta2, eps
    c.side = side
    c.w_dtype, c.g_dtype = _DTYPES[w_dtype], _DTYPES[g_dtype]
    if p_dtype is None:   # bf16 projector only where the gradient is bf16 too (tensor-core operands)
        p_dtype = "bf16" if c.g_dtype == BF16 else "f32"
    c.p_dtype = _DTYPES[p_dtype]
    c.state_fmt = {"f32": STATE_F32, "q8": STATE_Q8_BLOCK, "adafactor": STATE_ADAFACTOR, STATE_F32: STATE_F32,
                   STATE_Q8_BLOCK: STATE_Q8_BLOCK, STATE_ADAFACTOR: STATE_ADAFACTOR}[state_fmt]
    c.q_block, c.auto_refresh, c.path = q_block, int(bool(auto_refresh)), path
    c.refresh_tol, c.refresh_max_iters, c.refresh_oversample, c.seed = refresh_tol, refresh_max_iters, refresh_oversample, seed
    c.weight_decay = weight_decay
    c.adam_place = adam_place
    c.refresh_warm_iters = refresh_warm_iters
    return c


def galore_query_bytes(cfg: Config):
    sb, wb = C.c_size_t(0), C.c_size_t(0)
    _check(lib().galore_query_bytes(C.byref(cfg), C.byref(sb), C.byref(wb)), "galore_query_bytes")
    return sb.value, wb.value


def galore_q8_codebook(is_signed: bool):
    out = (C.c_float * 256)()
    _check(lib().galore_q8_codebook(int(is_signed), out), "galore_q8_codebook")
    return list(out)


STATE_TILE_COLS = 64


def _tile_of(x, block, tile):
    """(rows, cols, tile_rows, tile_cols) of a quantiser call: a flat tensor with `block` consecutive elements
    per block, or a matrix with tile = (tile_rows, tile_cols)."""
    if tile is None:
        return 1, x.numel(), 1, block
    assert x.dim() == 2
    return x.shape[0], x.shape[1], tile[0], tile[1]


def galore_q8_quantize(x: torch.Tensor, is_signed: bool, block: int = 2048, tile=None, stream=None):
    assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous()
    rows, cols, tr, tc = _tile_of(x, block, tile)
    codes = torch.empty(x.shape, dtype=torch.uint8, device=x.device)
    grid = ((rows + tr - 1) // tr, (cols + tc - 1) // tc) if x.numel() else (0, 0)
    absmax = torch.empty(grid if tile is not None else grid[0] * grid[1], dtype=torch.float32, device=x.device)
    _check(lib().galore_q8_quantize(x.data_ptr(), rows, cols, int(is_signed), tr, tc, codes.data_ptr(), absmax.data_ptr(),
                                    _stream_ptr(stream)), "galore_q8_quantize")
    return codes, absmax


def galore_q8_dequantize(codes: torch.Tensor, absmax: torch.Tensor, is_signed: bool, block: int = 2048, tile=None,
                         stream=None):
    rows, cols, tr, tc = _tile_of(codes, block, tile)
    out = torch.empty(codes.shape, dtype=torch.float32, device=codes.device)
    _check(lib().galore_q8_dequantize(codes.data_ptr(), absmax.data_ptr(), rows, cols, int(is_signed), tr, tc,
                                      out.data_ptr(), _stream_ptr(stream)), "galore_q8_dequantize")
    return out


STATIC_SCRATCH_BYTES = 16 * 1024 * 1024


def galore_step_static(P, M, V, W, G, lr, completed_steps, alpha=0.25, beta1=0.9, beta2=0.999, eps=1e-8,
                       side=SIDE_AUTO, want_flags=True, stream=None):
    """One fp32 step on explicit device arrays using the library's built-in scratch (no workspace,
    no allocation inside the library).  For callers that may not allocate device memory; layers
    whose intermediates exceed STATIC_SCRATCH_BYTES are refused.  Calls must not overlap on the GPU.
    Returns the device status bits (0 when want_flags is False)."""
    for t in (P, M, V, W, G):
        assert t.is_cuda and t.dtype == torch.float32
    assert P.is_contiguous() and M.is_contiguous() and V.is_contiguous()
    m, n = W.shape
    flags = C.c_int32(0)
    _check(lib().galore_step_static(m, n, P.shape[1], side, alpha, beta1, beta2, eps, completed_steps, P.data_ptr(),
                                    M.data_ptr(), V.data_ptr(), W.data_ptr(), W.stride(0), G.data_ptr(), G.stride(0),
                                    lr, C.byref(flags) if want_flags else None, _stream_ptr(stream)),
           "galore_step_static")
    return flags.value


def galore_static_status(stream=None) -> int:
    """Status bits latched by galore_step_static calls on the current device since the last read; clears them."""
    f = C.c_int32(0)
    _check(lib().galore_static_status(C.byref(f), _stream_ptr(stream)), "galore_static_status")
    return f.value


def galore_launch_count() -> int:
    return int(lib().galore_launch_count())


def galore_profile_enable(on: bool):
    _check(lib().galore_profile_enable(int(on)), "galore_profile_enable")


def galore_profile_read():
    """Accumulated (milliseconds, brackets) per phase: projection, Adam on R, back-projection."""
    ms = (C.c_double * 3)(0, 0, 0)
    cnt = (C.c_int64 * 3)(0, 0, 0)
    _check(lib().galore_profile_read(ms, cnt), "galore_profile_read")
    return list(ms), list(cnt)


class Layer:
    """One 2-D weight's GaLore state: owns the two device buffers (torch) and the C handle."""

    def __init__(self, cfg: Config, device="cuda:0", workspace: torch.Tensor | None = None, stream=None):
        self.cfg = cfg
        self.device = torch.device(device)
        self.state_bytes, self.workspace_bytes = galore_query_bytes(cfg)
        self.state = torch.empty(self.state_bytes, dtype=torch.uint8, device=self.device)
        if workspace is None:
            workspace = torch.empty(self.workspace_bytes, dtype=torch.uint8, device=self.device)
        if workspace.numel() < self.workspace_bytes:
            raise ValueError("shared workspace too small")
        self.workspace = workspace
        h = C.c_void_p()
        with torch.cuda.device(self.device):
            _check(lib().galore_init_layer(C.byref(cfg), self.state.data_ptr(), self.state.numel(),
                                           workspace.data_ptr(), workspace.numel(), _stream_ptr(stream), C.byref(h)),
                   "galore_init_layer")
        self.handle = h
        side, tp, sr, sc = C.c_int32(), C.c_int32(), C.c_int64(), C.c_int64()
        _check(lib().galore_layer_info(h, C.byref(side), C.byref(tp), C.byref(sr), C.byref(sc)), "galore_layer_info")
        self.side, self.uses_tensor_path, self.state_shape = side.value, bool(tp.value), (sr.value, sc.value)
        self.proj_rows = cfg.m if self.side == SIDE_LEFT else cfg.n

    def close(self):
        if getattr(self, "handle", None):
            lib().galore_free(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the hot path ---------------------------------------------------------
    def galore_step(self, W: torch.Tensor, G: torch.Tensor, lr: float, stream=None) -> int:
        return _check(lib().galore_step(self.handle, W.data_ptr(), W.stride(0), G.data_ptr(), G.stride(0), lr,
                                        _stream_ptr(stream)), "galore_step")

    def galore_step_host(self, W_host, G_host, W_dev, G_dev, lr: float, stream=None) -> int:
        return _check(lib().galore_step_host(self.handle, W_host.data_ptr(), G_host.data_ptr(), W_dev.data_ptr(),
                                             G_dev.data_ptr(), lr, _stream_ptr(stream)), "galore_step_host")

    def galore_refresh_projector(self, G: torch.Tensor, stream=None):
        info = RefreshInfo()
        st = _check(lib().galore_refresh_projector(self.handle, G.data_ptr(), G.stride(0), _stream_ptr(stream),
                                                   C.byref(info)), "galore_refresh_projector")
        return st, info

    # -- accessors ------------------------------------------------------------
    def get_unrounded_projector(self, stream=None) -> torch.Tensor:
        """fp64 projector of the last refresh before rounding to p_dtype (read it right after the refresh)."""
        rows = self.cfg.m if self.side == SIDE_LEFT else self.cfg.n
        out = torch.empty(rows, self.cfg.rank, dtype=torch.float64, device=self.device)
        _check(lib().galore_get_unrounded_projector(self.handle, out.data_ptr(), out.numel() * 8, _stream_ptr(stream)),
               "galore_get_unrounded_projector")
        return out

    def get_projector(self, stream=None) -> torch.Tensor:
        out = torch.empty(self.proj_rows, self.cfg.rank, dtype=torch.float32, device=self.device)
        _check(lib().galore_get_projector(self.handle, out.data_ptr(), out.numel() * 4, _stream_ptr(stream)),
               "galore_get_projector")
        return out

    def set_projector(self, P: torch.Tensor, stream=None):
        P = P.to(device=self.device, dtype=torch.float32).contiguous()
        assert tuple(P.shape) == (self.proj_rows, self.cfg.rank)
        _check(lib().galore_set_projector(self.handle, P.data_ptr(), P.numel() * 4, _stream_ptr(stream)),
               "galore_set_projector")
        torch.cuda.current_stream().synchronize() if stream is None else stream.synchronize()

    def get_moments(self, stream=None):
        M = torch.empty(self.state_shape, dtype=torch.float32, device=self.device)
        V = torch.empty(self.state_shape, dtype=torch.float32, device=self.device)
        _check(lib().galore_get_moments(self.handle, M.data_ptr(), V.data_ptr(), M.numel() * 4, _stream_ptr(stream)),
               "galore_get_moments")
        return M, V

    def get_adafactor_state(self, stream=None):
        rows, cols = self.state_shape
        M = torch.empty(rows, cols, dtype=torch.float32, device=self.device)
        v_row = torch.empty(rows, dtype=torch.float32, device=self.device)
        v_col = torch.empty(cols, dtype=torch.float32, device=self.device)
        _check(lib().galore_get_adafactor_state(self.handle, M.data_ptr(), v_row.data_ptr(), v_col.data_ptr(),
                                                _stream_ptr(stream)), "galore_get_adafactor_state")
        return M, v_row, v_col

    def get_q8_state(self, stream=None):
        rows, cols = self.state_shape
        tr = (self.cfg.q_block or 2048) // STATE_TILE_COLS
        grid = ((rows + tr - 1) // tr, (cols + STATE_TILE_COLS - 1) // STATE_TILE_COLS)
        Mc = torch.empty(rows, cols, dtype=torch.uint8, device=self.device)
        Vc = torch.empty(rows, cols, dtype=torch.uint8, device=self.device)
        Ma = torch.empty(grid, dtype=torch.float32, device=self.device)
        Va = torch.empty(grid, dtype=torch.float32, device=self.device)
        _check(lib().galore_get_q8_state(self.handle, Mc.data_ptr(), Ma.data_ptr(), Vc.data_ptr(), Va.data_ptr(),
                                         _stream_ptr(stream)), "galore_get_q8_state")
        return Mc, Ma, Vc, Va

    @property
    def step_count(self) -> int:
        k = C.c_int64()
        _check(lib().galore_get_step_count(self.handle, C.byref(k)), "galore_get_step_count")
        return k.value

    @step_count.setter
    def step_count(self, k: int):
        _check(lib().galore_set_step_count(self.handle, k), "galore_set_step_count")

    def check_device(self, stream=None) -> int:
        """galore_check_device: the latched device conditions as a status code (0 ok, negative error); does not raise."""
        return int(lib().galore_check_device(self.handle, _stream_ptr(stream)))

    def export_state(self, stream=None) -> torch.Tensor:
        """galore_export_state into a new pinned host buffer (uint8)."""
        n = C.c_size_t(0)
        _check(lib().galore_export_bytes(self.handle, C.byref(n)), "galore_export_bytes")
        buf = torch.empty(n.value, dtype=torch.uint8).pin_memory()
        _check(lib().galore_export_state(self.handle, buf.data_ptr(), buf.numel(), _stream_ptr(stream)), "galore_export_state")
        return buf

    def import_state(self, buf: torch.Tensor, stream=None):
        assert not buf.is_cuda and buf.dtype == torch.uint8 and buf.is_contiguous()
        _check(lib().galore_import_state(self.handle, buf.data_ptr(), buf.numel(), _stream_ptr(stream)), "galore_import_state")

    def device_status(self, stream=None) -> int:
        f = C.c_int32()
        _check(lib().galore_device_status(self.handle, C.byref(f), _stream_ptr(stream)), "galore_device_status")
        return f.value


class HostBatch:
    """Layers whose W and G stay in pinned host memory, stepped through galore_step_host_batch."""

    def __init__(self, layers, W_hosts, G_hosts, slots: int = 3, device=None):
        self.layers = list(layers)
        self.n = len(self.layers)
        self.slots = int(slots)
        self.device = device if device is not None else self.layers[0].device
        self._hs = (C.c_void_p * self.n)(*[l.handle.value for l in self.layers])
        out = C.c_size_t(0)
        _check(lib().galore_host_batch_query_bytes(self._hs, self.n, self.slots, C.byref(out)), "galore_host_batch_query_bytes")
        self.staging = torch.empty(max(out.value, 256), dtype=torch.uint8, device=self.device)
        self.rebind(W_hosts, G_hosts)

    def rebind(self, W_hosts, G_hosts):
        for t in list(W_hosts) + list(G_hosts):
            if not (t.is_pinned() and t.is_contiguous()):
                raise ValueError("host tensors must be pinned and contiguous")
        self.W_hosts, self.G_hosts = list(W_hosts), list(G_hosts)
        self._wp = (C.c_void_p * self.n)(*[w.data_ptr() for w in self.W_hosts])
        self._gp = (C.c_void_p * self.n)(*[g.data_ptr() for g in self.G_hosts])

    def galore_step_host_batch(self, lr: float, stream=None) -> int:
        return _check(lib().galore_step_host_batch(self._hs, self._wp, self._gp, self.n, lr, self.staging.data_ptr(),
                                                   self.staging.numel(), self.slots, _stream_ptr(stream)),
                      "galore_step_host_batch")


def galore_refresh_query_bytes(layer) -> int:
    out = C.c_size_t(0)
    _check(lib().galore_refresh_query_bytes(layer.handle, C.byref(out)), "galore_refresh_query_bytes")
    return out.value


def galore_refresh_batch(layers, Gs, stream=None, workspace=None, want_infos=True):
    """Refreshes the projectors of `layers` from `Gs` through one shared workspace; neighbours of one shape are
    refreshed together, as many at a time as the workspace holds copies of one layer's refresh workspace.

    workspace: a uint8 CUDA tensor (allocated here, for one layer at a time, when None).  Returns (status, infos);
    without want_infos the library skips its phase clock and the residual diagnostic, and infos is [].
    """
    n = len(layers)
    need = max(galore_refresh_query_bytes(l) for l in layers)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=layers[0].device)
    hs = (C.c_void_p * n)(*[l.handle.value for l in layers])
    gp = (C.c_void_p * n)(*[g.data_ptr() for g in Gs])
    lg = (C.c_int64 * n)(*[g.stride(0) for g in Gs])
    infos = (RefreshInfo * n)() if want_infos else None
    st = _check(lib().galore_refresh_batch(hs, gp, lg, n, workspace.data_ptr(), workspace.numel(), _stream_ptr(stream),
                                           infos), "galore_refresh_batch")
    return st, (list(infos) if want_infos else [])


def galore_batch_query_bytes(layers) -> int:
    n = len(layers)
    hs = (C.c_void_p * n)(*[l.handle.value for l in layers])
    out = C.c_size_t(0)
    _check(lib().galore_batch_query_bytes(hs, n, C.byref(out)), "galore_batch_query_bytes")
    return out.value


class Batch:
    """A fixed list of layers stepped together by galore_step_batch.

    Holds the batch workspace (torch) and the marshalled pointer arrays, so that a step is one
    call into the library.  W and G tensors are bound once; rebind() swaps them.
    """

    def __init__(self, layers, Ws, Gs, workspace_bytes=None, device=None, workspace=None):
        self.layers = list(layers)
        self.n = len(self.layers)
        self.device = device if device is not None else self.layers[0].device
        need = galore_batch_query_bytes(self.layers)
        if workspace is not None:          # a caller-owned buffer, e.g. shared by batches that never run together
            self.workspace_bytes = int(workspace.numel())
            self.workspace = workspace
        else:
            self.workspace_bytes = need if workspace_bytes is None else int(workspace_bytes)
            self.workspace = torch.empty(max(self.workspace_bytes, 256), dtype=torch.uint8, device=self.device)
        self._hs = (C.c_void_p * self.n)(*[l.handle.value for l in self.layers])
        self.rebind(Ws, Gs)

    def rebind(self, Ws, Gs):
        self.Ws, self.Gs = list(Ws), list(Gs)
        n = self.n
        self._wp = (C.c_void_p * n)(*[w.data_ptr() for w in self.Ws])
        self._gp = (C.c_void_p * n)(*[g.data_ptr() for g in self.Gs])
        self._lw = (C.c_int64 * n)(*[w.stride(0) for w in self.Ws])
        self._lg = (C.c_int64 * n)(*[g.stride(0) for g in self.Gs])

    def galore_step_batch(self, lr: float, stream=None) -> int:
        return _check(lib().galore_step_batch(self._hs, self._wp, self._lw, self._gp, self._lg, self.n, lr,
                                              self.workspace.data_ptr(), self.workspace_bytes, _stream_ptr(stream)),
                      "galore_step_batch")


def galore_step_batch(layers, Ws, Gs, lr: float, stream=None, workspace_bytes=None) -> int:
    """One-off convenience: builds a Batch (allocating its workspace) and steps it once."""
    return Batch(layers, Ws, Gs, workspace_bytes).galore_step_batch(lr, stream)
