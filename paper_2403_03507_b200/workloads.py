"""Seeded synthetic inputs shaped like the GaLore paper's workloads.

Holds no optimizer arithmetic: only shapes, hyper-parameter records and random
matrices.  Both the CPU oracle's tests and the CUDA path's tests draw their
inputs from here, so that the two sides always see the same arrays.

Shapes come from the LLaMA architecture table of the paper's pre-training
appendix ("Architecture and Hyperparameters"); ranks, refresh gap and scale
from its experiment sections.  The gradients are stand-ins for gradients of a
trained model: a decaying planted spectrum plus i.i.d. Gaussian noise,

    G = U diag(s) V^T + noise * N(0, 1),   s_i = i ** -p,

with U (m x k) and V (n x k), k = min(m, n), random orthonormal bases obtained
from QR factorisations of seeded Gaussian matrices.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

BASE_SEED = 0x2403035070


@dataclass(frozen=True)
class Workload:
    name: str
    shapes: tuple            # ((m, n, count), ...) over the whole layer set
    rank: int
    alpha: float
    refresh_gap: int
    w_dtype: str             # 'f32' | 'bf16'
    g_dtype: str
    state_fmt: str           # 'f32' | 'q8' (Adam moments) | 'adafactor'
    spectrum_p: float
    noise: float
    lr: float = 1e-2
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    q_block: int = 2048
    seed: int = BASE_SEED

    @property
    def params(self) -> int:
        return sum(m * n * c for m, n, c in self.shapes)

    @property
    def matrices(self) -> int:
        return sum(c for _, _, c in self.shapes)


def _llama(layers, hidden, inter):
    return ((hidden, hidden, 4 * layers), (hidden, inter, 2 * layers), (inter, hidden, layers))


WORKLOADS = {
    "single_60m_mlp": Workload("single_60m_mlp", ((512, 1376, 1),), 128, 0.25, 5, "f32", "f32", "f32",
                               1.0, 0.01, seed=BASE_SEED + 0),
    "llama_130m": Workload("llama_130m", _llama(12, 768, 2048), 256, 0.25, 200, "bf16", "f32", "f32",
                           1.0, 0.01, seed=BASE_SEED + 1),
    "llama_1b_f32": Workload("llama_1b_f32", _llama(24, 2048, 5461), 512, 0.25, 200, "bf16", "bf16", "f32",
                             0.8, 0.05, seed=BASE_SEED + 2),
    "llama_1b_q8": Workload("llama_1b_q8", _llama(24, 2048, 5461), 512, 0.25, 200, "bf16", "bf16", "q8",
                            0.8, 0.05, seed=BASE_SEED + 2),
    "llama_1b_adafactor": Workload("llama_1b_adafactor", _llama(24, 2048, 5461), 512, 0.25, 200, "bf16", "bf16",
                                   "adafactor", 0.8, 0.05, seed=BASE_SEED + 2),
    "llama_7b_q8": Workload("llama_7b_q8", _llama(32, 4096, 11008), 1024, 0.25, 500, "bf16", "bf16", "q8",
                            0.8, 0.05, seed=BASE_SEED + 3),
    "sweep_4096x11008": Workload("sweep_4096x11008", ((4096, 11008, 1),), 1024, 0.25, 200, "bf16", "bf16", "q8",
                                 1.0, 0.01, seed=BASE_SEED + 4),
}
SWEEP_RANKS = (64, 128, 256, 512, 1024, 2048)
SWEEP_GAPS = (50, 200, 1000)


def sub_seed(seed: int, *keys: int) -> int:
    """Independent stream id for (layer, matrix, step, ...) below a base seed."""
    s = np.random.SeedSequence([seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF, *[int(k) for k in keys]])
    return int(s.generate_state(1, dtype=np.uint64)[0])


def round_to(x: np.ndarray, dtype: str) -> np.ndarray:
    """Values of x rounded to the storage type, returned as fp64 (exactly representable)."""
    if dtype == "f32":
        return x.astype(np.float32).astype(np.float64)
    if dtype == "bf16":
        import torch
        return torch.from_numpy(np.ascontiguousarray(x)).to(torch.bfloat16).to(torch.float64).numpy()
    if dtype == "f64":
        return x.astype(np.float64)
    raise ValueError(dtype)


def random_orthonormal(rows: int, cols: int, rng: np.random.Generator) -> np.ndarray:
    q, _ = np.linalg.qr(rng.standard_normal((rows, cols)))
    return q


def make_gradient(m: int, n: int, seed: int, p: float = 1.0, noise: float = 0.01, dtype: str = "f32",
                  spectrum=None) -> np.ndarray:
    """Decaying-spectrum-plus-noise gradient, rounded to `dtype`, as fp64.

    `spectrum` (length min(m, n)) replaces s_i = i**-p when given; a spectrum
    with a gap after index r and noise = 0 yields an input whose top-r
    subspace is the planted one.
    """
    rng = np.random.default_rng(seed)
    k = min(m, n)
    U = random_orthonormal(m, k, rng)
    V = random_orthonormal(n, k, rng)
    s = np.arange(1, k + 1, dtype=np.float64) ** (-p) if spectrum is None else np.asarray(spectrum, np.float64)
    G = (U * s) @ V.T
    if noise:
        G = G + noise * rng.standard_normal((m, n))
    return round_to(G, dtype)


def make_planted(m: int, n: int, seed: int, spectrum, dtype: str = "f64"):
    """Returns (G, U, V) with G = U diag(spectrum) V^T exactly planted (before rounding)."""
    rng = np.random.default_rng(seed)
    k = len(spectrum)
    U = random_orthonormal(m, k, rng)
    V = random_orthonormal(n, k, rng)
    G = (U * np.asarray(spectrum, np.float64)) @ V.T
    return round_to(G, dtype), U, V


def make_rotating(m: int, n: int, seed: int, spectrum, drift: float, t: int, noise: float = 0.0, dtype: str = "f64"):
    """Gradient t of a sequence whose singular subspaces turn slowly (what makes a warm-started refresh pay):
    G_t = U_t diag(spectrum) V_t^T + noise, with U_t = orth(U_0 + t drift E_u), V_t likewise, E fixed Gaussian
    matrices: consecutive left (right) subspaces are about `drift` * sqrt(m) (sqrt(n)) radians apart."""
    rng = np.random.default_rng(seed)
    k = len(spectrum)
    U0, V0 = random_orthonormal(m, k, rng), random_orthonormal(n, k, rng)
    Eu, Ev = rng.standard_normal((m, k)), rng.standard_normal((n, k))
    U, _ = np.linalg.qr(U0 + t * drift * Eu)
    V, _ = np.linalg.qr(V0 + t * drift * Ev)
    G = (U * np.asarray(spectrum, np.float64)) @ V.T
    if noise:
        G = G + noise * np.random.default_rng(seed + 1 + t).standard_normal((m, n))
    return round_to(G, dtype)


def make_weight(m: int, n: int, seed: int, dtype: str = "f32", std: float = 0.02) -> np.ndarray:
    rng = np.random.default_rng(seed)
    return round_to(std * rng.standard_normal((m, n)), dtype)


def make_gradient_torch(m: int, n: int, seed: int, p: float, noise: float, device, dtype):
    """Same recipe generated with torch on `device` (for sizes where host generation is slow).

    Not bit-identical to `make_gradient`; used where no CPU copy is compared.
    """
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(seed & 0x7FFFFFFFFFFFFFFF)
    k = min(m, n)
    U, _ = torch.linalg.qr(torch.randn(m, k, generator=g, device=device, dtype=torch.float32))
    V, _ = torch.linalg.qr(torch.randn(n, k, generator=g, device=device, dtype=torch.float32))
    s = torch.arange(1, k + 1, device=device, dtype=torch.float32) ** (-p)
    G = (U * s) @ V.T
    del U, V
    G.add_(torch.randn(m, n, generator=g, device=device, dtype=torch.float32), alpha=noise)
    return G.to(dtype)
