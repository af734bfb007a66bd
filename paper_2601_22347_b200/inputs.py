"""Seeded synthetic activations for the PeRQ rotate+quantize path.

This module only draws random numbers and rounds them to bf16; it holds none of the
method's arithmetic (no Hadamard, no scales, no codes), so both the CPU oracle's tests
and the CUDA path's tests may import it.

The five workloads are stand-ins for the activations the paper feeds its online block
rotation (down-projection inputs and hidden states of Llama-3 1B / 8B; Sec. 5 "Models &
Datasets", Table "hadamard-op-counts" for the layer widths).  The real activations need
model checkpoints and a text corpus; here every tensor is drawn from a stated
distribution with a stated seed, with a few "outlier channels" scaled up to mimic the
massive-activation channels the paper's Figure 1 shows.

bf16 tensors are returned as numpy uint16 arrays holding the raw bit patterns
(row-major [T, d]); `bf16_to_f64` widens them exactly.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np

SEED_BASE = 22347_000


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even), return uint16 bit patterns."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = (u + 0x7FFF + lsb) >> 16
    return r.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to float32 exactly."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to float64 exactly."""
    return bf16_bits_to_f32(bits).astype(np.float64)


@dataclass
class Workload:
    """One synthetic call: activations, optional permutation and the call's parameters."""
    name: str
    x: np.ndarray                      # uint16 [T, d], bf16 bit patterns
    perm: Optional[np.ndarray]         # int32 [d] or None (identity)
    b: int                             # Hadamard block size
    fmt: str                           # "int4" | "mxfp4"
    group: int                         # 0 = per-token scale; else scale group size
    seed: int
    outlier_channels: np.ndarray = field(default_factory=lambda: np.zeros(0, np.int64))

    @property
    def T(self) -> int:
        return int(self.x.shape[0])

    @property
    def d(self) -> int:
        return int(self.x.shape[1])


def _seed(cfg: int, variant: int) -> int:
    return SEED_BASE + 10 * cfg + variant


def _finish(vals: np.ndarray, rng: np.random.Generator, n_out: int, factor: float):
    """Scale `n_out` channels (chosen after the values were drawn) and round to bf16."""
    d = vals.shape[1]
    ch = np.sort(rng.choice(d, size=n_out, replace=False)) if n_out > 0 else np.zeros(0, np.int64)
    vals = vals.astype(np.float32)
    if n_out > 0:
        vals[:, ch] *= np.float32(factor)
    return f32_to_bf16_bits(vals), ch


def gaussian_outliers(T: int, d: int, n_out: int, factor: float, seed: int):
    """N(0,1) per element, `n_out` channels multiplied by `factor`."""
    rng = np.random.default_rng(seed)
    return _finish(rng.standard_normal((T, d)), rng, n_out, factor)


def student_t_outliers(T: int, d: int, nu: float, n_out: int, factor: float, seed: int):
    """Student-t(nu) per element, `n_out` channels multiplied by `factor`."""
    rng = np.random.default_rng(seed)
    return _finish(rng.standard_t(nu, size=(T, d)), rng, n_out, factor)


def laplace_outliers(T: int, d: int, n_out: int, factor: float, seed: int):
    """Laplace(0,1) per element, `n_out` channels multiplied by `factor`."""
    rng = np.random.default_rng(seed)
    return _finish(rng.laplace(0.0, 1.0, size=(T, d)), rng, n_out, factor)


def swiglu_outliers(T: int, d: int, n_out: int, factor: float, seed: int):
    """SiLU(a)*c with a, c ~ N(0,1): the shape of an MLP down-projection input."""
    rng = np.random.default_rng(seed)
    a = rng.standard_normal((T, d))
    c = rng.standard_normal((T, d))
    return _finish(a / (1.0 + np.exp(-a)) * c, rng, n_out, factor)


def random_perm(d: int, seed: int) -> np.ndarray:
    return np.random.default_rng(seed).permutation(d).astype(np.int32)


# ----------------------------------------------------------------------------------------
# The five workloads.  `T` can be overridden (rows are independent, so a smaller T is the
# same workload with fewer tokens); everything else follows the configuration list.
# ----------------------------------------------------------------------------------------

def config1(T: int = 256, variant: int = 0) -> Workload:
    """T x 2048, N(0,1), 8 outlier channels x50, identity perm, b=16, INT4 per-token."""
    s = _seed(1, variant)
    x, ch = gaussian_outliers(T, 2048, 8, 50.0, s)
    return Workload("cfg1", x, None, 16, "int4", 0, s, ch)


def config2(T: int = 4096, b: int = 32, variant: int = 0) -> Workload:
    """Llama-3-1B hidden: T x 2048, Student-t(3), 16 channels x100, random perm, INT4 g=128."""
    s = _seed(2, variant)
    x, ch = student_t_outliers(T, 2048, 3.0, 16, 100.0, s)
    return Workload("cfg2", x, random_perm(2048, s + 1), b, "int4", 128, s, ch)


def config3(T: int = 4096, variant: int = 0) -> Workload:
    """Llama-3-1B down-proj input: T x 8192, SiLU(a)*c, 32 channels x30, b=32, MXFP4.

    The permutation of this workload is produced by the method itself (channel-mass
    statistic + greedy assignment), so `perm` is None here and the caller fills it in.
    """
    s = _seed(3, variant)
    x, ch = swiglu_outliers(T, 8192, 32, 30.0, s)
    return Workload("cfg3", x, None, 32, "mxfp4", 32, s, ch)


def config4(T: int = 16384, b: int = 32, fmt: str = "int4", variant: int = 0) -> Workload:
    """Llama-3-8B hidden: T x 4096, Laplace(0,1), 0.1% of channels x200, no perm."""
    s = _seed(4, variant)
    x, ch = laplace_outliers(T, 4096, int(round(0.001 * 4096)), 200.0, s)
    return Workload("cfg4", x, None, b, fmt, 32 if fmt == "mxfp4" else 0, s, ch)


def config5(T: int = 1024, b: int = 32, variant: int = 0) -> Workload:
    """Llama-3-8B down-proj input: T x 14336, N(0,1), 64 channels x50, random perm, INT4 g=128."""
    s = _seed(5, variant)
    x, ch = gaussian_outliers(T, 14336, 64, 50.0, s)
    return Workload("cfg5", x, random_perm(14336, s + 1), b, "int4", 128, s, ch)
