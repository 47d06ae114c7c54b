"""Seeded synthetic input generators shared by the tests, the smoke check and the benchmark.

This module holds none of the method's arithmetic: it only draws random tensors (numpy's PCG64
``default_rng``) with the shapes and value distributions of the paper's statistical workload and
of a training step's activations / weights / gradients, and converts between fp32 and bf16 bit
patterns.  Both the CUDA path and the CPU oracle consume the very same host arrays.
"""
from __future__ import annotations

import numpy as np


def _rng(seed: int, stream: int = 0) -> np.random.Generator:
    return np.random.default_rng([int(seed), int(stream)])


# ---- dtype plumbing -----------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest-even) and return the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to fp32 exactly."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


# ---- element distributions -----------------------------------------------------------------------
def normal(n, seed=0, stream=0, sigma=1.0) -> np.ndarray:
    return (_rng(seed, stream).standard_normal(n) * sigma).astype(np.float32)


def laplace(n, seed=0, stream=0, scale=1.0) -> np.ndarray:
    return _rng(seed, stream).laplace(0.0, scale, n).astype(np.float32)


def student_t(n, seed=0, stream=0, nu=3.0) -> np.ndarray:
    return _rng(seed, stream).standard_t(nu, n).astype(np.float32)


def normal_with_outliers(n, seed=0, stream=0, frac=1e-3, gain=100.0) -> np.ndarray:
    """N(0,1) with an i.i.d. Bernoulli(frac) subset of elements multiplied by ``gain``."""
    g = _rng(seed, stream)
    x = g.standard_normal(n)
    mask = g.random(n) < frac
    x[mask] *= gain
    return x.astype(np.float32)


def variable_variance_vectors(nvec, length, seed=0, stream=0) -> np.ndarray:
    """Vectors X ~ N(0, |z|) with one z ~ N(0,1) per vector (the design-sweep distribution)."""
    g = _rng(seed, stream)
    var = np.abs(g.standard_normal((nvec, 1)))
    return (g.standard_normal((nvec, length)) * np.sqrt(var)).astype(np.float32)


SWEEP_DISTRIBUTIONS = ("normal", "laplace", "student_t3", "normal_outliers")


def sweep_distribution(name: str, n: int, seed: int = 0) -> np.ndarray:
    """The four distributions of the design-space sweep workload, by name."""
    idx = SWEEP_DISTRIBUTIONS.index(name)
    return (normal, laplace, student_t, normal_with_outliers)[idx](n, seed=seed, stream=100 + idx)


# ---- matrix workloads ----------------------------------------------------------------------------
def outlier_channel_matrix(rows, cols, seed=0, stream=0, dist="laplace", frac=0.01, gain=50.0, sigma=1.0):
    """[rows, cols] fp32 matrix with a seeded choice of round(frac*cols) columns scaled by ``gain``."""
    g = _rng(seed, stream)
    if dist == "laplace":
        x = g.laplace(0.0, sigma, (rows, cols)).astype(np.float32)
    else:
        x = (g.standard_normal((rows, cols)) * sigma).astype(np.float32)
    nout = int(round(frac * cols))
    if nout:
        chosen = g.choice(cols, size=nout, replace=False)
        x[:, chosen] *= np.float32(gain)
    return x


def normal_matrix(rows, cols, seed=0, stream=0, sigma=1.0) -> np.ndarray:
    return (_rng(seed, stream).standard_normal((rows, cols)) * sigma).astype(np.float32)


# ---- adversarial / edge-case tensors for parity tests --------------------------------------------
def edge_case_values(n, seed=0, stream=0) -> np.ndarray:
    """Finite fp32 values that stress exponent extremes, ties, signed zeros and subnormals."""
    g = _rng(seed, stream)
    kinds = g.integers(0, 8, n)
    exps = g.integers(-149, 128, n)
    mant = g.integers(0, 1 << 24, n)
    x = np.ldexp(mant.astype(np.float64) / (1 << 23), exps.clip(-149, 126)).astype(np.float32)
    x = np.where(kinds == 0, 0.0, x)
    x = np.where(kinds == 1, np.ldexp(1.0, exps.clip(-149, 127)), x)                     # powers of two
    x = np.where(kinds == 2, np.ldexp(g.integers(0, 64, n) + 0.5, g.integers(-20, 20, n)), x)  # half-way cases
    x = np.where(kinds == 3, g.standard_normal(n), x)
    x = np.where(kinds == 4, np.ldexp(mant.astype(np.float64), -149), x)                 # subnormals
    x = np.where(kinds == 5, g.standard_normal(n) * 1e30, x)
    x = np.where(kinds == 6, g.standard_normal(n) * 1e-30, x)
    x = x.astype(np.float32)
    x = np.where(np.isfinite(x), x, np.float32(3.0e38)).astype(np.float32)
    sign = g.integers(0, 2, n).astype(np.uint32) << 31
    return (x.view(np.uint32) | sign).view(np.float32)
