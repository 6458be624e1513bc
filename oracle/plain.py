"""Plain definitions of the two producers, all in double with one rounding at the end.

TEST INFRASTRUCTURE ONLY, like everything in this package.

The oracle functions the CUDA kernels are compared with bit for bit (`oracle.rmsnorm`, `oracle.swiglu`) fix the
element-wise arithmetic in fp32 steps, because the values they produce decide integer codes further down
(Algorithm 2's scale and E2M1 codes, the E4M3 codes of the Section 3.4 fallback).  The functions here are what
those step-wise definitions approximate: the textbook formula evaluated in IEEE double and rounded once to
bf16.  The tests bound the step-wise oracle, and the kernels, against them (one bf16 unit), so that the
step-wise definitions cannot drift with an implementation.

    rmsnorm_plain:  y[m,k] = bf16( x[m,k] * gamma[k] / sqrt( mean_k x[m,k]^2 + eps ) )
    swiglu_plain:   h[m,i] = bf16( g / (1 + exp(-g)) * u ),   g = GU[m,i], u = GU[m,I+i]
"""
from __future__ import annotations

import math

import numpy as np

from .rmsnorm import _bf16_bits_to_f64, f64_to_bf16_bits


def rmsnorm_plain_f64(H: np.ndarray, gamma: np.ndarray, eps: float) -> np.ndarray:
    """The normalized rows as doubles, before the one rounding to bf16."""
    x = _bf16_bits_to_f64(H)
    g = _bf16_bits_to_f64(gamma)
    K = x.shape[1]
    ms = np.array([math.fsum(row) for row in x * x]) / K
    with np.errstate(divide="ignore", over="ignore", invalid="ignore"):
        return x * g[None, :] / np.sqrt(ms + float(np.float32(eps)))[:, None]


def rmsnorm_plain(H: np.ndarray, gamma: np.ndarray, eps: float) -> np.ndarray:
    """H [M, K] bf16 bits, gamma [K] bf16 bits -> bf16 bits [M, K]; every operation in double."""
    return f64_to_bf16_bits(rmsnorm_plain_f64(H, gamma, eps))


def swiglu_plain_f64(GU: np.ndarray, I: int) -> np.ndarray:
    """silu(g) * u as doubles, before the one rounding to bf16."""
    v = _bf16_bits_to_f64(GU)
    g, u = v[:, :I], v[:, I:2 * I]
    with np.errstate(over="ignore", invalid="ignore", under="ignore"):
        return g / (1.0 + np.exp(-g)) * u


def swiglu_plain(GU: np.ndarray, I: int) -> np.ndarray:
    """GU [M, >= 2I] bf16 bits (gate columns [0, I), up columns [I, 2I)) -> bf16 bits [M, I]; double throughout."""
    return f64_to_bf16_bits(swiglu_plain_f64(GU, I))


def bf16_units_apart(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    """Distance between bf16 bit patterns counted in representable values (+0 and -0 coincide)."""
    def ordinal(x):
        x = np.asarray(x, dtype=np.uint16).astype(np.int64)
        mag = x & 0x7FFF
        return np.where(x >> 15, -mag, mag)
    return np.abs(ordinal(a) - ordinal(b))
