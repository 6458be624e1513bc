"""CPU oracle of the RMSNorm that feeds the quantizer when the two are fused (the producer of the QKV and
gate/up inputs of a decoder layer; Section 3.3 places Algorithm 2 directly behind the operator that
produces the activations).

TEST INFRASTRUCTURE ONLY, like everything in this package.

Definition (the paper does not state the arithmetic of the producer; this is the usual one: statistics in
high precision, the element-wise part in fp32, one final rounding to bf16):

    r[m]    = fl32( 1 / sqrt( (1/K) sum_k x[m, k]^2 + eps ) )        sum exact, the rest in IEEE double
    y[m, k] = bf16( fl32( fl32( x[m, k] * r[m] ) * gamma[k] ) )       two fp32 multiplications, then nearest-even

with x, gamma bf16 values and eps an fp32 value.  The fused path is this function followed by Algorithm 2
on its output.

residual_add / add_rmsnorm: the residual update of a decoder layer in front of the norm, h' = bf16(h + r).

Pins (tests/test_oracle_rmsnorm.py): torch's float64 rms_norm as the library routine (agreement to one bf16
unit, equality almost everywhere), closed forms (constant rows, one non-zero per row, eps = 0 rows of +-1),
power-of-two scale invariance at eps = 0, hand-worked double -> bf16 roundings (ties, subnormals, overflow,
signed zero).
"""
from __future__ import annotations

import math

import numpy as np


def _bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    u = np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def f64_to_bf16_bits(y: np.ndarray) -> np.ndarray:
    """Nearest bf16 (ties to even) of doubles, in one rounding: scale so that the bf16 quantum of each value
    is 1, round to integer, scale back.  bf16 = 8 significant bits, exponents as fp32 (subnormal quantum
    2^-133, overflow to infinity at 2^128 - 2^119 and above)."""
    y = np.asarray(y, dtype=np.float64)
    _, e = np.frexp(y)                         # |y| in [2^(e-1), 2^e)
    q = np.maximum(e - 8, -133)                # exponent of the quantum
    n = np.rint(np.ldexp(y, -q))               # exact scaling; rint rounds halves to even
    v = np.ldexp(n, q)                         # a bf16 value (or 2^128 after rounding up)
    with np.errstate(over="ignore"):
        f = v.astype(np.float32)               # exact for every finite bf16 value; 2^128 -> inf
    bits = (f.view(np.uint32) >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(y)
    if nan.any():
        bits = np.where(nan, np.uint16(0x7FC0), bits)
    return bits


def rmsnorm(H: np.ndarray, gamma: np.ndarray, eps: float) -> np.ndarray:
    """H [M, K] bf16 bits, gamma [K] bf16 bits, eps -> normalized rows as bf16 bits [M, K]."""
    x = _bf16_bits_to_f64(H)
    g32 = _bf16_bits_to_f64(gamma).astype(np.float32)
    K = x.shape[1]
    ms = np.array([math.fsum(row) for row in x * x]) / K      # squares are exact in double; fsum is the exact sum, rounded once
    with np.errstate(divide="ignore", over="ignore", invalid="ignore"):
        r32 = (1.0 / np.sqrt(ms + float(np.float32(eps)))).astype(np.float32)
        t = x.astype(np.float32) * r32[:, None]                # fp32 product, rounded to nearest
        y = t * g32[None, :]                                   # second fp32 product
    return f64_to_bf16_bits(y.astype(np.float64))              # exact widening, then the one rounding to bf16


def residual_add(H: np.ndarray, R: np.ndarray) -> np.ndarray:
    """The residual update in front of the norm: bf16 bits of the exact sum h + r, rounded once, nearest even.
    The double addition is exact while the exponents differ by fewer than 45 binades; beyond that the smaller
    addend is more than 2^35 times smaller than half a bf16 step of the larger one, which lies on the bf16 grid, so
    it cannot carry the sum across a rounding boundary (checked against rational arithmetic in the tests)."""
    return f64_to_bf16_bits(_bf16_bits_to_f64(H) + _bf16_bits_to_f64(R))


def add_rmsnorm(H: np.ndarray, R: np.ndarray, gamma: np.ndarray, eps: float):
    """-> (H' = residual_add(H, R), rmsnorm(H', gamma, eps))."""
    Hs = residual_add(H, R)
    return Hs, rmsnorm(Hs, gamma, eps)

