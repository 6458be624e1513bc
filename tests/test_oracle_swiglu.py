"""Pins of the SwiGLU oracle (the producer fused in front of the FP8 quantizer of the down projection).

The arithmetic is a fixed sequence of fp32 operations (so that the CUDA kernel can reproduce it bit for bit); what
pins it is the mathematics it approximates: the library exponential, torch's float64 silu, exact special values,
the identity silu(g) - silu(-g) = g.
"""
import math

import numpy as np
import torch

from paper_2604_12782_b200 import synth


def bits(a):
    return synth.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


def test_exp32_against_the_library_exponential(oracle):
    worst = 0.0
    for z in np.linspace(-44.0, 87.0, 20001):   # t = z log2(e) inside the clamp [-64, 126]
        z = float(np.float32(z))
        worst = max(worst, abs(oracle.exp32(z) - math.exp(z)) / math.exp(z))
    assert worst < 8e-6                      # z * log2(e) rounded to fp32 (~2^-24 |t| absolute in t) + the degree-5 truncation (2.4e-6)
    for z in np.linspace(-1.0, 1.0, 2001):   # small arguments: the truncation error of the polynomial dominates
        z = float(np.float32(z))
        assert abs(oracle.exp32(z) - math.exp(z)) <= 3.5e-6 * math.exp(z)
    assert oracle.exp32(0.0) == 1.0
    assert abs(oracle.exp32(1.0) - math.e) < 3.5e-6 * math.e
    assert oracle.exp32(200.0) == oracle.exp32(126.0 / 1.4426950408889634 + 1.0)      # clamped at 2^126
    assert 0.0 < oracle.exp32(-200.0) <= 2.0 ** -64 * 1.0001                            # and at 2^-64


def test_silu32_special_values_and_identity(oracle):
    assert oracle.silu32(0.0) == 0.0
    for g in (45.0, 100.0, float(np.float32(3e30))):   # exp(-g) is dropped: silu(g) = g exactly
        assert oracle.silu32(g) == g
    assert -2e-36 < oracle.silu32(-100.0) < 0.0          # -100 / (1 + 2^126): far below anything bf16 h can show
    for g in np.linspace(0.01, 30.0, 500):
        g = float(np.float32(g))
        assert abs(oracle.silu32(g) - g / (1.0 + math.exp(-g))) <= 6e-6 * g
        assert abs((oracle.silu32(g) - oracle.silu32(-g)) - g) <= 1e-5 * g     # sigma(g) + sigma(-g) = 1


def test_swiglu_against_torch_float64(oracle):
    rng = np.random.default_rng(0)
    M, I = 48, 640
    GU = bits(np.concatenate([rng.standard_normal((M, I)) * 3.0, rng.standard_normal((M, I))], axis=1))
    got = oracle.swiglu(GU, I)
    g = torch.from_numpy(synth.bf16_bits_to_f64(GU[:, :I]))
    u = torch.from_numpy(synth.bf16_bits_to_f64(GU[:, I:]))
    want = oracle.f64_to_bf16_bits((torch.nn.functional.silu(g) * u).numpy())
    diff = np.abs(got.astype(np.int32) - want.astype(np.int32))
    assert diff.max() <= 1                                  # one bf16 unit where the double value sits at a boundary
    assert np.count_nonzero(diff) <= 5e-3 * got.size


def test_swiglu_layout_and_exact_cases(oracle):
    I = 128
    g = np.zeros((3, I), np.float32)
    u = np.ones((3, I), np.float32)
    g[0] = 64.0                      # silu = g exactly; h = g * u
    u[0] = np.linspace(-2.0, 2.0, I)
    g[1] = np.linspace(-8.0, 8.0, I)  # u = 1: h = bf16(silu32(g))
    g[2] = 0.0                       # h = 0 whatever u is
    u[2] = 1e30
    GU = bits(np.concatenate([g, u], axis=1))
    H = oracle.swiglu(np.concatenate([GU, np.full((3, 8), 0x7FC0, np.uint16)], axis=1), I)   # trailing columns are ignored
    gb, ub = synth.bf16_bits_to_f64(GU[:, :I]), synth.bf16_bits_to_f64(GU[:, I:])
    assert np.array_equal(H[0], oracle.f64_to_bf16_bits(64.0 * ub[0]))
    assert np.array_equal(H[1], oracle.f64_to_bf16_bits(np.array([oracle.silu32(float(x)) for x in gb[1]])))
    assert not H[2].any()
