"""Pins of the RMSNorm oracle (the producer that is fused in front of Algorithm 2).

None of them re-types the oracle's formula: a library routine (torch's float64 rms_norm), closed forms whose
results are exact, an invariance, and hand-worked roundings of the double -> bf16 step.
"""
import numpy as np
import torch

from paper_2604_12782_b200 import synth


def bits(a):
    return synth.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


def test_double_to_bf16_rounding_hand_worked(oracle):
    cases = [
        (1.0, 0x3F80),
        (1 + 2.0 ** -8, 0x3F80),                 # tie between 0x3F80 and 0x3F81 -> even
        (1 + 3 * 2.0 ** -8, 0x3F82),             # tie between 0x3F81 and 0x3F82 -> even
        (1 + 2.0 ** -8 + 2.0 ** -40, 0x3F81),    # just above the tie (a float32 detour would lose the 2^-40)
        (1 + 2.0 ** -8 - 2.0 ** -40, 0x3F80),
        (-0.0, 0x8000),
        (2.0 ** -134, 0x0000),                   # half the smallest subnormal: tie -> 0
        (-(2.0 ** -134) * (1 + 2.0 ** -30), 0x8001),
        (1.5 * 2.0 ** -133, 0x0002),
        (2.0 ** -126, 0x0080),                   # smallest normal
        (float(np.float32(3.3895314e38)), 0x7F7F),
        (2.0 ** 128 * (1 - 2.0 ** -9), 0x7F80),  # tie at the top of the range rounds to infinity
        (2.0 ** 128 * (1 - 2.0 ** -9) * (1 - 2.0 ** -40), 0x7F7F),
        (-1e39, 0xFF80),
    ]
    got = oracle.f64_to_bf16_bits(np.array([c[0] for c in cases]))
    assert [int(g) for g in got] == [c[1] for c in cases]


def test_constant_rows_and_unit_rows_closed_form(oracle):
    K = 256
    rng = np.random.default_rng(0)
    gamma = bits(rng.uniform(0.5, 2.0, K))
    # eps = 0, every element +-1: mean square 1, so y = +-gamma exactly
    sign = rng.choice([-1.0, 1.0], size=(3, K))
    got = oracle.rmsnorm(bits(sign), gamma, 0.0)
    want = gamma[None, :] ^ np.where(sign < 0, 0x8000, 0).astype(np.uint16)
    assert np.array_equal(got, want)
    # eps = 0, every element c (any bf16 value): y = sign(c) * gamma, whatever |c|
    for c in (3.0, -0.0078125, 1.5e-30, 2.0e30):
        got = oracle.rmsnorm(bits(np.full((1, K), c)), gamma, 0.0)
        want = gamma ^ np.uint16(0x8000 if c < 0 else 0)
        assert np.array_equal(got[0], want), c


def test_single_nonzero_per_row_closed_form(oracle):
    # one element a, the rest 0, K = 256, eps = 0: mean square a^2/256, r = 16/|a|, y = 16 sign(a) gamma there, 0 elsewhere
    K = 256
    gamma = bits(np.linspace(0.25, 4.0, K))
    H = np.zeros((4, K), np.float32)
    pos, val = [0, 17, 255, 100], [5.0, -0.375, 7e-20, -3e20]
    for m in range(4):
        H[m, pos[m]] = val[m]
    got = synth.bf16_bits_to_f64(oracle.rmsnorm(bits(H), gamma, 0.0))
    g = synth.bf16_bits_to_f64(gamma)
    for m in range(4):
        want = np.zeros(K)
        want[pos[m]] = 16.0 * np.sign(val[m]) * g[pos[m]]      # 16 * gamma is a bf16 value: exact
        assert np.array_equal(got[m], want)


def test_power_of_two_scaling_is_invisible_at_eps_zero(oracle):
    rng = np.random.default_rng(1)
    H = rng.standard_normal((8, 384)).astype(np.float32)
    gamma = bits(rng.uniform(0.5, 1.5, 384))
    base = oracle.rmsnorm(bits(H), gamma, 0.0)
    for k in (-20, 3, 40):
        assert np.array_equal(oracle.rmsnorm(bits(np.ldexp(H, k)), gamma, 0.0), base)


def test_against_torch_float64_rms_norm(oracle):
    rng = np.random.default_rng(2)
    M, K, eps = 64, 512, 1e-6
    Hb = bits(rng.standard_t(4, size=(M, K)) * rng.uniform(0.01, 30.0, size=(M, 1)))
    gb = bits(rng.uniform(0.2, 3.0, K))
    x = torch.from_numpy(synth.bf16_bits_to_f64(Hb))
    g = torch.from_numpy(synth.bf16_bits_to_f64(gb))
    y = torch.nn.functional.rms_norm(x, (K,), weight=g, eps=float(np.float32(eps)))
    # the library works in double throughout, the oracle rounds r and the two products to fp32: the bf16 results
    # agree unless the double value sits within ~2^-23 (relative) of a bf16 rounding boundary, and then by one unit
    want = oracle.f64_to_bf16_bits(y.numpy())
    got = oracle.rmsnorm(Hb, gb, eps)
    diff = np.abs(got.astype(np.int32) - want.astype(np.int32))
    assert diff.max() <= 1
    assert np.count_nonzero(diff) <= 1e-3 * got.size
    # and the result has unit mean square before gamma, to bf16 accuracy
    z = synth.bf16_bits_to_f64(got) / synth.bf16_bits_to_f64(gb)[None, :]
    assert np.allclose((z * z).mean(axis=1), 1.0, atol=5e-3)


def test_eps_matters_for_small_rows(oracle):
    K, eps = 128, 1e-5
    gamma = bits(np.ones(K))
    H = bits(np.full((1, K), 2.0 ** -10))
    got = synth.bf16_bits_to_f64(oracle.rmsnorm(H, gamma, eps))[0, 0]
    want = 2.0 ** -10 / np.sqrt(2.0 ** -20 + float(np.float32(eps)))
    assert abs(got - want) <= 2.0 ** -9 * want      # half a bf16 ulp, relative
    assert got < 0.5                                   # without eps it would be 1
