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


# ---- the residual update in front of the norm

def _bf16_value(b):
    """Exact rational value of a finite bf16 bit pattern."""
    from fractions import Fraction
    s = -1 if b & 0x8000 else 1
    e, m = (b >> 7) & 0xFF, b & 0x7F
    if e == 0:
        return s * Fraction(m, 1 << 7) * Fraction(2) ** -126
    return s * (1 + Fraction(m, 1 << 7)) * Fraction(2) ** (e - 127)


def _round_to_bf16(q):
    """Nearest bf16 (ties to even) of an exact rational, by search over the bit patterns of the right sign."""
    from fractions import Fraction
    if q == 0:
        return None   # sign of zero: checked separately
    sign = 0x8000 if q < 0 else 0
    a = abs(q)
    lo, hi = 0, 0x7F80          # magnitudes are ordered like their bit patterns; 0x7F80 stands for 2^128
    top = Fraction(2) ** 128
    val = lambda b: top if b == 0x7F80 else _bf16_value(b)
    while hi - lo > 1:
        mid = (lo + hi) // 2
        if val(mid) <= a:
            lo = mid
        else:
            hi = mid
    dl, dh = a - val(lo), val(hi) - a
    pick = lo if dl < dh else hi if dh < dl else (lo if lo % 2 == 0 else hi)
    return sign | pick


def test_residual_add_against_rational_arithmetic(oracle):
    rng = np.random.default_rng(5)
    a = rng.integers(0, 0x7F80, size=3000).astype(np.uint16) | (rng.integers(0, 2, size=3000).astype(np.uint16) << 15)
    b = rng.integers(0, 0x7F80, size=3000).astype(np.uint16) | (rng.integers(0, 2, size=3000).astype(np.uint16) << 15)
    # near-equal exponents (cancellation, carries, ties) are rare among random patterns: plant them
    b[:1500] = (a[:1500] & 0x8000) ^ (rng.integers(0, 2, size=1500).astype(np.uint16) << 15) | \
        np.clip((a[:1500] & 0x7FFF).astype(np.int32) + rng.integers(-1200, 1200, size=1500), 0, 0x7F7F).astype(np.uint16)
    got = oracle.residual_add(a.reshape(1, -1), b.reshape(1, -1)).ravel()
    for x, y, g in zip(a, b, got):
        q = _bf16_value(int(x)) + _bf16_value(int(y))
        want = _round_to_bf16(q)
        if want is None:
            assert int(g) & 0x7FFF == 0
        else:
            assert int(g) == want, (hex(int(x)), hex(int(y)), hex(int(g)), hex(want))


def test_residual_add_special_cases(oracle):
    one, ulp = 0x3F80, 2.0 ** -7
    cases = [
        (bits([1.0]), bits([0.0]), 0x3F80),
        (bits([1.0]), bits([2.0 ** -8]), 0x3F80),            # tie -> even
        (bits([1.0 + ulp]), bits([2.0 ** -8]), 0x3F82),      # tie from an odd pattern -> up to the even one
        (bits([1.0]), bits([2.0 ** -8 + 2.0 ** -15]), 0x3F81),
        (bits([1.0]), bits([-1.0]), 0x0000),                 # exact cancellation: +0
        (bits([3.0e38]), bits([3.0e38]), 0x7F80),            # overflow -> +inf
        (bits([1.0]), bits([1e-30]), 0x3F80),
        (bits([2.0 ** -126]), bits([-(2.0 ** -127)]), 0x0040),   # into the subnormals, exact
    ]
    for h, r, want in cases:
        got = int(oracle.residual_add(h.reshape(1, 1), r.reshape(1, 1))[0, 0])
        assert got == want, (hex(got), hex(want))
    rng = np.random.default_rng(6)
    H, R = bits(rng.standard_normal((4, 64))), bits(rng.standard_normal((4, 64)) * 0.1)
    assert np.array_equal(oracle.residual_add(H, R), oracle.residual_add(R, H))            # commutative
    assert np.array_equal(oracle.residual_add(H, bits(np.zeros((4, 64)))), H)


def test_add_rmsnorm_is_the_norm_of_the_updated_stream(oracle):
    rng = np.random.default_rng(7)
    H, R = bits(rng.standard_normal((5, 256)) * 3), bits(rng.standard_normal((5, 256)))
    g = bits(rng.uniform(0.5, 2.0, 256))
    Hs, Y = oracle.add_rmsnorm(H, R, g, 1e-6)
    assert np.array_equal(Hs, oracle.residual_add(H, R))
    assert np.array_equal(Y, oracle.rmsnorm(Hs, g, 1e-6))
    # against torch: float64 sum rounded through torch's own bf16 conversion, then torch's rms_norm
    hs_t = (torch.from_numpy(synth.bf16_bits_to_f64(H)) + torch.from_numpy(synth.bf16_bits_to_f64(R))).to(torch.bfloat16)
    assert np.array_equal(hs_t.view(torch.int16).numpy().view(np.uint16), Hs)
