"""Pins for the MXFP8 form of the fallback (Section 3.4; Section 4 "Implementation Details"): a hand-worked
group, the closed-form scale rule, an independent library codec (ml_dtypes) driven by numpy, idempotence,
and the GEMM against a dense double-precision product of the dequantized operands and brute force."""
import os

import ml_dtypes
import numpy as np

from paper_2604_12782_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _gold():
    out = {}
    with open(os.path.join(GOLD, "mxfp8_group_vector.txt")) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                k, *v = line.split()
                out.setdefault(k, []).append(v)
    return out


def _sf_of(oracle, sf, M, K):
    """scale bytes as [M, K/32] through brute-force use of the index function (pinned on its own elsewhere)"""
    return np.array([[sf[oracle.sf_index(r, g, K)] for g in range(K // 32)] for r in range(M)], np.uint8)


def test_worked_group_vector(oracle):
    g = _gold()
    x = np.array([float(v) for v in g["x"][0]], np.float32)
    want = np.array([int(b, 16) for b in g["bytes"][0]], np.uint8)
    X = np.zeros((1, 128), np.float32)
    X[0, 32:64] = x                      # second group of the row: the others are all-zero groups
    x8, sf = oracle.mxfp8_quantize(synth.f32_to_bf16_bits(X))
    assert np.array_equal(x8[0, 32:64], want)
    codes = _sf_of(oracle, sf, 1, 128)[0]
    assert codes[1] == int(g["scale_code"][0][0]) and codes[0] == 0 and codes[2] == 0
    assert not x8[0, :32].any() and not x8[0, 64:].any()
    k = int(g["shift"][0][0])
    x8b, sfb = oracle.mxfp8_quantize(synth.f32_to_bf16_bits(X * 2.0 ** k))
    assert np.array_equal(x8b, x8) and _sf_of(oracle, sfb, 1, 128)[0, 1] == int(g["shift_scale_code"][0][0])
    for amax, code in g["spot"]:
        assert oracle.e8m0_from_amax_emax(float(amax), 8) == int(code), amax


def test_scale_rule_closed_form_on_all_bf16(oracle):
    bits = np.arange(1, 0x7F80, dtype=np.uint32).astype(np.uint16)   # positive finite non-zero
    vals = synth.bf16_bits_to_f64(bits)
    for b, v in zip(bits[::37], vals[::37]):
        assert oracle.e8m0_from_amax_emax(v, 8) == max(int(b >> 7) - 8, 0)
    # emax = 2 reproduces the MXFP4 rule
    for v in (6.0, 1.0, 0.02, 3.99):
        assert oracle.e8m0_from_amax_emax(v, 2) == oracle.e8m0_from_amax(v)


def _library_mxfp8(Xbits):
    """The same quantizer from numpy + ml_dtypes: floor(log2) via frexp, clip to +-448, library E4M3 rounding."""
    x = synth.bf16_bits_to_f64(Xbits)
    M, K = x.shape
    g = x.reshape(M, K // 32, 32)
    amax = np.abs(g).max(axis=2)
    _, ex = np.frexp(amax)
    code = np.where(amax > 0, np.clip(ex - 1 - 8 + 127, 0, 254), 0)
    v = g * np.exp2(127.0 - code)[:, :, None]
    v = np.clip(v, -448.0, 448.0).astype(np.float32)
    return v.astype(ml_dtypes.float8_e4m3fn).view(np.uint8).reshape(M, K), code.astype(np.uint8)


def test_quantizer_matches_library_codec(oracle):
    rng = np.random.default_rng(5)
    X = rng.standard_t(3, size=(70, 256)).astype(np.float32)
    X[3] *= 1e-20                      # tiny rows: E8M0 clamps, subnormal codes
    X[4] *= 1e20
    X[5, 32:64] = 0.0                  # an all-zero group
    X[6, ::2] *= -1.0
    Xb = synth.f32_to_bf16_bits(X)
    x8, sf = oracle.mxfp8_quantize(Xb)
    lib8, libcode = _library_mxfp8(Xb)
    assert np.array_equal(_sf_of(oracle, sf, 70, 256), libcode)
    assert np.array_equal(x8, lib8)
    # every group with a non-zero maximum reaches the top binade or saturates: |code| >= 0x78 (256)
    top = (x8.reshape(70, 8, 32) & 0x7F).max(axis=2)
    nz = np.abs(synth.bf16_bits_to_f64(Xb)).reshape(70, 8, 32).max(axis=2) > 1e-30
    assert (top[nz] >= 0x78).all() and (top[nz] <= 0x7E).all()


def _dequant(oracle, x8, sf, M, K):
    vals = np.arange(256, dtype=np.uint8).view(ml_dtypes.float8_e4m3fn).astype(np.float64)
    codes = _sf_of(oracle, sf, M, K).astype(np.int64)
    return (vals[x8].reshape(M, K // 32, 32) * np.exp2(codes - 127.0)[:, :, None]).reshape(M, K)


def test_quantizer_is_idempotent(oracle):
    c = synth.fp8_linear_case(2, 33, 256, 8)
    x8, sf = oracle.mxfp8_quantize(c["X"])
    d = _dequant(oracle, x8, sf, 33, 256)
    x8b, sfb = oracle.mxfp8_quantize(synth.f32_to_bf16_bits(d.astype(np.float32)))
    # dequantized values have at most 4 significant bits: exact in bf16
    assert np.array_equal(x8b, x8) and np.array_equal(sfb, sf)


def test_gemm_equals_dense_product_of_dequantized_operands(oracle):
    c = synth.fp8_linear_case(3, 37, 384, 50)
    Y, T, (x8, sfa), (w8, sfw) = oracle.mxfp8_linear(c["X"], c["W"])
    dx = _dequant(oracle, x8, sfa, 37, 384)
    dw = _dequant(oracle, w8, sfw, 50, 384)
    ref = dx @ dw.T
    assert np.allclose(Y, ref, rtol=1e-12, atol=1e-12 * np.abs(ref).max())
    assert np.allclose(T, np.abs(dx) @ np.abs(dw).T, rtol=1e-12)
    # sampled rows give the same numbers as the full call
    rows = np.array([36, 0, 5], np.int32)
    Y2, _ = oracle.mxfp8_gemm(x8, sfa, w8, sfw, rows)
    assert np.array_equal(Y2, Y[rows])


def test_gemm_bruteforce_tiny(oracle):
    rng = np.random.default_rng(9)
    X = synth.f32_to_bf16_bits(rng.normal(size=(3, 128)).astype(np.float32))
    W = synth.f32_to_bf16_bits((rng.normal(size=(2, 128)) * 0.05).astype(np.float32))
    Y, T, (x8, sfa), (w8, sfw) = oracle.mxfp8_linear(X, W)
    for m in range(3):
        for n in range(2):
            acc = 0.0
            for g in range(4):
                s = 2.0 ** (int(sfa[oracle.sf_index(m, g, 128)]) - 127) * 2.0 ** (int(sfw[oracle.sf_index(n, g, 128)]) - 127)
                p = 0.0
                for c in range(32 * g, 32 * g + 32):
                    p += oracle.e4m3_decode(int(x8[m, c])) * oracle.e4m3_decode(int(w8[n, c]))
                acc += s * p
            assert Y[m, n] == acc


def test_error_ordering_against_4bit_and_per_token_forms(oracle):
    """On diffuse heavy-tailed inputs (the W2 case) the 8-bit micro-scaled product is far closer to the exact
    product than unprotected MXFP4, which is why the fallback exists (Section 3.4)."""
    c = synth.fp8_linear_case(4, 64, 512, 48)
    x = synth.bf16_bits_to_f64(c["X"])
    w = synth.bf16_bits_to_f64(c["W"])
    exact = x @ w.T
    Y8, *_ = oracle.mxfp8_linear(c["X"], c["W"])
    lut = np.full((512 // 32, 1), -1, np.int8)
    Y4, *_ = oracle.linear(c["X"], c["W"], lut)
    e8 = np.linalg.norm(Y8 - exact) / np.linalg.norm(exact)
    e4 = np.linalg.norm(Y4 - exact) / np.linalg.norm(exact)
    assert e8 < 0.05 and e8 < e4 / 3
