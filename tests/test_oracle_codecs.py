"""Pins for the oracle's scalar codecs, scale rule, table handling and scale layout.

Everything here is checked against something other than the oracle itself:
hand-worked vectors (tests/golden), closed forms, an independent library codec
(ml_dtypes) and brute-force numpy indexing.
"""
import os

import ml_dtypes
import numpy as np
import pytest

from paper_2604_12782_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _gold_lines(name):
    out = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                out.append(line.split())
    return out


def all_bf16_finite():
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    vals = synth.bf16_bits_to_f64(bits)
    keep = np.isfinite(vals)
    return bits[keep], vals[keep]


# ----------------------------------------------------------------- E2M1 (pin P1)

def test_e2m1_value_table_roundtrip(oracle):
    expect = [0, .5, 1, 1.5, 2, 3, 4, 6]
    for code in range(16):
        v = oracle.e2m1_decode(code)
        assert abs(v) == expect[code & 7]
        assert np.signbit(v) == bool(code & 8)
        assert oracle.e2m1_encode(v) == code


def test_e2m1_matches_library_codec_on_all_bf16(oracle):
    bits, vals = all_bf16_finite()
    for scale in (1.0, 0.25, 8.0, 2.0 ** -20):
        v = vals * scale
        lib_codes = v.astype(np.float32).astype(ml_dtypes.float4_e2m1fn).view(np.uint8) & 0xF
        mine = np.array([oracle.e2m1_encode(x) for x in v[::7]], dtype=np.uint8)
        assert np.array_equal(mine, lib_codes[::7])


def test_e2m1_ties_and_saturation(oracle):
    # midpoints go to the even code; beyond 6 saturates; sign of zero kept
    for v, code in [(0.25, 0), (0.75, 2), (1.25, 2), (1.75, 4), (2.5, 4), (3.5, 6), (5.0, 6),
                    (5.0001, 7), (6.0, 7), (7.9, 7), (1e30, 7), (-0.0, 8), (-0.1, 8), (-0.26, 9), (-1e9, 15)]:
        assert oracle.e2m1_encode(v) == code, v


# ----------------------------------------------------------------- E8M0 (pin P2)

def test_e8m0_spot_values(oracle):
    for kind, *rest in _gold_lines("scale_and_fp8_vectors.txt"):
        if kind == "e8m0":
            assert oracle.e8m0_from_amax(float(rest[0])) == int(rest[1])


def test_e8m0_closed_form_on_all_bf16(oracle):
    bits, vals = all_bf16_finite()
    pos = vals >= 0
    expo_field = (bits[pos].astype(np.int64) >> 7) & 0xFF
    expect = np.maximum(expo_field - 2, 0)
    got = np.array([oracle.e8m0_from_amax(v) for v in vals[pos]])
    assert np.array_equal(got, expect)


def test_scaling_group_by_power_of_two_shifts_code_only(oracle):
    rng = np.random.default_rng(3)
    K = 128
    X = synth.f32_to_bf16_bits(rng.standard_normal((4, K)).astype(np.float32))
    lut = np.full((K // 32, 1), -1, np.int8)
    base = oracle.quantize_extract(X, lut)
    for k in (-9, 5):
        Xs = synth.f32_to_bf16_bits((synth.bf16_bits_to_f64(X) * 2.0 ** k).astype(np.float32))
        q = oracle.quantize_extract(Xs, lut)
        assert np.array_equal(q["xq"], base["xq"])
        for r in range(4):
            for g in range(K // 32):
                i = oracle.sf_index(r, g, K)
                assert int(q["sf"][i]) == int(base["sf"][i]) + k


def test_quantizer_is_idempotent(oracle):
    rng = np.random.default_rng(5)
    X = synth.f32_to_bf16_bits((rng.standard_normal((8, 256)) * 3).astype(np.float32))
    lut = np.full((8, 1), -1, np.int8)
    q1 = oracle.quantize_extract(X, lut)
    # dequantize with numpy, requantize: codes and scales must reproduce
    deq = dequantize(oracle, q1["xq"], q1["sf"], 256)
    q2 = oracle.quantize_extract(synth.f32_to_bf16_bits(deq.astype(np.float32)), lut)
    assert np.array_equal(q1["sf"], q2["sf"])
    mag1, mag2 = q1["xq"] & 0x77, q2["xq"] & 0x77
    assert np.array_equal(mag1, mag2)


def dequantize(oracle, xq, sf, K):
    M = xq.shape[0]
    vals = np.array([0, .5, 1, 1.5, 2, 3, 4, 6])
    lo, hi = xq & 0xF, xq >> 4
    nib = np.stack([lo, hi], axis=-1).reshape(M, K)
    v = np.where(nib & 8, -1.0, 1.0) * vals[nib & 7]
    out = np.zeros((M, K))
    for r in range(M):
        for g in range(K // 32):
            out[r, g * 32:(g + 1) * 32] = v[r, g * 32:(g + 1) * 32] * 2.0 ** (int(sf[oracle.sf_index(r, g, K)]) - 127)
    return out


# ------------------------------------------------------ worked group (golden)

def test_worked_group_vector(oracle):
    rows = {r[0]: r[1:] for r in _gold_lines("mxfp4_group_vector.txt")}
    x = np.array([float(t) for t in rows["x"]], dtype=np.float32)
    # one group only -> pad K to 128 with zeros so the shape precondition holds
    X = np.zeros((1, 128), np.float32)
    X[0, :32] = x
    Xb = synth.f32_to_bf16_bits(X)
    assert np.array_equal(synth.bf16_bits_to_f64(Xb)[0, :32], x.astype(np.float64))
    for case in "AB":
        lut = np.full((4, 1), -1, np.int8)
        lut[0, 0] = int(rows[f"{case}_lut"][0])
        q = oracle.quantize_extract(Xb, lut)
        assert int(q["sf"][oracle.sf_index(0, 0, 128)]) == int(rows[f"{case}_scale_code"][0])
        expect = bytes(int(b, 16) for b in rows[f"{case}_bytes"])
        assert bytes(q["xq"][0, :16]) == expect
        if case == "A":
            assert q["K_o"] == 1 and q["K_o_pad"] == 64
            assert synth.bf16_bits_to_f64(q["xo"])[0, 0] == float(rows["A_xo"][0])
            assert not q["xo"][0, 1:].any()
        else:
            assert q["K_o"] == 0 and q["xo"].shape == (1, 0)


# ----------------------------------------------- table handling (pins P3)

def test_lut_normalize_and_extraction_bruteforce(oracle):
    rng = np.random.default_rng(11)
    M, K = 5, 256
    X = synth.f32_to_bf16_bits(rng.standard_normal((M, K)).astype(np.float32))
    lut = np.full((K // 32, 3), -1, np.int8)
    lut[0] = [7, 3, -1]
    lut[2] = [-1, 31, 0]
    lut[5] = [9, -1, -1]
    lut[7] = [1, 2, 30]
    q = oracle.quantize_extract(X, lut)
    cols = sorted(32 * k + int(j) for k in range(K // 32) for j in lut[k] if j >= 0)
    assert q["K_o"] == len(cols) == 8
    assert list(q["idx_o"]) == cols
    assert np.array_equal(q["xo"][:, :8], X[:, cols])
    assert q["xo"].shape[1] == 64 and not q["xo"][:, 8:].any()
    assert list(q["prefix"]) == [0, 2, 2, 4, 4, 4, 5, 5]
    assert q["mask"][0] == (1 << 7 | 1 << 3) and q["mask"][2] == (1 << 31 | 1)
    # the zeroed slots quantize to +0 codes
    nib = np.stack([q["xq"] & 0xF, q["xq"] >> 4], -1).reshape(M, K)
    assert not nib[:, cols].any()
    # entry order inside a group is irrelevant
    lut2 = lut.copy()
    lut2[7] = [30, 1, 2]
    lut2[0] = [-1, 3, 7]
    q2 = oracle.quantize_extract(X, lut2)
    for key in ("xq", "sf", "xo"):
        assert np.array_equal(q[key], q2[key])


def test_lut_rejects_bad_entries(oracle):
    X = np.zeros((1, 128), np.uint16)
    bad = np.full((4, 2), -1, np.int8)
    bad[1] = [4, 4]
    with pytest.raises(ValueError):
        oracle.quantize_extract(X, bad)
    bad[1] = [32, -1]
    with pytest.raises(ValueError):
        oracle.quantize_extract(X, bad)
    bad[1] = [-2, -1]
    with pytest.raises(ValueError):
        oracle.quantize_extract(X, bad)


def test_zeroing_only_shrinks_scales(oracle):
    case = synth.tiny_case()
    plain = oracle.quantize_extract(case["X"], np.full((16, 1), -1, np.int8))
    prot = oracle.quantize_extract(case["X"], case["lut"])
    assert (prot["sf"] <= plain["sf"]).all()
    valid = [oracle.sf_index(r, g, 512) for r in range(64) for g in range(16)]
    assert (prot["sf"][valid] < plain["sf"][valid]).mean() > 0.9   # x50 channels dominate nearly every group


# ------------------------------------------------- scale layout (pin P4)

def test_sf_index_hand_values_and_bijection(oracle):
    for kind, *rest in _gold_lines("scale_and_fp8_vectors.txt"):
        if kind == "sf":
            K, r, g, off = map(int, rest)
            assert oracle.sf_index(r, g, K) == off
    K, R = 512, 300
    seen = np.zeros(oracle.sf_bytes(R, K), np.int32)
    assert seen.size == 3 * 4 * 512
    for r in range(384):
        for g in range(K // 32):
            seen[oracle.sf_index(r, g, K)] += 1
    assert (seen == 1).all()
    # rows r, r+32, r+64, r+96 of one 4-group column share 16 contiguous bytes
    b = oracle.sf_index(5, 8, K)
    assert [oracle.sf_index(5 + 32 * q, 8 + j, K) for q in range(4) for j in range(4)] == list(range(b, b + 16))


# ----------------------------------------------------------- E4M3 (pin P7)

def test_e4m3_roundtrip_and_spot_values(oracle):
    for code in range(256):
        if code & 0x7F == 0x7F:
            continue
        assert oracle.e4m3_encode(oracle.e4m3_decode(code)) == code
    assert oracle.e4m3_decode(0x7E) == 448.0 and oracle.e4m3_decode(0x01) == 2.0 ** -9
    for kind, *rest in _gold_lines("scale_and_fp8_vectors.txt"):
        if kind == "e4m3":
            assert oracle.e4m3_encode(float(rest[0])) == int(rest[1], 16), rest


def test_e4m3_matches_library_codec(oracle):
    bits, vals = all_bf16_finite()
    keep = np.abs(vals) <= 448.0
    v = vals[keep][::5]
    lib_codes = v.astype(np.float32).astype(ml_dtypes.float8_e4m3fn).view(np.uint8)
    mine = np.array([oracle.e4m3_encode(x) for x in v], dtype=np.uint8)
    assert np.array_equal(mine, lib_codes)
    # and the decode table against the library's values
    allc = np.arange(256, dtype=np.uint8)
    ok = (allc & 0x7F) != 0x7F
    libv = allc.view(ml_dtypes.float8_e4m3fn).astype(np.float64)
    mine = np.array([oracle.e4m3_decode(int(c)) for c in allc])
    assert np.array_equal(mine[ok], libv[ok])


def test_fp8_per_token_scale_vector(oracle):
    # row amax 3.0: inv = fl32(448/3), sx = fl32(3/448); 3.0 -> 448 -> 0x7E; 1.0 -> 149.33 -> 144 -> 0x71
    X = np.zeros((2, 128), np.float32)
    X[0, 0], X[0, 1], X[0, 2] = 3.0, 1.0, -3.0
    x8, sx = oracle.fp8_quantize(synth.f32_to_bf16_bits(X))
    assert x8[0, 0] == 0x7E and x8[0, 1] == 0x71 and x8[0, 2] == 0xFE
    assert sx[0] == np.float32(3.0) / np.float32(448.0)
    # an all-zero row: amax floors at 2^-40, codes stay zero
    assert sx[1] == np.float32(2.0 ** -40) / np.float32(448.0) and not x8[1].any()


def test_fp8_row_max_hits_448(oracle):
    case = synth.fp8_linear_case(1, 16, 256, 8)
    x8, sx = oracle.fp8_quantize(case["X"])
    assert ((x8 & 0x7F).max(axis=1) == 0x7E).all()
    x = synth.bf16_bits_to_f64(case["X"])
    # decoded * scale reproduces x within half an E4M3 step (2^-4 relative) plus the subnormal step
    dec = np.array([[oracle.e4m3_decode(int(c)) for c in row] for row in x8]) * sx[:, None].astype(np.float64)
    assert (np.abs(dec - x) <= np.abs(x) * 2.0 ** -4 + sx[:, None] * 2.0 ** -10 + 1e-12).all()
