"""Pins for the NVFP4 / G = 16 variant: hand-worked blocks, an independent numpy float32 + ml_dtypes restatement,
the scale layout, reduction to the pinned MXFP4 path on data whose block maxima are 6 * 2^k, the GEMM against a
dense product of the dequantized operands and brute force, and the error ordering with / without the table."""
import os

import ml_dtypes
import numpy as np

from paper_2604_12782_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _gold():
    out = {}
    with open(os.path.join(GOLD, "nvfp4_block_vectors.txt")) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                k, *v = line.split()
                out.setdefault(k, []).append(v)
    return out


def _codes(oracle, sf, M, K):
    return np.array([[sf[oracle.sf16_index(r, b, K)] for b in range(K // 16)] for r in range(M)], np.uint8)


NOLUT = lambda K: np.full((K // 16, 1), -1, np.int8)  # noqa: E731


def test_worked_blocks_and_scale_index(oracle):
    g = _gold()
    X = np.zeros((1, 64), np.float32)
    X[0, 0:16] = [float(v) for v in g["A_x"][0]]
    X[0, 32:48] = [float(v) for v in g["B_x"][0]]
    q = oracle.nvfp4_quantize_extract(synth.f32_to_bf16_bits(X), NOLUT(64), 0)
    codes = _codes(oracle, q["sf"], 1, 64)[0]
    assert codes[0] == int(g["A_scale"][0][0], 16) and codes[2] == int(g["B_scale"][0][0], 16)
    assert codes[1] == 0 and codes[3] == 0
    assert [f"{b:02X}" for b in q["xq"][0, 0:8]] == g["A_bytes"][0]
    assert [f"{b:02X}" for b in q["xq"][0, 16:24]] == g["B_bytes"][0]
    assert not q["xq"][0, 8:16].any() and not q["xq"][0, 24:].any()
    for r, b, K, want in g["sfidx"]:
        assert oracle.sf16_index(int(r), int(b), int(K)) == int(want)
    # bijection onto the buffer
    K, R = 256, 200
    idx = {oracle.sf16_index(r, b, K) for r in range(256) for b in range(K // 16)}
    assert idx == set(range(2 * (K // 64) * 512)) and R <= 256


def test_backed_up_channel_in_the_subnormal_range_is_rounded_not_flushed(oracle):
    """Hand-worked: a flagged channel whose scaled value x * 2^-e falls below the bf16 normal range is stored rounded
    to nearest-even on the subnormal grid."""
    for bits, e, want in _gold()["xo_sub"]:
        X = np.zeros((1, 64), np.uint16)
        X[0, 5] = int(bits, 16)
        lut = NOLUT(64).copy()
        lut[0, 0] = 5
        q = oracle.nvfp4_quantize_extract(X, lut, int(e))
        assert q["xo"][0, 0] == int(want, 16), (bits, e, want, hex(int(q["xo"][0, 0])))
        assert not q["xo"][0, 1:].any() and not q["xq"].any()      # the slot is zeroed, nothing else in the row


def _numpy_nvfp4(Xb, lut16, e):
    """Independent restatement: numpy float32 arithmetic + ml_dtypes codecs."""
    x = synth.bf16_bits_to_f64(Xb)
    M, K = x.shape
    xs = (x * 2.0 ** -e).astype(np.float32)                      # exact for the magnitudes used here
    flagged = np.zeros(K, bool)
    for g, row in enumerate(lut16):
        for j in row:
            if j >= 0:
                flagged[16 * g + int(j)] = True
    xo = xs[:, flagged]
    xr = xs.copy()
    xr[:, flagged] = 0.0
    blk = xr.reshape(M, K // 16, 16)
    amax = np.abs(blk).max(axis=2)
    t = (amax * np.float32(np.float32(1.0) / np.float32(6.0))).astype(np.float32)
    sb = np.minimum(t, np.float32(448.0)).astype(ml_dtypes.float8_e4m3fn)
    sbv = sb.astype(np.float32)
    with np.errstate(divide="ignore"):
        inv = np.where(sbv > 0, np.float32(1.0) / sbv, np.float32(0.0)).astype(np.float32)
    v = (blk * inv[:, :, None]).astype(np.float32)
    nib = np.clip(v, -6.0, 6.0).astype(ml_dtypes.float4_e2m1fn).view(np.uint8).reshape(M, K) & 0xF
    return (nib[:, 0::2] | (nib[:, 1::2] << 4)).astype(np.uint8), sb.view(np.uint8), xo


def test_quantizer_matches_numpy_float32_restatement(oracle):
    rng = np.random.default_rng(31)
    c = synth.osc16_linear_case(1, 37, 256, 8)
    Xb = c["X"].copy()
    X = synth.bf16_bits_to_f64(Xb).astype(np.float32)
    X[2, 16:32] = 0.0
    X[3, ::3] *= -1.0
    X[4] *= 0.01
    Xb = synth.f32_to_bf16_bits(X)
    lut = np.stack([rng.permutation(16)[:2] for _ in range(16)]).astype(np.int8)
    lut[5] = -1
    for e in (synth.nvfp4_tensor_exponent(Xb), 0, 2):
        q = oracle.nvfp4_quantize_extract(Xb, lut, e)
        xq, sb, xo = _numpy_nvfp4(Xb, lut, e)
        assert np.array_equal(_codes(oracle, q["sf"], 37, 256), sb), e
        assert np.array_equal(q["xq"], xq), e
        assert q["K_o"] == 30 and q["K_o_pad"] == 64
        assert np.array_equal(synth.bf16_bits_to_f64(q["xo"][:, :30]), xo.astype(np.float64))
        assert not q["xo"][:, 30:].any()


def test_reduces_to_mxfp4_when_block_maxima_are_six_times_a_power_of_two(oracle):
    """If both 16-halves of every 32-group have maximum 6 * 2^k, the MXFP4 scale 2^k and the NVFP4 scale
    fl32(6 * 2^k / 6) = 2^k coincide, so the element codes must be those of the pinned MXFP4 quantizer."""
    rng = np.random.default_rng(32)
    M, K = 20, 128
    X = rng.uniform(-1, 1, size=(M, K)).astype(np.float32)
    k = rng.integers(-3, 4, size=(M, K // 32))
    for m in range(M):
        for g in range(K // 32):
            X[m, 32 * g:32 * g + 32] *= 5.9 * 2.0 ** k[m, g]
            X[m, 32 * g + 3] = 6.0 * 2.0 ** k[m, g]
            X[m, 32 * g + 20] = -6.0 * 2.0 ** k[m, g]
    Xb = synth.f32_to_bf16_bits(X)
    nv = oracle.nvfp4_quantize_extract(Xb, NOLUT(K), 0)
    mx = oracle.quantize_extract(Xb, np.full((K // 32, 1), -1, np.int8))
    assert np.array_equal(nv["xq"], mx["xq"])
    codes = _codes(oracle, nv["sf"], M, K).astype(np.uint8).view(ml_dtypes.float8_e4m3fn).astype(np.float64)
    assert np.array_equal(codes[:, 0::2], 2.0 ** k) and np.array_equal(codes[:, 1::2], 2.0 ** k)


def _dequant(oracle, q, M, K):
    e2m1 = np.array([0, .5, 1, 1.5, 2, 3, 4, 6, -0., -.5, -1, -1.5, -2, -3, -4, -6])
    nib = np.stack([q["xq"] & 15, q["xq"] >> 4], axis=2).reshape(M, K)
    sc = _codes(oracle, q["sf"], M, K).view(ml_dtypes.float8_e4m3fn).astype(np.float64)
    return (e2m1[nib].reshape(M, K // 16, 16) * sc[:, :, None]).reshape(M, K)


def test_gemm_equals_dense_product_and_bruteforce(oracle):
    c = synth.osc16_linear_case(2, 19, 128, 10)
    ex, ew = synth.nvfp4_tensor_exponent(c["X"]), synth.nvfp4_tensor_exponent(c["W"])
    Y, T, act, wts = oracle.nvfp4_linear(c["X"], c["W"], c["lut16"], ex, ew)
    ref = (_dequant(oracle, act, 19, 128) @ _dequant(oracle, wts, 10, 128).T
           + synth.bf16_bits_to_f64(act["xo"]) @ synth.bf16_bits_to_f64(wts["xo"]).T) * 2.0 ** (ex + ew)
    assert np.allclose(Y, ref, rtol=1e-12, atol=1e-12 * np.abs(ref).max())
    # brute force for one output
    m, n = 7, 3
    acc = 0.0
    for b in range(8):
        sa = float(np.uint8(act["sf"][oracle.sf16_index(m, b, 128)]).view(ml_dtypes.float8_e4m3fn))
        sw = float(np.uint8(wts["sf"][oracle.sf16_index(n, b, 128)]).view(ml_dtypes.float8_e4m3fn))
        p = 0.0
        for ch in range(16 * b, 16 * b + 16):
            xa, wa = int(act["xq"][m, ch // 2]), int(wts["xq"][n, ch // 2])
            p += oracle.e2m1_decode((xa >> 4) if ch & 1 else (xa & 15)) * oracle.e2m1_decode((wa >> 4) if ch & 1 else (wa & 15))
        acc += sa * sw * p
    xo_m, wo_n = synth.bf16_bits_to_f64(act["xo"][m]), synth.bf16_bits_to_f64(wts["xo"][n])
    for t in range(act["xo"].shape[1]):
        acc += float(xo_m[t]) * float(wo_n[t])
    assert Y[m, n] == acc * 2.0 ** (ex + ew)
    # sampled rows
    Y2, _ = oracle.nvfp4_gemm(act, wts, np.array([18, 0], np.int32))
    assert np.array_equal(Y2, Y[[18, 0]])


def test_error_ordering_and_restoration(oracle):
    c = synth.osc16_linear_case(3, 64, 512, 48)
    ex, ew = synth.nvfp4_tensor_exponent(c["X"]), synth.nvfp4_tensor_exponent(c["W"])
    x, w = synth.bf16_bits_to_f64(c["X"]), synth.bf16_bits_to_f64(c["W"])
    exact = x @ w.T

    def err(Y):
        return np.linalg.norm(Y - exact) / np.linalg.norm(exact)
    e_osc = err(oracle.nvfp4_linear(c["X"], c["W"], c["lut16"], ex, ew)[0])
    e_plain = err(oracle.nvfp4_linear(c["X"], c["W"], NOLUT(512), ex, ew)[0])
    assert e_osc < 0.5 * e_plain and e_osc < 0.05
