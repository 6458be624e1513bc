"""Pins for the oracle's dual-path GEMM (Eq. 5) and FP8 fallback GEMM.

Independent references used here: exact rational arithmetic (fractions) on tiny
shapes, numpy's double-precision matmul, and ml_dtypes as an independent MXFP4
codec.  None of them re-uses oracle code.
"""
import os
from fractions import Fraction

import ml_dtypes
import numpy as np

from paper_2604_12782_b200 import roofline, synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")
E2M1 = [Fraction(0), Fraction(1, 2), Fraction(1), Fraction(3, 2), Fraction(2), Fraction(3), Fraction(4), Fraction(6)]


def frac_pow2(e):
    return Fraction(2) ** e


def nibble(buf, r, c, K):
    b = int(buf[r, c // 2])
    return (b >> 4) if (c & 1) else (b & 15)


def frac_e2m1(n):
    return -E2M1[n & 7] if n & 8 else E2M1[n & 7]


def frac_bf16(bits):
    return Fraction(float(synth.bf16_bits_to_f64(np.array([bits], np.uint16))[0]))


def brute_dual(oracle, act, wts, m, n, K):
    """Eq. 5 for one output element in exact rational arithmetic."""
    acc = Fraction(0)
    for g in range(K // 32):
        sa = int(act["sf"][oracle.sf_index(m, g, K)])
        sw = int(wts["sf"][oracle.sf_index(n, g, K)])
        part = sum(frac_e2m1(nibble(act["xq"], m, c, K)) * frac_e2m1(nibble(wts["xq"], n, c, K))
                   for c in range(32 * g, 32 * g + 32))
        acc += frac_pow2(sa - 127) * frac_pow2(sw - 127) * part
    for t in range(act["xo"].shape[1]):
        acc += frac_bf16(act["xo"][m, t]) * frac_bf16(wts["xo"][n, t])
    return acc


def test_bruteforce_tiny_shapes(oracle):
    rng = np.random.default_rng(21)
    M, N, K = 3, 4, 128          # M != N catches a transposed operand
    X = rng.standard_normal((M, K)) * np.exp(rng.standard_normal((M, 1)) * 3)
    W = rng.standard_normal((N, K)) * 0.05
    X[:, 5] *= 40
    X[:, 70] *= -25
    lut = np.array([[5], [-1], [6], [-1]], np.int8)
    Y, T, act, wts = oracle.linear(synth.f32_to_bf16_bits(X.astype(np.float32)),
                                   synth.f32_to_bf16_bits(W.astype(np.float32)), lut)
    assert Y.shape == (M, N)
    for m in range(M):
        for n in range(N):
            exact = brute_dual(oracle, act, wts, m, n, K)
            assert abs(Fraction(float(Y[m, n])) - exact) <= abs(exact) * Fraction(1, 2 ** 45) + Fraction(1, 2 ** 200)
            assert T[m, n] >= abs(Y[m, n]) * (1 - 1e-12)


def independent_mxfp4_dequant(Xf64):
    """MXFP4 quantize-dequantize with ml_dtypes' E2M1 cast; scale = 2^(floor(log2 amax)-2)."""
    M, K = Xf64.shape
    g = Xf64.reshape(M, K // 32, 32)
    amax = np.abs(g).max(-1)
    _, ex = np.frexp(amax)
    scale = np.where(amax > 0, 2.0 ** np.maximum(ex - 1 - 2, -127), 2.0 ** -127)
    q = (g / scale[..., None]).astype(np.float32).astype(ml_dtypes.float4_e2m1fn).astype(np.float64)
    return (q * scale[..., None]).reshape(M, K)


def test_empty_table_is_plain_w4a4(oracle):
    case = synth.tiny_case(seed=4, M=24, K=256, N=40)
    empty = np.full((8, 1), -1, np.int8)
    Y, T, act, wts = oracle.linear(case["X"], case["W"], empty)
    assert act["K_o"] == 0 and act["xo"].shape[1] == 0
    dX = independent_mxfp4_dequant(synth.bf16_bits_to_f64(case["X"]))
    dW = independent_mxfp4_dequant(synth.bf16_bits_to_f64(case["W"]))
    ref = dX @ dW.T
    assert np.allclose(Y, ref, rtol=0, atol=1e-12 * np.abs(T).max())


def test_full_table_is_a_bf16_gemm(oracle):
    case = synth.tiny_case(seed=6, M=16, K=128, N=24)
    full = np.tile(np.arange(32, dtype=np.int8), (4, 1))
    Y, T, act, wts = oracle.linear(case["X"], case["W"], full)
    assert act["K_o"] == 128
    assert not act["xq"].any() and not wts["xq"].any()           # Path A operands are all +0
    ref = synth.bf16_bits_to_f64(case["X"]) @ synth.bf16_bits_to_f64(case["W"]).T
    assert np.allclose(Y, ref, rtol=0, atol=1e-13 * np.abs(T).max())
    assert np.array_equal(act["xo"], case["X"]) and np.array_equal(wts["xo"], case["W"])


def scatter_back(oracle, q, K):
    """X-hat = deq(Q(X_r)) + scatter(X_o): one dense matrix equivalent to the two paths."""
    M = q["xq"].shape[0]
    vals = np.array([0, .5, 1, 1.5, 2, 3, 4, 6])
    nib = np.stack([q["xq"] & 0xF, q["xq"] >> 4], -1).reshape(M, K)
    v = np.where(nib & 8, -1.0, 1.0) * vals[nib & 7]
    sf = np.array([[int(q["sf"][oracle.sf_index(r, g, K)]) for g in range(K // 32)] for r in range(M)])
    v = (v.reshape(M, K // 32, 32) * 2.0 ** (sf[..., None] - 127.0)).reshape(M, K)
    v[:, q["idx_o"]] += synth.bf16_bits_to_f64(q["xo"][:, :q["K_o"]])
    return v


def test_restoration_identity(oracle):
    case = synth.tiny_case()
    Y, T, act, wts = oracle.linear(case["X"], case["W"], case["lut"])
    Xh, Wh = scatter_back(oracle, act, 512), scatter_back(oracle, wts, 512)
    assert np.allclose(Y, Xh @ Wh.T, rtol=0, atol=1e-12 * T.max())
    # the protected columns of X-hat are the original values exactly
    assert np.array_equal(Xh[:, act["idx_o"]], synth.bf16_bits_to_f64(case["X"])[:, act["idx_o"]])


def rel_fro(Y, ref):
    return np.linalg.norm(Y - ref) / np.linalg.norm(ref)


def test_osc_error_below_unprotected_mxfp4(oracle):
    case = synth.tiny_case()
    ref = synth.bf16_bits_to_f64(case["X"]) @ synth.bf16_bits_to_f64(case["W"]).T
    Y_osc, *_ = oracle.linear(case["X"], case["W"], case["lut"])
    Y_plain, *_ = oracle.linear(case["X"], case["W"], np.full((16, 1), -1, np.int8))
    e_osc, e_plain = rel_fro(Y_osc, ref), rel_fro(Y_plain, ref)
    assert e_osc < 0.3 * e_plain
    assert 0.01 < e_osc < 0.03 and 0.12 < e_plain < 0.3


def test_false_positive_table_entries_are_harmless(oracle):
    case = synth.tiny_case(seed=9, M=16, K=256, N=32)
    lut = np.concatenate([case["lut"], (case["lut"] + 5) % 32], axis=1).astype(np.int8)  # one extra ordinary channel
    ref = synth.bf16_bits_to_f64(case["X"]) @ synth.bf16_bits_to_f64(case["W"]).T
    Y1, *_ = oracle.linear(case["X"], case["W"], case["lut"])
    Y2, *_ = oracle.linear(case["X"], case["W"], lut)
    assert rel_fro(Y2, ref) <= rel_fro(Y1, ref) * 1.05


def test_row_subset_matches_full(oracle):
    case = synth.tiny_case(seed=2, M=40, K=128, N=16)
    Y, T, act, wts = oracle.linear(case["X"], case["W"], case["lut"])
    rows = np.array([39, 0, 17], np.int32)
    Ys, Ts = oracle.gemm_dual(act, wts, rows)
    assert np.array_equal(Ys, Y[rows]) and np.array_equal(Ts, T[rows])


def test_grouped_quantizer_places_experts_on_128_row_blocks(oracle):
    rng = np.random.default_rng(8)
    counts = np.array([3, 0, 130, 1])
    off = synth.offsets_from_counts(counts)
    K = 128
    X = synth.f32_to_bf16_bits(rng.standard_normal((int(counts.sum()), K)).astype(np.float32))
    lut = np.array([[1], [-1], [4], [9]], np.int8)
    gq = oracle.quantize_extract_grouped(X, off, lut)
    assert list(gq["sf_row_base"]) == [0, 128, 128, 384] and gq["sf_rows"] == 512
    for e in range(4):
        r0, r1 = off[e], off[e + 1]
        solo = oracle.quantize_extract(X[r0:r1], lut)
        assert np.array_equal(gq["xq"][r0:r1], solo["xq"]) and np.array_equal(gq["xo"][r0:r1], solo["xo"])
        for r in range(r1 - r0):
            for g in range(K // 32):
                assert gq["sf"][oracle.sf_index(gq["sf_row_base"][e] + r, g, K)] == solo["sf"][oracle.sf_index(r, g, K)]


# --------------------------------------------------------------- FP8 fallback

def test_fp8_gemm_bruteforce(oracle):
    case = synth.fp8_linear_case(3, 3, 128, 5)
    Y, T, (x8, sx), (w8, sw) = oracle.fp8_linear(case["X"], case["W"])
    libv = np.arange(256, dtype=np.uint8).view(ml_dtypes.float8_e4m3fn).astype(np.float64)
    for m in range(3):
        for n in range(5):
            acc = sum(Fraction(float(libv[x8[m, k]])) * Fraction(float(libv[w8[n, k]])) for k in range(128))
            exact = Fraction(float(sx[m])) * Fraction(float(sw[n])) * acc
            assert abs(Fraction(float(Y[m, n])) - exact) <= abs(exact) * Fraction(1, 2 ** 45)
    ref = synth.bf16_bits_to_f64(case["X"]) @ synth.bf16_bits_to_f64(case["W"]).T
    assert rel_fro(Y, ref) < 0.05          # E4M3 keeps ~2^-4 relative precision per element


# ------------------------------------------------------- Table 3 closed form

def test_table3_compute_bound_column():
    with open(os.path.join(GOLD, "table3_efficiency.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    for name, Gs, printed, nd in rows:
        Gs, printed, nd = int(Gs), float(printed), int(nd)
        if name == "speedup_vs_w8a8":
            assert round(roofline.analytic_speedup_vs_w8a8(Gs), nd) == printed
        elif name == "cycle_saving_pct":
            assert round(100 * roofline.analytic_cycle_saving_vs_w8a8(Gs), nd) == printed
        elif name == "branch_overhead_pct":
            # printed "about 12.6 %"; the closed form gives 12.5 %
            assert abs(100 * roofline.analytic_branch_overhead(Gs) - printed) < 0.2
    # two protected channels per group (the QKV workload) cap the gain at 1.6x
    assert roofline.analytic_speedup_vs_w8a8(32, 2) == 1.6


def test_roofline_model_matches_its_definition():
    pk = roofline.peaks(1645.4, 6539.9)
    # QKV, M=8192: compute bound, (2MNK)/P4 + (2MN K_o)/P16
    t = roofline.osc_roofline_seconds(8192, 6144, 4096, 256, pk)
    assert abs(t - (2 * 8192 * 6144 * 4096 / (4 * 1645.4e12) + 2 * 8192 * 6144 * 256 / 1645.4e12)) < 1e-12
    # M=16: weight streaming binds
    t16 = roofline.osc_roofline_seconds(16, 6144, 4096, 256, pk)
    assert abs(t16 - roofline.osc_bytes(16, 6144, 4096, 256) / 6539.9e9) < 1e-12
