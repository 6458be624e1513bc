"""Property tests (hypothesis) of the oracle on small random shapes: facts the paper states or implies that must
hold for every input, not just the seeded cases - the order of a group's table entries is irrelevant, a -1 entry
leaves its group untouched, rows are independent, power-of-two scaling of a group moves only its scale code, zeroing
before CalculateScale can only shrink a scale, and the two-path sum equals one dense product of restored operands."""
import numpy as np
from hypothesis import given, settings, strategies as st

from paper_2604_12782_b200 import synth

SET = settings(max_examples=25, deadline=None, derandomize=True, database=None)   # the same examples on every run


def case(seed, M, Kg, cpg):
    rng = np.random.default_rng(seed)
    K = 32 * Kg
    X = (rng.standard_normal((M, K)) * np.exp(rng.normal(size=(M, K)))).astype(np.float32)
    lut = np.full((Kg, max(cpg, 1)), -1, np.int8)
    for g in range(Kg):
        n = int(rng.integers(0, cpg + 1))
        lut[g, :n] = rng.permutation(32)[:n]
    return synth.f32_to_bf16_bits(X), lut, rng


@SET
@given(st.integers(0, 2 ** 31), st.integers(1, 9), st.sampled_from([4, 8, 12]), st.integers(0, 4))
def test_entry_order_and_minus_one_entries_do_not_matter(oracle, seed, M, Kg, cpg):
    X, lut, rng = case(seed, M, Kg, cpg)
    a = oracle.quantize_extract(X, lut)
    shuffled = np.stack([rng.permutation(row) for row in lut])
    padded = np.concatenate([shuffled, np.full((Kg, 2), -1, np.int8)], axis=1)
    b = oracle.quantize_extract(X, padded)
    for k in ("xq", "sf", "xo"):
        assert np.array_equal(a[k], b[k])
    # groups without an entry equal the plain MXFP4 of the same data
    plain = oracle.quantize_extract(X, np.full((Kg, 1), -1, np.int8))
    for g in range(Kg):
        if (lut[g] < 0).all():
            assert np.array_equal(a["xq"][:, 16 * g:16 * g + 16], plain["xq"][:, 16 * g:16 * g + 16])


@SET
@given(st.integers(0, 2 ** 31), st.integers(2, 9), st.sampled_from([4, 8]), st.integers(0, 3))
def test_rows_are_independent(oracle, seed, M, Kg, cpg):
    X, lut, rng = case(seed, M, Kg, cpg)
    perm = rng.permutation(M)
    a, b = oracle.quantize_extract(X, lut), oracle.quantize_extract(X[perm], lut)
    assert np.array_equal(a["xq"][perm], b["xq"]) and np.array_equal(a["xo"][perm], b["xo"])
    W = synth.f32_to_bf16_bits((0.05 * rng.standard_normal((5, 32 * Kg))).astype(np.float32))
    wts = oracle.prepare_weights(W, lut)
    Ya, _ = oracle.gemm_dual(a, wts)
    Yb, _ = oracle.gemm_dual(b, wts)
    assert np.array_equal(Ya[perm], Yb)
    sub = np.array([M - 1, 0], np.int32)
    assert np.array_equal(oracle.gemm_dual(a, wts, sub)[0], Ya[sub])


@SET
@given(st.integers(0, 2 ** 31), st.integers(-6, 6))
def test_power_of_two_scaling_moves_only_the_scale_code(oracle, seed, k):
    X, lut, _ = case(seed, 3, 4, 1)
    x = synth.bf16_bits_to_f64(X) * 2.0 ** k
    a, b = oracle.quantize_extract(X, lut), oracle.quantize_extract(synth.f32_to_bf16_bits(x.astype(np.float32)), lut)
    assert np.array_equal(a["xq"], b["xq"])
    for r in range(3):
        for g in range(4):
            ca, cb = int(a["sf"][oracle.sf_index(r, g, 128)]), int(b["sf"][oracle.sf_index(r, g, 128)])
            assert cb == ca + k or ca == 0 or cb == 0      # (codes clamp at 0 for all-zero groups)


@SET
@given(st.integers(0, 2 ** 31), st.sampled_from([4, 8]), st.integers(1, 3))
def test_zeroing_only_shrinks_scales_and_restoration_is_exact(oracle, seed, Kg, cpg):
    X, lut, rng = case(seed, 6, Kg, cpg)
    K = 32 * Kg
    a = oracle.quantize_extract(X, lut)
    plain = oracle.quantize_extract(X, np.full((Kg, 1), -1, np.int8))
    idx = [oracle.sf_index(r, g, K) for r in range(6) for g in range(Kg)]
    assert (a["sf"][idx] <= plain["sf"][idx]).all()
    # dual-path sum == dense product of (dequantized residual + scattered protected channels), Path B on bf16 weights
    W = synth.f32_to_bf16_bits((0.05 * rng.standard_normal((4, K))).astype(np.float32))
    wts = oracle.prepare_weights(W, lut)
    Y, _ = oracle.gemm_dual(a, wts)
    e2m1 = np.array([0, .5, 1, 1.5, 2, 3, 4, 6, -0., -.5, -1, -1.5, -2, -3, -4, -6])

    def restored(q, rows):
        nib = np.stack([q["xq"] & 15, q["xq"] >> 4], axis=2).reshape(rows, K)
        codes = np.array([[q["sf"][oracle.sf_index(r, g, K)] for g in range(Kg)] for r in range(rows)], np.int64)
        d = (e2m1[nib].reshape(rows, Kg, 32) * np.exp2(codes - 127.0)[:, :, None]).reshape(rows, K)
        d[:, a["idx_o"]] += synth.bf16_bits_to_f64(q["xo"][:, :a["K_o"]])
        return d
    ref = restored(a, 6) @ restored(wts, 4).T
    assert np.allclose(Y, ref, rtol=1e-12, atol=1e-12 * max(np.abs(ref).max(), 1e-30))
