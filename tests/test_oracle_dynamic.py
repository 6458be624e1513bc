"""Pins for the dynamic-protection control group (Section 4.2): brute-force numpy argmax, reduction to the
already pinned static path when the table names every token's run-time maximum, restoration identity through a
dense double product, and the error ordering dynamic <= static <= unprotected on outlier-planted inputs."""
import ml_dtypes
import numpy as np

from paper_2604_12782_b200 import synth


def test_index_and_value_against_numpy_argmax(oracle):
    rng = np.random.default_rng(21)
    X = rng.standard_t(3, size=(40, 256)).astype(np.float32)
    X[3, 32:64] = 0.0                     # all-zero group: lowest channel, value +0
    X[4, 64:96] = 2.0                     # all equal: lowest channel
    X[5, 100] = -7.0
    X[5, 101] = 7.0                       # equal magnitudes, opposite signs: lowest channel (the negative one)
    Xb = synth.f32_to_bf16_bits(X)
    d = oracle.dyn_quantize_extract(Xb)
    a = np.abs(synth.bf16_bits_to_f64(Xb)).reshape(40, 8, 32)
    want = a.argmax(axis=2)               # numpy argmax returns the first maximum
    assert np.array_equal(d["idx"], want)
    assert np.array_equal(d["val"], np.take_along_axis(Xb.reshape(40, 8, 32), want[:, :, None], axis=2)[:, :, 0])
    assert d["idx"][3, 1] == 0 and d["val"][3, 1] == 0
    assert d["idx"][4, 2] == 0 and d["idx"][5, 3] == 100 - 96 and d["val"][5, 3] == synth.f32_to_bf16_bits(np.float32(-7.0))
    # the scattered buffer holds exactly those elements
    nz = d["xo"] != 0
    assert nz.sum() <= 40 * 8 and np.array_equal(d["xo"][nz], Xb[nz])


def test_residual_matches_library_mxfp4_of_the_zeroed_tensor(oracle):
    """What is left after the extraction is plain MXFP4 of the tensor with those elements set to +0: compare
    with a numpy + ml_dtypes quantizer that knows nothing about the oracle."""
    rng = np.random.default_rng(22)
    X = (rng.normal(size=(24, 128)) * np.exp(rng.normal(size=(24, 128)))).astype(np.float32)
    Xb = synth.f32_to_bf16_bits(X)
    d = oracle.dyn_quantize_extract(Xb)
    x = synth.bf16_bits_to_f64(Xb).reshape(24, 4, 32)
    j = np.abs(x).argmax(axis=2)
    xr = x.copy()
    np.put_along_axis(xr, j[:, :, None], 0.0, axis=2)
    amax = np.abs(xr).max(axis=2)
    _, ex = np.frexp(amax)
    code = np.where(amax > 0, np.clip(ex - 1 - 2 + 127, 0, 254), 0)
    v = np.clip(xr * np.exp2(127.0 - code)[:, :, None], -6.0, 6.0).astype(np.float32)
    nib = v.astype(ml_dtypes.float4_e2m1fn).view(np.uint8).reshape(24, 128) & 0xF
    want = (nib[:, 0::2] | (nib[:, 1::2] << 4)).astype(np.uint8)
    assert np.array_equal(d["xq"], want)
    got_codes = np.array([[d["sf"][oracle.sf_index(r, g, 128)] for g in range(4)] for r in range(24)])
    assert np.array_equal(got_codes, code)


def test_reduces_to_static_path_when_the_table_names_every_maximum(oracle):
    """If one channel per group dominates every token, run-time detection and the static table agree, so the
    dynamic quantizer must reproduce the (separately pinned) Algorithm 2 outputs."""
    rng = np.random.default_rng(23)
    M, K = 50, 256
    ch = rng.integers(0, 32, size=K // 32)
    X = rng.normal(size=(M, K)).astype(np.float32)
    for g, c in enumerate(ch):
        X[:, 32 * g + c] = rng.choice([-1.0, 1.0], size=M) * rng.uniform(200, 300, size=M)
    Xb = synth.f32_to_bf16_bits(X)
    lut = ch.astype(np.int8).reshape(-1, 1)
    st = oracle.quantize_extract(Xb, lut)
    dy = oracle.dyn_quantize_extract(Xb)
    assert np.array_equal(dy["idx"], np.tile(ch.astype(np.uint8), (M, 1)))
    assert np.array_equal(dy["xq"], st["xq"]) and np.array_equal(dy["sf"], st["sf"])
    assert np.array_equal(dy["val"], st["xo"][:, :K // 32])


def test_linear_equals_dense_product_of_restored_operands(oracle):
    c = synth.osc_linear_case(5, 20, 256, 24, 1)
    Y, T, act, wts = oracle.dyn_linear(c["X"], c["W"])
    e2m1 = np.array([0, .5, 1, 1.5, 2, 3, 4, 6, -0., -.5, -1, -1.5, -2, -3, -4, -6])

    def deq(q):
        R = q["xq"].shape[0]
        nib = np.stack([q["xq"] & 15, q["xq"] >> 4], axis=2).reshape(R, -1)
        codes = np.array([[q["sf"][oracle.sf_index(r, g, 256)] for g in range(8)] for r in range(R)], np.int64)
        return (e2m1[nib].reshape(R, 8, 32) * np.exp2(codes - 127.0)[:, :, None]).reshape(R, 256)
    xhat = deq(act) + synth.bf16_bits_to_f64(act["xo"])
    # Path A uses the quantized weights, Path B the bf16 weights
    ref = deq(act) @ deq(wts).T + synth.bf16_bits_to_f64(act["xo"]) @ synth.bf16_bits_to_f64(c["W"]).T
    assert np.allclose(Y, ref, rtol=1e-12, atol=1e-12 * np.abs(ref).max())
    assert np.abs(xhat - synth.bf16_bits_to_f64(c["X"])).max() < np.abs(synth.bf16_bits_to_f64(c["X"])).max()


def test_error_ordering_dynamic_static_unprotected(oracle):
    c = synth.osc_linear_case(6, 64, 512, 48, 1)
    x = synth.bf16_bits_to_f64(c["X"])
    w = synth.bf16_bits_to_f64(c["W"])
    exact = x @ w.T

    def err(Y):
        return np.linalg.norm(Y - exact) / np.linalg.norm(exact)
    e_dyn = err(oracle.dyn_linear(c["X"], c["W"])[0])
    e_osc = err(oracle.linear(c["X"], c["W"], c["lut"])[0])
    e_plain = err(oracle.linear(c["X"], c["W"], np.full((16, 1), -1, np.int8))[0])
    assert e_dyn <= e_osc * 1.05 and e_osc < 0.5 * e_plain
