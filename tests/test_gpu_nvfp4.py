"""GPU parity of the NVFP4 / G = 16 variant against the oracle: packed codes, E4M3 scale bytes and backed-up
channels bit for bit (activations and weights), outputs within the stated tolerance."""
import numpy as np
import pytest
import torch

from paper_2604_12782_b200 import synth

pytestmark = pytest.mark.gpu

from gpu_util import assert_within_tolerance, dev_bf16, host_f64, host_u8, poison  # noqa: E402


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_12782_b200 import binding
    return binding


def sf16_valid(rows, K):
    r = np.arange(rows)[:, None]
    b = np.arange(K // 16)[None, :]
    return (((r // 128) * (K // 64) + b // 4) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + (b % 4)).ravel()


def check_quantized(q, xq, sf, xo, rows, K):
    assert np.array_equal(xq.reshape(rows, K // 2), q["xq"])
    v = sf16_valid(rows, K)
    assert np.array_equal(sf[:q["sf"].size][v], q["sf"][v])
    if q["K_o_pad"]:
        assert np.array_equal(xo.view(np.uint16).reshape(rows, q["K_o_pad"]), q["xo"])


def run_case(B, oracle, Xb, Wb, lut16, what):
    M, K = Xb.shape
    N = Wb.shape[0]
    ex, ew = synth.nvfp4_tensor_exponent(Xb), synth.nvfp4_tensor_exponent(Wb)
    w = B.osc_nvfp4_prepare_weights(dev_bf16(Wb), lut16, ew)
    sz = B.osc_nvfp4_act_sizes(w, M)
    ws = poison(sz.workspace_bytes)
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_nvfp4_linear(w, dev_bf16(Xb), ex, Y, ws)
    B.osc_sync_check()
    Yref, T, act, wts = oracle.nvfp4_linear(Xb, Wb, lut16, ex, ew)
    h = host_u8(ws)
    check_quantized(act, h[sz.xq_offset:sz.xq_offset + sz.xq_bytes], h[sz.sfa_offset:sz.sfa_offset + sz.sfa_bytes],
                    h[sz.xo_offset:sz.xo_offset + sz.xo_bytes], M, K)
    check_quantized(wts, host_u8(w.keep["wq"])[:w.sizes.wq_bytes], host_u8(w.keep["sfw"])[:w.sizes.sfw_bytes],
                    host_u8(w.keep["wo"])[:w.sizes.wo_bytes], N, K)
    assert_within_tolerance(host_f64(Y), Yref, T, what)
    return w, sz, ws, Y, ex


# The last three rows reach the 128-row-tile kernel with 64-, 128- and 192-column tiles (65-128 rows; the width follows
# from the number of tiles against the number of SMs), the first two the few-row kernel, the rest the pair kernel.
@pytest.mark.parametrize("M,K,N,kind", [(1, 128, 64, "one"), (64, 512, 512, "one"), (127, 384, 192, "two"),
                                        (129, 256, 320, "empty"), (300, 640, 448, "one"), (515, 128, 64, "two"),
                                        (100, 640, 320, "two"), (97, 256, 12288, "one"), (128, 128, 24576, "two")])
def test_nvfp4_linear_small(B, oracle, M, K, N, kind):
    c = synth.osc16_linear_case(M + K, M, K, N)
    rng = np.random.default_rng(N)
    lut16 = {"one": c["lut16"], "empty": np.full((K // 16, 1), -1, np.int8),
             "two": np.stack([rng.permutation(16)[:2] for _ in range(K // 16)]).astype(np.int8)}[kind]
    w, sz, ws, Y, ex = run_case(B, oracle, c["X"], c["W"], lut16, f"nvfp4 {M}x{K}x{N} {kind}")
    Y2 = torch.full((M, N + 8), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_nvfp4_gemm(w, ws[sz.xq_offset:], ws[sz.sfa_offset:], ws[sz.xo_offset:], M, ex, Y2)
    B.osc_sync_check()
    assert torch.equal(Y2[:, :N], Y) and torch.isnan(Y2[:, N:].float()).all()
    with pytest.raises(B.OscError):
        B.osc_linear(w, dev_bf16(c["X"]), Y, ws)      # an NVFP4 handle is refused by the MXFP4 entry points


def test_nvfp4_edge_values(B, oracle):
    rng = np.random.default_rng(41)
    M, K = 40, 256
    X = rng.standard_t(3, size=(M, K)).astype(np.float32)
    X[2, 16:32] = 0.0                      # all-zero block: scale byte 0, sign-only codes
    X[3, ::3] *= -1.0
    X[4] *= 0.001                          # tiny blocks: subnormal E4M3 scales
    X[5, 0:16] = [6.0, -3.0, 1.25, 0.75, 0.25, -0.0, 2.5, 3.5, 5.0] + [0.5] * 7
    Xb = synth.f32_to_bf16_bits(X)
    W = synth.f32_to_bf16_bits((0.02 * rng.standard_normal((64, K))).astype(np.float32))
    run_case(B, oracle, Xb, W, np.full((K // 16, 1), 3, np.int8), "nvfp4 edge")


def test_nvfp4_qkv_shape(B, oracle):
    M, K, N = 1024, 4096, 6144
    c = synth.osc16_linear_case(0, M, K, N)
    ex, ew = synth.nvfp4_tensor_exponent(c["X"]), synth.nvfp4_tensor_exponent(c["W"])
    w = B.osc_nvfp4_prepare_weights(dev_bf16(c["W"]), c["lut16"], ew)
    sz = B.osc_nvfp4_act_sizes(w, M)
    ws = poison(sz.workspace_bytes)
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_nvfp4_linear(w, dev_bf16(c["X"]), ex, Y, ws)
    B.osc_sync_check()
    act = oracle.nvfp4_quantize_extract(c["X"], c["lut16"], ex)
    wts = oracle.nvfp4_quantize_extract(c["W"], c["lut16"], ew)
    h = host_u8(ws)
    check_quantized(act, h[sz.xq_offset:sz.xq_offset + sz.xq_bytes], h[sz.sfa_offset:sz.sfa_offset + sz.sfa_bytes],
                    h[sz.xo_offset:sz.xo_offset + sz.xo_bytes], M, K)
    check_quantized(wts, host_u8(w.keep["wq"])[:w.sizes.wq_bytes], host_u8(w.keep["sfw"])[:w.sizes.sfw_bytes],
                    host_u8(w.keep["wo"])[:w.sizes.wo_bytes], N, K)
    rows = np.array(sorted({0, 1, 127, 128, 255, 256, 257, M - 257, M - 1}
                           | set(int(r) for r in np.random.default_rng(0).integers(0, M, size=12))), np.int32)
    Yref, T = oracle.nvfp4_gemm(act, wts, rows)
    assert_within_tolerance(host_f64(Y[torch.from_numpy(rows.astype(np.int64)).cuda()]), Yref, T, "nvfp4 qkv")
    assert not torch.isnan(Y.float()).any()


@pytest.mark.parametrize("counts", [[3, 0, 130, 1, 257, 128], [300, 0, 5, 256, 129, 511, 1, 385], [700, 64, 0, 900]])
def test_nvfp4_grouped(B, oracle, counts):
    """Grouped (MoE) NVFP4: per expert equal to the dense call on that expert's rows and weights (same kernels, same
    operands, scale rows shifted to the expert's 128-row block), and within tolerance of the oracle; small experts
    take 128-row tiles, large ones the pair kernel; experts that end inside a tile, empty and one-row experts."""
    counts = np.array(counts)
    E, K, N = counts.size, 384, 320
    M = int(counts.sum())
    off_h = synth.offsets_from_counts(counts)
    c = synth.osc16_linear_case(50 + E, M, K, N)
    rng = np.random.default_rng(E)
    Wb = synth.f32_to_bf16_bits((0.02 * rng.standard_normal((E, N, K))).astype(np.float32))
    ex, ew = synth.nvfp4_tensor_exponent(c["X"]), synth.nvfp4_tensor_exponent(Wb)
    w = B.osc_nvfp4_prepare_weights_grouped(dev_bf16(Wb.reshape(E * N, K)).view(E, N, K), c["lut16"], ew)
    sz = B.osc_nvfp4_act_sizes(w, M)
    ws = poison(sz.workspace_bytes)
    big = torch.full((M + 2, N + 8), 7.0, dtype=torch.bfloat16, device="cuda")
    Y = big[1:M + 1, :N]
    B.osc_nvfp4_linear_grouped(w, dev_bf16(c["X"]), torch.from_numpy(off_h).cuda(), ex, Y, ws)
    B.osc_sync_check()
    guard = big.clone()
    guard[1:M + 1, :N] = 7.0
    assert (guard == 7.0).all(), "wrote outside Y"
    Yh = host_f64(Y)
    for e in range(E):
        r0, r1 = int(off_h[e]), int(off_h[e + 1])
        if r1 > r0:
            Yref, T, act, _ = oracle.nvfp4_linear(c["X"][r0:r1], Wb[e], c["lut16"], ex, ew)
            assert_within_tolerance(Yh[r0:r1], Yref, T, f"grouped nvfp4, expert {e} ({r1 - r0} rows)")
            # the quantizer's codes of the expert's rows: bit for bit
            got = host_u8(ws)[sz.xq_offset:sz.xq_offset + sz.xq_bytes].reshape(M, K // 2)[r0:r1]
            assert np.array_equal(got, act["xq"])
    wd = B.osc_nvfp4_prepare_weights(dev_bf16(Wb[0]), c["lut16"], ew)
    with pytest.raises(B.OscError):
        B.osc_nvfp4_linear_grouped(wd, dev_bf16(c["X"]), torch.from_numpy(off_h).cuda(), ex, Y, ws)
    with pytest.raises(B.OscError):
        B.osc_nvfp4_linear(w, dev_bf16(c["X"]), ex, Y, ws)


# ---- the producer fusion and the dispatch gather in the NVFP4 form ---------------------------------------------

@pytest.mark.parametrize("M,K,N,kind", [(1, 128, 64, "one"), (37, 384, 192, "two"), (130, 1024, 320, "one"),
                                        (300, 4096, 256, "one"), (64, 8192, 64, "empty"), (700, 512, 448, "two")])
def test_nvfp4_rmsnorm_fused(B, oracle, M, K, N, kind):
    """RMSNorm + the NVFP4 form of Algorithm 2 in one kernel: codes, E4M3 scale bytes and backed-up channels bit for
    bit what the oracle's RMSNorm followed by its NVFP4 quantizer gives, and byte for byte the library's own two-step
    path; the linear within the tolerance."""
    from producer_inputs import gamma_bits, residual_rows
    rng = np.random.default_rng(M + K)
    Hb, gb = residual_rows(rng, M, K), gamma_bits(rng, K)
    lut16 = {"one": rng.integers(0, 16, size=(K // 16, 1)).astype(np.int8), "empty": np.full((K // 16, 1), -1, np.int8),
             "two": np.stack([rng.permutation(16)[:2] for _ in range(K // 16)]).astype(np.int8)}[kind]
    Wb = synth.f32_to_bf16_bits((0.02 * rng.standard_normal((N, K))).astype(np.float32))
    eps = 1e-6
    Xn = oracle.rmsnorm(Hb, gb, eps)
    ex, ew = synth.nvfp4_tensor_exponent(Xn), synth.nvfp4_tensor_exponent(Wb)
    w = B.osc_nvfp4_prepare_weights(dev_bf16(Wb), lut16, ew)
    sz = B.osc_nvfp4_act_sizes(w, M)
    ws = poison(sz.workspace_bytes)
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_nvfp4_rmsnorm_linear(w, dev_bf16(Hb), dev_bf16(gb), eps, ex, Y, ws)
    B.osc_sync_check()
    Yref, T, act, _ = oracle.nvfp4_linear(Xn, Wb, lut16, ex, ew)
    h = host_u8(ws)
    check_quantized(act, h[sz.xq_offset:sz.xq_offset + sz.xq_bytes], h[sz.sfa_offset:sz.sfa_offset + sz.sfa_bytes],
                    h[sz.xo_offset:sz.xo_offset + sz.xo_bytes], M, K)
    assert_within_tolerance(host_f64(Y), Yref, T, f"nvfp4 rmsnorm linear M={M} K={K}")
    # two-step path of the library: own RMSNorm kernel, then the stand-alone NVFP4 quantizer
    Xd = torch.empty(M, K, dtype=torch.bfloat16, device="cuda")
    B.osc_rmsnorm(dev_bf16(Hb), dev_bf16(gb), eps, Xd)
    ws2 = poison(sz.workspace_bytes)
    B.osc_nvfp4_quantize_extract(w, Xd, ex, ws2[sz.xq_offset:], ws2[sz.sfa_offset:], ws2[sz.xo_offset:])
    ws3 = poison(sz.workspace_bytes)
    B.osc_nvfp4_rmsnorm_quantize_extract(w, dev_bf16(Hb), dev_bf16(gb), eps, ex, ws3[sz.xq_offset:], ws3[sz.sfa_offset:],
                                         ws3[sz.xo_offset:])
    B.osc_sync_check()
    h2, h3 = host_u8(ws2), host_u8(ws3)
    for o, n in ((sz.xq_offset, sz.xq_bytes), (sz.xo_offset, sz.xo_bytes)):
        assert np.array_equal(h2[o:o + n], h3[o:o + n])
    v = sf16_valid(M, K)
    assert np.array_equal(h2[sz.sfa_offset:sz.sfa_offset + sz.sfa_bytes][v], h3[sz.sfa_offset:sz.sfa_offset + sz.sfa_bytes][v])
    B.osc_nvfp4_rmsnorm_linear(w, dev_bf16(Hb)[:0], dev_bf16(gb), eps, ex, Y[:0], ws)     # M == 0: a no-op
    wm = B.osc_prepare_weights(dev_bf16(Wb), np.full((K // 32, 1), -1, np.int8))
    with pytest.raises(B.OscError):                                                        # an MXFP4 handle is refused
        B.osc_nvfp4_rmsnorm_linear(wm, dev_bf16(Hb), dev_bf16(gb), eps, ex, Y, ws)


@pytest.mark.parametrize("counts,with_norm", [([3, 0, 130, 1, 257, 128], False), ([300, 0, 5, 256, 129, 511, 1, 385], True),
                                              ([700, 64, 0, 900], False)])
def test_nvfp4_grouped_gather(B, oracle, counts, with_norm):
    """The dispatch fused behind the NVFP4 quantizer: T tokens quantized once and their quantized rows gathered; bit
    for bit what osc_nvfp4_linear_grouped gives on the permuted matrix X[row_token] (and, behind an RMSNorm, on the
    permuted normalized rows)."""
    from producer_inputs import gamma_bits
    counts = np.array(counts)
    E, K, N = counts.size, 512, 320
    M = int(counts.sum())
    T = max(1, M // 3)
    off_h = synth.offsets_from_counts(counts)
    off = torch.from_numpy(off_h).cuda()
    rng = np.random.default_rng(E + M)
    c = synth.osc16_linear_case(60 + E, T, K, N)
    row_token_h = rng.integers(0, T, size=M).astype(np.int32)
    row_token = torch.from_numpy(row_token_h).cuda()
    Wb = synth.f32_to_bf16_bits((0.02 * rng.standard_normal((E, N, K))).astype(np.float32))
    gb = gamma_bits(rng, K)
    src = oracle.rmsnorm(c["X"], gb, 1e-6) if with_norm else c["X"]
    ex, ew = synth.nvfp4_tensor_exponent(src), synth.nvfp4_tensor_exponent(Wb)
    w = B.osc_nvfp4_prepare_weights_grouped(dev_bf16(Wb.reshape(E * N, K)).view(E, N, K), c["lut16"], ew)
    wsg = poison(B.osc_nvfp4_gather_workspace_bytes(w, T, M))
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    if with_norm:
        B.osc_nvfp4_rmsnorm_linear_grouped_gather(w, dev_bf16(c["X"]), dev_bf16(gb), 1e-6, row_token, off, ex, Y, wsg)
    else:
        B.osc_nvfp4_linear_grouped_gather(w, dev_bf16(c["X"]), row_token, off, ex, Y, wsg)
    B.osc_sync_check()
    # the grouped call on the permuted matrix
    Xp = np.ascontiguousarray(src[row_token_h])
    sz = B.osc_nvfp4_act_sizes(w, M)
    ws = poison(sz.workspace_bytes)
    Y2 = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_nvfp4_linear_grouped(w, dev_bf16(Xp), off, ex, Y2, ws)
    B.osc_sync_check()
    assert torch.equal(Y.view(torch.int16), Y2.view(torch.int16))
    hg, hp = host_u8(wsg), host_u8(ws)
    for o, n in ((sz.xq_offset, sz.xq_bytes), (sz.xo_offset, sz.xo_bytes)):
        assert np.array_equal(hg[o:o + n], hp[o:o + n])
    # and against the oracle, expert by expert
    Yh = host_f64(Y)
    for e in range(E):
        r0, r1 = int(off_h[e]), int(off_h[e + 1])
        if r1 > r0:
            Yref, Tt, *_ = oracle.nvfp4_linear(Xp[r0:r1], Wb[e], c["lut16"], ex, ew)
            assert_within_tolerance(Yh[r0:r1], Yref, Tt, f"gathered grouped nvfp4, expert {e}")
    assert not torch.isnan(Y.float()).any()
