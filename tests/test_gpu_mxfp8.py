"""GPU parity of the MXFP8 form of the fallback (Section 3.4) against the oracle: element bytes and scale
bytes bit for bit (in full, padding rows included as zeros), GEMM outputs within the stated tolerance."""
import numpy as np
import pytest
import torch

from paper_2604_12782_b200 import synth

pytestmark = pytest.mark.gpu

from gpu_util import assert_within_tolerance, dev_bf16, host_f64, host_u8, poison, valid_sf_bytes  # noqa: E402


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_12782_b200 import binding
    return binding


def check_scales(oracle, got, want, rows, K):
    v = valid_sf_bytes(oracle, rows, K)
    assert np.array_equal(got[v], want[v])
    pad = np.ones(got.size, bool)
    pad[v] = False
    assert not got[pad].any(), "scale bytes of padding rows must be zero"


@pytest.mark.parametrize("M,K,N", [(1, 128, 64), (127, 384, 192), (129, 256, 320), (300, 640, 448), (515, 128, 64)])
def test_mxfp8_linear_small(B, oracle, M, K, N):
    c = synth.fp8_linear_case(M + K + N, M, K, N)
    w = B.osc_mxfp8_prepare_weights(dev_bf16(c["W"]))
    sz = B.osc_mxfp8_act_sizes(w, M)
    ws = poison(sz.workspace_bytes)
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_mxfp8_linear(w, dev_bf16(c["X"]), Y, ws)
    B.osc_sync_check()
    x8, sfa = oracle.mxfp8_quantize(c["X"])
    w8, sfw = oracle.mxfp8_quantize(c["W"])
    ws_h = host_u8(ws)
    assert np.array_equal(ws_h[sz.x8_offset:sz.x8_offset + M * K].reshape(M, K), x8)
    check_scales(oracle, ws_h[sz.sfa_offset:sz.sfa_offset + sz.sfa_bytes], sfa, M, K)
    assert np.array_equal(host_u8(w.keep["w8"])[:N * K].reshape(N, K), w8)
    check_scales(oracle, host_u8(w.keep["sfw"])[:w.sizes.sfw_bytes], sfw, N, K)
    Yref, T = oracle.mxfp8_gemm(x8, sfa, w8, sfw)
    assert_within_tolerance(host_f64(Y), Yref, T, f"mxfp8 M={M} K={K} N={N}")
    # GEMM-only entry point on the same operands, into a padded output
    Y2 = torch.full((M, N + 8), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_mxfp8_gemm(w, ws[sz.x8_offset:], ws[sz.sfa_offset:], M, Y2)
    B.osc_sync_check()
    assert torch.equal(Y2[:, :N], Y) and torch.isnan(Y2[:, N:].float()).all()


@pytest.mark.parametrize("N", [64, 9600, 19200, 28672])
def test_mxfp8_128_row_tiles_all_widths(B, oracle, N):
    """Up to 128 rows the dense MXFP8 GEMM runs on the 128-row-tile kernel; with one row tile its cost model takes
    64-, 128-, 192- and 256-column tiles for these four N (the narrowest width whose tiles still fit in one wave)."""
    M, K = 100, 256
    c = synth.fp8_linear_case(N, M, K, N)
    w = B.osc_mxfp8_prepare_weights(dev_bf16(c["W"]))
    ws = poison(B.osc_mxfp8_act_sizes(w, M).workspace_bytes)
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_mxfp8_linear(w, dev_bf16(c["X"]), Y, ws)
    B.osc_sync_check()
    Yref, T, *_ = oracle.mxfp8_linear(c["X"], c["W"])
    assert_within_tolerance(host_f64(Y), Yref, T, f"mxfp8 128-row tiles N={N}")


def test_mxfp8_quantizer_edge_values(B, oracle):
    """Ties, saturation, signed zeros, subnormal results, tiny and huge groups, all-zero groups, strided input."""
    rng = np.random.default_rng(11)
    M, K = 70, 256
    X = rng.standard_t(3, size=(M, K)).astype(np.float32)
    X[3] *= 1e-20
    X[4] *= 1e20
    X[5, 32:64] = 0.0
    X[6, ::2] *= -1.0
    X[7, :12] = [1.0, 0.5, -1.0625, 1.1875, 1.9375, 2.0 ** -9, -0.0, 1.5, 2.0 ** -18, 3 * 2.0 ** -19, 0.75, 0.1]
    X[7, 12:32] = 0.0
    X[8] = 2.0 ** -130                      # below the smallest scale: code 0
    Xb = synth.f32_to_bf16_bits(X)
    big = torch.zeros((M, K + 64), dtype=torch.bfloat16, device="cuda")
    big[:, :K] = dev_bf16(Xb)
    x8 = poison(M * K)
    sf = poison(1 * (K // 128) * 512)
    B.osc_mxfp8_quantize(big[:, :K], x8, sf)
    B.osc_sync_check()
    r8, rsf = oracle.mxfp8_quantize(Xb)
    assert np.array_equal(host_u8(x8)[:M * K].reshape(M, K), r8)
    check_scales(oracle, host_u8(sf)[:rsf.size], rsf, M, K)


def test_mxfp8_rejects_bad_arguments(B):
    W = torch.zeros((64, 128), dtype=torch.bfloat16, device="cuda")
    w = B.osc_mxfp8_prepare_weights(W)
    with pytest.raises(B.OscError) as e:
        B.osc_mxfp8_prepare_weights(torch.zeros((60, 128), dtype=torch.bfloat16, device="cuda"))
    assert e.value.status == -2
    X = torch.zeros((4, 128), dtype=torch.bfloat16, device="cuda")
    Y = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.OscError) as e:
        B.osc_mxfp8_linear(w, X, Y, torch.zeros(16, dtype=torch.uint8, device="cuda"))
    assert e.value.status == -5
    B.osc_mxfp8_linear(w, X[:0], Y[:0], torch.zeros(16, dtype=torch.uint8, device="cuda"))   # M == 0: no-op
    B.osc_sync_check()


def test_mxfp8_down_projection_full_size(B, oracle):
    M, K, N = 2048, 12288, 4096
    c = synth.fp8_linear_case(0, M, K, N)
    w = B.osc_mxfp8_prepare_weights(dev_bf16(c["W"]))
    sz = B.osc_mxfp8_act_sizes(w, M)
    ws = poison(sz.workspace_bytes)
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_mxfp8_linear(w, dev_bf16(c["X"]), Y, ws)
    B.osc_sync_check()
    x8, sfa = oracle.mxfp8_quantize(c["X"])
    w8, sfw = oracle.mxfp8_quantize(c["W"])
    ws_h = host_u8(ws)
    assert np.array_equal(ws_h[sz.x8_offset:sz.x8_offset + M * K].reshape(M, K), x8)
    assert np.array_equal(ws_h[sz.sfa_offset:sz.sfa_offset + sz.sfa_bytes], sfa)
    assert np.array_equal(host_u8(w.keep["w8"])[:N * K].reshape(N, K), w8)
    assert np.array_equal(host_u8(w.keep["sfw"])[:w.sizes.sfw_bytes], sfw)
    rows = np.array(sorted({0, 1, 127, 128, 255, 256, 257, 1023, 1024, M - 257, M - 256, M - 129, M - 1}
                           | set(int(r) for r in np.random.default_rng(0).integers(0, M, size=24))), np.int32)
    Yref, T = oracle.mxfp8_gemm(x8, sfa, w8, sfw, rows)
    assert_within_tolerance(host_f64(Y[torch.from_numpy(rows.astype(np.int64)).cuda()]), Yref, T, "mxfp8 down")
    assert not torch.isnan(Y.float()).any()


def _grouped_check(B, oracle, counts, K, N, seed, sample=None):
    E = counts.size
    c = synth.moe_down_case(E, counts, K=K, N=N, seed=seed, weight_pool=min(E, 4))
    M = c["M"]
    off_h = synth.offsets_from_counts(counts)
    w = B.osc_mxfp8_prepare_weights_grouped(dev_bf16(c["W"].reshape(E * N, K)).view(E, N, K))
    sz = B.osc_mxfp8_act_sizes(w, M)
    ws = poison(sz.workspace_bytes)
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_mxfp8_linear_grouped(w, dev_bf16(c["X"]), torch.from_numpy(off_h).cuda(), Y, ws)
    B.osc_sync_check()
    x8, sf, parts = oracle.mxfp8_quantize_grouped(c["X"], off_h)
    h = host_u8(ws)
    assert np.array_equal(h[sz.x8_offset:sz.x8_offset + M * K].reshape(M, K), x8)
    # activation scales, expert by expert (valid rows; padding rows of a block must be zero)
    base = 0
    sf_h = h[sz.sfa_offset:sz.sfa_offset + sz.sfa_bytes]
    for e in range(E):
        m = int(counts[e])
        nb = (m + 127) // 128 * (K // 128) * 512
        if m:
            check_scales(oracle, sf_h[base:base + nb], parts[e][1], m, K)
        base += nb
    Yh = host_f64(Y)
    wq = {}
    experts = range(E) if sample is None else sample
    for e in experts:
        r0, r1 = int(off_h[e]), int(off_h[e + 1])
        if r1 == r0:
            continue
        key = e % min(E, 4)
        if key not in wq:
            wq[key] = oracle.mxfp8_quantize(c["W"][e])
        rows = np.arange(r1 - r0, dtype=np.int32) if sample is None else \
            np.unique(np.array([0, r1 - r0 - 1, min(127, r1 - r0 - 1), min(128, r1 - r0 - 1), (r1 - r0) // 2], np.int32))
        Yref, T = oracle.mxfp8_gemm(parts[e][0], parts[e][1], wq[key][0], wq[key][1], rows)
        assert_within_tolerance(Yh[r0 + rows], Yref, T, f"grouped mxfp8 expert {e}")
    assert not torch.isnan(Y.float()).any()


# experts averaging under 96 rows run on 128-row tiles, larger ones on 256-row pair tiles
@pytest.mark.parametrize("counts", [np.array([3, 0, 130, 1, 257, 128]), np.array([300, 0, 5, 256, 129, 511, 1, 385]),
                                    np.array([1, 64, 0, 0, 127, 5, 90, 33, 128, 2])])
def test_mxfp8_grouped_small(B, oracle, counts):
    _grouped_check(B, oracle, counts, 384, 320, 7)


def test_mxfp8_grouped_moe_down_full_size(B, oracle):
    counts = synth.zipf_expert_rows()
    E = counts.size
    big = np.argsort(-counts)
    _grouped_check(B, oracle, counts, 768, 2048, 0, sample=[int(big[0]), int(big[-1]), 0, E - 1, E // 2])
