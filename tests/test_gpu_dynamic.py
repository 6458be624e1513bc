"""GPU parity of the dynamic-protection control group (Section 4.2) against the oracle: codes, scales, index
list, extracted values and the dense high-precision operand bit for bit; outputs within the stated tolerance."""
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


def run(B, oracle, Xb, Wb, what):
    M, K = Xb.shape
    N = Wb.shape[0]
    w = B.osc_dyn_prepare_weights(dev_bf16(Wb))
    sz = B.osc_dyn_act_sizes(w, M)
    ws = poison(sz.workspace_bytes)
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_dyn_linear(w, dev_bf16(Xb), Y, ws)
    B.osc_sync_check()
    ref = oracle.dyn_quantize_extract(Xb)
    h = host_u8(ws)
    assert np.array_equal(h[sz.xq_offset:sz.xq_offset + sz.xq_bytes].reshape(M, K // 2), ref["xq"])
    v = valid_sf_bytes(oracle, M, K)
    assert np.array_equal(h[sz.sfa_offset:sz.sfa_offset + sz.sfa_bytes][v], ref["sf"][v])
    assert np.array_equal(h[sz.idx_offset:sz.idx_offset + sz.idx_bytes].reshape(M, K // 32), ref["idx"])
    assert np.array_equal(h[sz.val_offset:sz.val_offset + sz.val_bytes].view(np.uint16).reshape(M, K // 32), ref["val"])
    assert np.array_equal(h[sz.xo_offset:sz.xo_offset + sz.xo_bytes].view(np.uint16).reshape(M, K), ref["xo"])
    wts = oracle.dyn_prepare_weights(Wb)
    assert np.array_equal(host_u8(w.keep["wq"])[:N * K // 2].reshape(N, K // 2), wts["xq"])
    assert np.array_equal(host_u8(w.keep["wo"])[:N * K * 2].view(np.uint16).reshape(N, K), Wb)
    return w, Y, ref, wts


@pytest.mark.parametrize("M,K,N", [(1, 128, 64), (20, 384, 192), (129, 256, 320), (300, 1024, 448)])
def test_dynamic_linear_small(B, oracle, M, K, N):
    c = synth.osc_linear_case(M + K, M, K, N, 1)
    Xb = c["X"].copy()
    if M > 5:
        X = synth.bf16_bits_to_f64(Xb).astype(np.float32)
        X[3, 32:64] = 0.0       # all-zero group
        X[4, 64:96] = 2.0       # all equal
        X[5, 100], X[5, 101] = -7.0, 7.0
        Xb = synth.f32_to_bf16_bits(X)
    w, Y, ref, wts = run(B, oracle, Xb, c["W"], f"dyn {M}x{K}x{N}")
    Yref, T = oracle.gemm_dual(ref, wts)
    assert_within_tolerance(host_f64(Y), Yref, T, f"dyn linear M={M} K={K} N={N}")
    # a handle of the dynamic baseline is refused by the static entry points and vice versa
    with pytest.raises(B.OscError):
        B.osc_linear(w, dev_bf16(Xb), Y, poison(1 << 20))


def test_dynamic_linear_qkv_shape(B, oracle):
    M, K, N = 1024, 4096, 6144
    c = synth.osc_linear_case(0, M, K, N, 2)
    w, Y, ref, wts = run(B, oracle, c["X"], c["W"], "dyn qkv")
    rows = np.array(sorted({0, 1, 127, 128, 255, 256, 257, M - 257, M - 1}
                           | set(int(r) for r in np.random.default_rng(0).integers(0, M, size=12))), np.int32)
    Yref, T = oracle.gemm_dual(ref, wts, rows)
    assert_within_tolerance(host_f64(Y[torch.from_numpy(rows.astype(np.int64)).cuda()]), Yref, T, "dyn qkv")
    assert not torch.isnan(Y.float()).any()
