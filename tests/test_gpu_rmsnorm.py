"""GPU parity of the RMSNorm fused in front of Algorithm 2 (Section 3.3: the quantizer sits directly behind the
operator that produces the activations).  The normalized rows, the packed codes, the scale bytes and the gathered
channels are compared bit for bit with the oracle (double arithmetic, one rounding to bf16, then Algorithm 2);
the fused kernel is also compared byte for byte with the library's own two-step path."""
import numpy as np
import pytest
import torch

from paper_2604_12782_b200 import synth

pytestmark = pytest.mark.gpu

from gpu_util import assert_within_tolerance, dev_bf16, host_bf16_bits, host_f64, host_u8, poison, valid_sf_bytes  # noqa: E402
from producer_inputs import RMSNORM_ROW_CASES, gamma_bits, residual_rows  # noqa: E402


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_12782_b200 import binding
    return binding


def rand_lut(rng, K, C, p_none=0.2):
    lut = np.full((K // 32, C), -1, np.int8)
    for k in range(K // 32):
        ch = rng.permutation(32)[:C]
        for c in range(C):
            if rng.random() > p_none:
                lut[k, c] = ch[c]
    return lut


@pytest.mark.parametrize("M,K,eps", RMSNORM_ROW_CASES)
def test_rmsnorm_rows_bit_exact(B, oracle, M, K, eps):
    rng = np.random.default_rng(M + K)
    Hb, gb = residual_rows(rng, M, K), gamma_bits(rng, K)
    ldx = K + 8
    Xbig = torch.full((M, ldx), 7.0, dtype=torch.bfloat16, device="cuda")
    B.osc_rmsnorm(dev_bf16(Hb), dev_bf16(gb), eps, Xbig[:, :K])
    B.osc_sync_check()
    want = oracle.rmsnorm(Hb, gb, eps)
    got = host_bf16_bits(Xbig[:, :K].contiguous())
    assert np.array_equal(got, want), f"{np.count_nonzero(got != want)} of {got.size} elements differ"
    assert (Xbig[:, K:] == 7.0).all()
    # and against the plain all-double definition (one rounding): never more than one bf16 unit away
    from oracle import plain
    assert plain.bf16_units_apart(got, plain.rmsnorm_plain(Hb, gb, eps)).max() <= 1


def test_rmsnorm_special_rows(B, oracle):
    """Constant rows (an exact power-of-two r), one non-zero per row, subnormal inputs, results that overflow bf16."""
    K = 256
    H = np.zeros((6, K), np.float32)
    H[0] = 3.0
    H[1, 17] = -0.375
    H[2] = 1e-39                      # bf16 subnormals
    H[3] = 2.0 ** 100
    H[4] = np.where(np.arange(K) % 2, 1.0, -1.0)
    H[5, 0] = 3e38
    Hb = synth.f32_to_bf16_bits(H)
    g = np.ones(K, np.float32)
    g[:8] = 3e38                      # y = x r gamma overflows for these channels
    g[8:16] = 1e-38
    gb = synth.f32_to_bf16_bits(g)
    for eps in (0.0, 1e-6):
        X = torch.empty(6, K, dtype=torch.bfloat16, device="cuda")
        B.osc_rmsnorm(dev_bf16(Hb), dev_bf16(gb), eps, X)
        B.osc_sync_check()
        assert np.array_equal(host_bf16_bits(X), oracle.rmsnorm(Hb, gb, eps))


@pytest.mark.parametrize("M,K,C", [(1, 128, 1), (129, 384, 2), (300, 1024, 2), (70, 4096, 1), (40, 8192, 3)])
def test_fused_quantize_extract_bit_exact(B, oracle, M, K, C):
    rng = np.random.default_rng(M * 3 + K)
    Hb, gb = residual_rows(rng, M, K), gamma_bits(rng, K)
    lut = rand_lut(rng, K, C)
    W = synth.osc_weights_only(1, K, 64, 1)["W"]
    w = B.osc_prepare_weights(dev_bf16(W), lut)
    sz = B.osc_act_sizes(w, M)
    xq, sfa, xo = poison(sz.xq_bytes), poison(sz.sfa_bytes), poison(sz.xo_bytes)
    B.osc_rmsnorm_quantize_extract(w, dev_bf16(Hb), dev_bf16(gb), 1e-6, xq, sfa, xo)
    B.osc_sync_check()
    ref = oracle.quantize_extract(oracle.rmsnorm(Hb, gb, 1e-6), lut)
    assert np.array_equal(host_u8(xq)[:sz.xq_bytes].reshape(M, K // 2), ref["xq"])
    sf_h = host_u8(sfa)[:sz.sfa_bytes]
    valid = valid_sf_bytes(oracle, M, K)
    assert np.array_equal(sf_h[valid], ref["sf"][valid])
    pad = np.ones(sf_h.size, bool)
    pad[valid] = False
    assert not sf_h[pad].any(), "scale bytes of rows beyond M must be 0"
    if ref["K_o_pad"]:
        assert np.array_equal(host_u8(xo)[:sz.xo_bytes].view(np.uint16).reshape(M, ref["K_o_pad"]), ref["xo"])


@pytest.mark.parametrize("M,K", [(1000, 4096), (8192, 4096)])
def test_fused_equals_two_step_path_byte_for_byte(B, M, K):
    """osc_rmsnorm_quantize_extract against osc_rmsnorm + osc_quantize_extract, at the benchmark's size too."""
    rng = np.random.default_rng(5)
    Hb, _ = synth.osc_activations_only(7, M, K, 2)
    gb = gamma_bits(rng, K)
    W = synth.osc_weights_only(1, K, 64, 2)
    w = B.osc_prepare_weights(dev_bf16(W["W"]), W["lut"])
    sz = B.osc_act_sizes(w, M)
    H, g = dev_bf16(Hb), dev_bf16(gb)
    a = [poison(sz.xq_bytes), poison(sz.sfa_bytes), poison(sz.xo_bytes)]
    b = [poison(sz.xq_bytes), poison(sz.sfa_bytes), poison(sz.xo_bytes)]
    B.osc_rmsnorm_quantize_extract(w, H, g, 1e-6, *a)
    X = torch.empty(M, K, dtype=torch.bfloat16, device="cuda")
    B.osc_rmsnorm(H, g, 1e-6, X)
    B.osc_quantize_extract(w, X, *b)
    B.osc_sync_check()
    for u, v, n in zip(a, b, (sz.xq_bytes, sz.sfa_bytes, sz.xo_bytes)):
        assert torch.equal(u[:n], v[:n])


@pytest.mark.parametrize("M,K,N", [(200, 1024, 320), (24, 4096, 256), (1500, 512, 768)])   # 128-row tiles, few-row kernel, pair tiles
def test_rmsnorm_linear_within_tolerance(B, oracle, M, K, N):
    rng = np.random.default_rng(9)
    Hb, gb = residual_rows(rng, M, K), gamma_bits(rng, K)
    c = synth.osc_linear_case(3, M, K, N, 2)
    w = B.osc_prepare_weights(dev_bf16(c["W"]), c["lut"])
    ws = poison(B.osc_act_sizes(w, M).workspace_bytes)
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_rmsnorm_linear(w, dev_bf16(Hb), dev_bf16(gb), 1e-6, Y, ws)
    B.osc_sync_check()
    Yref, T, *_ = oracle.linear(oracle.rmsnorm(Hb, gb, 1e-6), c["W"], c["lut"])
    assert_within_tolerance(host_f64(Y), Yref, T, "rmsnorm_linear")
    # M == 0 is a no-op; too long a row and a missing gamma are refused before any launch
    B.osc_rmsnorm_linear(w, dev_bf16(Hb)[:0], dev_bf16(gb), 1e-6, Y[:0], ws)
    with pytest.raises(B.OscError) as e:
        B.osc_rmsnorm(torch.zeros(2, 8192 + 128, dtype=torch.bfloat16, device="cuda"),
                      torch.zeros(8192 + 128, dtype=torch.bfloat16, device="cuda"), 1e-6,
                      torch.zeros(2, 8192 + 128, dtype=torch.bfloat16, device="cuda"))
    assert e.value.status == -2


# ---- the residual update in front of the norm: H' = bf16(H + R)

def branch_rows(rng, Hb):
    """A branch output to add: mostly smaller than the stream, with entries that cancel it exactly, entries many
    binades below and above it, and half-step ties."""
    H = synth.bf16_bits_to_f64(Hb)
    R = rng.standard_normal(H.shape) * np.abs(H).mean(axis=1, keepdims=True) * 0.3
    Rb = synth.f32_to_bf16_bits(R.astype(np.float32))
    flat_h, flat_r = Hb.reshape(-1), Rb.reshape(-1)
    idx = rng.choice(flat_h.size, size=max(8, flat_h.size // 50), replace=False)
    q = idx.size // 4
    flat_r[idx[:q]] = flat_h[idx[:q]] ^ 0x8000                                              # exact cancellation
    flat_r[idx[q:2 * q]] = synth.f32_to_bf16_bits((H.reshape(-1)[idx[q:2 * q]] * 2.0 ** -8).astype(np.float32))   # ties
    flat_r[idx[2 * q:3 * q]] = synth.f32_to_bf16_bits((H.reshape(-1)[idx[2 * q:3 * q]] * 2.0 ** -30).astype(np.float32))
    flat_r[idx[3 * q:]] = synth.f32_to_bf16_bits((H.reshape(-1)[idx[3 * q:]] * 2.0 ** 20).astype(np.float32))
    return Rb


@pytest.mark.parametrize("M,K,where", [(1, 128, "new"), (37, 384, "H"), (130, 1024, "R"), (64, 4096, "new"), (9, 8192, "H"),
                                       (300, 2048, "new")])
def test_add_rmsnorm_bit_exact(B, oracle, M, K, where):
    rng = np.random.default_rng(M + 2 * K)
    Hb, gb = residual_rows(rng, M, K), gamma_bits(rng, K)
    Rb = branch_rows(rng, Hb)
    Hs_ref, X_ref = oracle.add_rmsnorm(Hb, Rb, gb, 1e-6)
    ld = K + 16
    Hbig = torch.full((M, ld), 7.0, dtype=torch.bfloat16, device="cuda")
    Rbig = torch.full((M, ld), 7.0, dtype=torch.bfloat16, device="cuda")
    Obig = torch.full((M, ld), 7.0, dtype=torch.bfloat16, device="cuda")
    Hbig[:, :K], Rbig[:, :K] = dev_bf16(Hb), dev_bf16(Rb)
    out = {"new": Obig, "H": Hbig, "R": Rbig}[where][:, :K]           # a fresh tensor, or the update in place
    X = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    B.osc_add_rmsnorm(Hbig[:, :K], Rbig[:, :K], dev_bf16(gb), 1e-6, out, X)
    B.osc_sync_check()
    assert np.array_equal(host_bf16_bits(out), Hs_ref)
    assert np.array_equal(host_bf16_bits(X), X_ref)
    for big in (Hbig, Rbig, Obig):
        assert (big[:, K:] == 7.0).all(), "wrote into the padding"
    if where != "H":
        assert np.array_equal(host_bf16_bits(Hbig[:, :K]), Hb)
    if where != "R":
        assert np.array_equal(host_bf16_bits(Rbig[:, :K]), Rb)


@pytest.mark.parametrize("M,K,C", [(129, 384, 2), (300, 1024, 2), (70, 4096, 1), (40, 8192, 3)])
def test_add_rmsnorm_quantize_extract_bit_exact(B, oracle, M, K, C):
    rng = np.random.default_rng(M * 5 + K)
    Hb, gb = residual_rows(rng, M, K), gamma_bits(rng, K)
    Rb = branch_rows(rng, Hb)
    lut = rand_lut(rng, K, C)
    w = B.osc_prepare_weights(dev_bf16(synth.osc_weights_only(1, K, 64, 1)["W"]), lut)
    sz = B.osc_act_sizes(w, M)
    xq, sfa, xo = poison(sz.xq_bytes), poison(sz.sfa_bytes), poison(sz.xo_bytes)
    H = dev_bf16(Hb)
    B.osc_add_rmsnorm_quantize_extract(w, H, dev_bf16(Rb), dev_bf16(gb), 1e-6, H, xq, sfa, xo)     # stream updated in place
    B.osc_sync_check()
    Hs_ref, X_ref = oracle.add_rmsnorm(Hb, Rb, gb, 1e-6)
    assert np.array_equal(host_bf16_bits(H), Hs_ref)
    ref = oracle.quantize_extract(X_ref, lut)
    assert np.array_equal(host_u8(xq)[:sz.xq_bytes].reshape(M, K // 2), ref["xq"])
    valid = valid_sf_bytes(oracle, M, K)
    assert np.array_equal(host_u8(sfa)[:sz.sfa_bytes][valid], ref["sf"][valid])
    if ref["K_o_pad"]:
        assert np.array_equal(host_u8(xo)[:sz.xo_bytes].view(np.uint16).reshape(M, ref["K_o_pad"]), ref["xo"])


def test_add_rmsnorm_linear(B, oracle):
    M, K, N = 333, 1024, 448
    rng = np.random.default_rng(21)
    Hb, gb = residual_rows(rng, M, K), gamma_bits(rng, K)
    Rb = branch_rows(rng, Hb)
    c = synth.osc_linear_case(3, M, K, N, 2)
    w = B.osc_prepare_weights(dev_bf16(c["W"]), c["lut"])
    ws = poison(B.osc_act_sizes(w, M).workspace_bytes)
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    Hout = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    B.osc_add_rmsnorm_linear(w, dev_bf16(Hb), dev_bf16(Rb), dev_bf16(gb), 1e-6, Hout, Y, ws)
    B.osc_sync_check()
    Hs_ref, X_ref = oracle.add_rmsnorm(Hb, Rb, gb, 1e-6)
    assert np.array_equal(host_bf16_bits(Hout), Hs_ref)
    Yref, T, *_ = oracle.linear(X_ref, c["W"], c["lut"])
    assert_within_tolerance(host_f64(Y), Yref, T, "add + rmsnorm + linear")
    with pytest.raises(B.OscError) as err:          # a missing branch tensor is refused before any launch
        B.osc_add_rmsnorm_linear(w, dev_bf16(Hb), dev_bf16(Rb)[:0], dev_bf16(gb), 1e-6, Hout, Y, ws)
    assert err.value.status == -1
