"""GPU parity of the SwiGLU fused in front of the per-token FP8 quantizer (Sections 3.3 / 3.4): the activation
rows, the E4M3 codes and the per-row scales are compared bit for bit with the oracle (the same fixed fp32 steps),
the fused kernel byte for byte with the library's own two-step path, the linear within the stated tolerance."""
import numpy as np
import pytest
import torch

from paper_2604_12782_b200 import synth

pytestmark = pytest.mark.gpu

from gpu_util import assert_within_tolerance, dev_bf16, host_bf16_bits, host_f64, host_u8, poison  # noqa: E402
from producer_inputs import SWIGLU_ROW_CASES, gate_up  # noqa: E402


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_12782_b200 import binding
    return binding


@pytest.mark.parametrize("M,I", SWIGLU_ROW_CASES)
def test_swiglu_rows_bit_exact(B, oracle, M, I):
    rng = np.random.default_rng(M + I)
    GUb = gate_up(rng, M, I, pad=8)
    H = torch.full((M, I + 8), 7.0, dtype=torch.bfloat16, device="cuda")
    B.osc_swiglu(dev_bf16(GUb), I, H[:, :I])
    B.osc_sync_check()
    want = oracle.swiglu(GUb, I)
    got = host_bf16_bits(H[:, :I].contiguous())
    assert np.array_equal(got, want), f"{np.count_nonzero(got != want)} of {got.size} elements differ"
    assert (H[:, I:] == 7.0).all()
    # and against the plain all-double definition (one rounding): one bf16 unit at most, except where the clamp of
    # the exponential shows, which is only in results below 2^-100 in magnitude
    from oracle import plain
    ref = plain.swiglu_plain(GUb, I)
    far = plain.bf16_units_apart(got, ref) > 1
    tiny = np.abs(synth.bf16_bits_to_f64(got)) + np.abs(synth.bf16_bits_to_f64(ref)) < 2.0 ** -100
    assert not (far & ~tiny).any()


@pytest.mark.parametrize("M,I", [(1, 128), (129, 384), (300, 1024), (33, 12288), (7, 16384)])
def test_fused_quantize_bit_exact(B, oracle, M, I):
    rng = np.random.default_rng(M * 3 + I)
    GUb = gate_up(rng, M, I)
    x8 = poison(M * I)
    sx = torch.full((M,), float("nan"), dtype=torch.float32, device="cuda")
    B.osc_swiglu_fp8_quantize(dev_bf16(GUb), I, x8, sx)
    B.osc_sync_check()
    ref8, refs = oracle.fp8_quantize(oracle.swiglu(GUb, I))
    assert np.array_equal(host_u8(x8)[:M * I].reshape(M, I), ref8)
    assert np.array_equal(sx.cpu().numpy().view(np.uint32), refs.view(np.uint32))


@pytest.mark.parametrize("M,I", [(1000, 4096), (4096, 12288)])
def test_fused_equals_two_step_path_byte_for_byte(B, M, I):
    rng = np.random.default_rng(5)
    GU = dev_bf16(gate_up(rng, M, I))
    a8, b8 = poison(M * I), poison(M * I)
    asx, bsx = (torch.empty(M, dtype=torch.float32, device="cuda") for _ in range(2))
    B.osc_swiglu_fp8_quantize(GU, I, a8, asx)
    H = torch.empty(M, I, dtype=torch.bfloat16, device="cuda")
    B.osc_swiglu(GU, I, H)
    B.osc_fp8_quantize(H, b8, bsx)
    B.osc_sync_check()
    assert torch.equal(a8[:M * I], b8[:M * I]) and torch.equal(asx.view(torch.int32), bsx.view(torch.int32))


@pytest.mark.parametrize("M,I,N", [(200, 1024, 320), (16, 2048, 256), (1200, 512, 512)])   # 128-row tiles, few-row kernel, pair tiles
def test_swiglu_fp8_linear_within_tolerance(B, oracle, M, I, N):
    rng = np.random.default_rng(9)
    GUb = gate_up(rng, M, I)
    W = synth.fp8_linear_case(3, 1, I, N)["W"]
    w = B.osc_fp8_prepare_weights(dev_bf16(W))
    ws = poison(B.osc_fp8_act_sizes(w, M).workspace_bytes)
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_swiglu_fp8_linear(w, dev_bf16(GUb), Y, ws)
    B.osc_sync_check()
    Yref, T, *_ = oracle.fp8_linear(oracle.swiglu(GUb, I), W)
    assert_within_tolerance(host_f64(Y), Yref, T, "swiglu_fp8_linear")
    B.osc_swiglu_fp8_linear(w, dev_bf16(GUb)[:0], Y[:0], ws)          # M == 0: a no-op
    with pytest.raises(B.OscError) as e:                                 # a row of h must fit in registers
        B.osc_swiglu(torch.zeros(2, 2 * 16512, dtype=torch.bfloat16, device="cuda"), 16512,
                     torch.zeros(2, 16512, dtype=torch.bfloat16, device="cuda"))
    assert e.value.status == -2
