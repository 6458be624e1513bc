"""Few-row kernel (operands swapped, K split over a thread-block cluster; a 64-row and a 256-row form) against
the oracle.

The library routes to it by itself for few rows; here OSC_DECODE=2 forces it for every M <= 256 and
OSC_DECODE_SPLIT forces cluster sizes (1 = no reduction, up to 8), so that every reduction path, ranks whose
K slice holds only Path-B blocks, odd numbers of 128-channel scale blocks, feature tiles cut by N and token
counts that are not multiples of 16 are all covered.  OSC_DECODE=0 keeps the 128-row-tile kernel covered
for the same shapes."""
import os

import numpy as np
import pytest
import torch

from paper_2604_12782_b200 import synth

pytestmark = pytest.mark.gpu

from gpu_util import assert_within_tolerance, dev_bf16, host_f64, poison  # noqa: E402


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_12782_b200 import binding
    return binding


@pytest.fixture
def env():
    saved = {k: os.environ.get(k) for k in ("OSC_DECODE", "OSC_DECODE_SPLIT", "OSC_DECODE_FUSED_ROWS")}

    def set_(decode, split=None, fused_rows=0):
        os.environ["OSC_DECODE"] = str(decode)
        os.environ["OSC_DECODE_FUSED_ROWS"] = str(fused_rows)   # 0: the quantizer kernel runs in front
        if split is None:
            os.environ.pop("OSC_DECODE_SPLIT", None)
        else:
            os.environ["OSC_DECODE_SPLIT"] = str(split)
    yield set_
    for k, v in saved.items():
        if v is None:
            os.environ.pop(k, None)
        else:
            os.environ[k] = v


def lut_for(rng, K, kind):
    Kg = K // 32
    if kind == "empty":
        return np.full((Kg, 1), -1, np.int8)
    if kind == "full":
        return np.tile(np.arange(32, dtype=np.int8), (Kg, 1))
    c = {"one": 1, "two": 2}[kind]
    return np.stack([rng.permutation(32)[:c] for _ in range(Kg)]).astype(np.int8)


CASES = [  # M, K, N, table, split (None = the library's choice)
    (1, 128, 64, "one", None), (16, 512, 512, "two", None), (17, 384, 320, "one", 2), (33, 640, 192, "two", 3),
    (64, 1024, 448, "one", 4), (48, 2048, 256, "two", 8), (5, 256, 128, "empty", 1), (64, 128, 64, "full", 2),
    (31, 1536, 1024, "one", 5), (64, 4096, 512, "two", None), (20, 4096, 384, "two", 3), (64, 3072, 256, "one", 5),
    (32, 4096, 128, "two", 7),
    # sixteen rows or fewer also run with the quantizer inside the kernel
    (16, 4096, 384, "two", 3), (9, 640, 192, "two", 3), (16, 1536, 1024, "one", 5), (13, 128, 64, "full", 2),
    (2, 3072, 256, "one", 8), (16, 2048, 128, "two", 1), (11, 1024, 64, "full", 4),
    (8, 2048, 128, "full", 2),      # more than 1024 flagged channels: the quantizer stays a kernel of its own
    # the 256-row form: one and two 128-row scale blocks of activations, token counts off the multiples of 16
    (65, 512, 192, "two", None), (128, 1024, 256, "one", 2), (129, 384, 320, "two", 3), (200, 2048, 128, "one", 4),
    (256, 640, 448, "two", 1), (250, 4096, 64, "two", 8), (144, 256, 128, "empty", 2), (256, 128, 64, "full", 2),
]


@pytest.mark.parametrize("M,K,N,kind,split", CASES)
def test_decode_kernel_osc(B, oracle, env, M, K, N, kind, split):
    rng = np.random.default_rng(M * 7 + K + N)
    c = synth.osc_linear_case(M + N, M, K, N, 1)
    lut = lut_for(rng, K, kind)
    Yref, T, act, _ = oracle.linear(c["X"], c["W"], lut)
    w = B.osc_prepare_weights(dev_bf16(c["W"]), lut)
    sz = B.osc_act_sizes(w, M)
    outs = {}
    for mode in (2, 0):
        env(mode, split if mode else None)
        ws = poison(sz.workspace_bytes)
        Ybig = torch.full((M + 2, N + 64), 7.0, dtype=torch.bfloat16, device="cuda")
        Y = Ybig[1:M + 1, :N]
        B.osc_linear(w, dev_bf16(c["X"]), Y, ws)
        B.osc_sync_check()
        assert np.array_equal(ws[sz.xq_offset:sz.xq_offset + sz.xq_bytes].cpu().numpy().reshape(M, K // 2), act["xq"])
        assert_within_tolerance(host_f64(Y), Yref, T, f"decode={mode} M={M} K={K} N={N} {kind} S={split}")
        guard = Ybig.clone()
        guard[1:M + 1, :N] = 7.0
        assert (guard == 7.0).all(), "wrote outside Y"
        outs[mode] = Y.clone()
    # the two kernels add the same exact products in different orders: equal up to fp32 rounding of the sums
    d = (outs[2].float() - outs[0].float()).abs().cpu().numpy().astype(np.float64)
    assert (d <= 2.0 ** -7 * np.abs(Yref) + 1e-3 * T).all()
    if M <= 16:
        # the form that quantizes the activations of its K slice inside the few-row kernel: no workspace traffic,
        # the same codes, scales and accumulation order, hence the same bits
        env(2, split, fused_rows=16)
        ws = poison(sz.workspace_bytes)
        before = ws.clone()
        Ybig = torch.full((M + 2, N + 64), 7.0, dtype=torch.bfloat16, device="cuda")
        Y = Ybig[1:M + 1, :N]
        B.osc_linear(w, dev_bf16(c["X"]), Y, ws)
        B.osc_sync_check()
        assert torch.equal(ws, before) == (w.K_o_pad <= 1024), "the quantizing form does not use the workspace"
        assert torch.equal(Y.view(torch.int16), outs[2].view(torch.int16))
        guard = Ybig.clone()
        guard[1:M + 1, :N] = 7.0
        assert (guard == 7.0).all(), "wrote outside Y"


@pytest.mark.parametrize("M,K,N,split", [(1, 128, 64, None), (16, 768, 320, 3), (40, 1536, 1024, 4), (64, 12288, 256, 8),
                                         (64, 256, 192, 2), (9, 4096, 128, 1),
                                         (65, 768, 192, None), (128, 8192, 256, 4), (200, 1536, 320, 3), (256, 12288, 128, 8),
                                         (255, 128, 64, 1)])
def test_decode_kernel_fp8(B, oracle, env, M, K, N, split):
    c = synth.fp8_linear_case(M + K, M, K, N)
    Yref, T, (x8, sx), _ = oracle.fp8_linear(c["X"], c["W"])
    w = B.osc_fp8_prepare_weights(dev_bf16(c["W"]))
    sz = B.osc_fp8_act_sizes(w, M)
    for mode in (2, 0):
        env(mode, split if mode else None)
        ws = poison(sz.workspace_bytes)
        Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        B.osc_fp8_linear(w, dev_bf16(c["X"]), Y, ws)
        B.osc_sync_check()
        assert np.array_equal(ws[sz.x8_offset:sz.x8_offset + M * K].cpu().numpy().reshape(M, K), x8)
        assert_within_tolerance(host_f64(Y), Yref, T, f"fp8 decode={mode} M={M} K={K} N={N} S={split}")


def test_decode_kernel_is_deterministic(B, env):
    env(2, 4)
    c = synth.osc_linear_case(3, 24, 2048, 768, 2)
    w = B.osc_prepare_weights(dev_bf16(c["W"]), c["lut"])
    sz = B.osc_act_sizes(w, 24)
    ws = poison(sz.workspace_bytes)
    X = dev_bf16(c["X"])
    Ys = []
    for _ in range(3):
        Y = torch.empty((24, 768), dtype=torch.bfloat16, device="cuda")
        B.osc_linear(w, X, Y, ws)
        Ys.append(Y)
    B.osc_sync_check()
    assert torch.equal(Ys[0], Ys[1]) and torch.equal(Ys[0], Ys[2])


@pytest.mark.parametrize("M,K,N,split", [(1, 128, 64, None), (16, 768, 320, 3), (40, 1536, 1024, 4), (64, 12288, 256, 8),
                                         (33, 384, 192, 2),
                                         (65, 768, 192, None), (128, 8192, 256, 4), (129, 1536, 320, 3), (256, 12288, 128, 8),
                                         (250, 128, 64, 1)])
def test_decode_kernel_mxfp8(B, oracle, env, M, K, N, split):
    c = synth.fp8_linear_case(M + K + 1, M, K, N)
    Yref, T, (x8, sfa), _ = oracle.mxfp8_linear(c["X"], c["W"])
    w = B.osc_mxfp8_prepare_weights(dev_bf16(c["W"]))
    sz = B.osc_mxfp8_act_sizes(w, M)
    for mode in (2, 0):
        env(mode, split if mode else None)
        ws = poison(sz.workspace_bytes)
        Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        B.osc_mxfp8_linear(w, dev_bf16(c["X"]), Y, ws)
        B.osc_sync_check()
        assert np.array_equal(ws[sz.x8_offset:sz.x8_offset + M * K].cpu().numpy().reshape(M, K), x8)
        assert_within_tolerance(host_f64(Y), Yref, T, f"mxfp8 decode={mode} M={M} K={K} N={N} S={split}")


@pytest.mark.parametrize("M,K,N,kind,split", [
    (1, 128, 64, "one", None), (16, 512, 512, "two", None), (17, 384, 320, "one", 2), (33, 640, 192, "two", 3),
    (64, 1024, 448, "one", 4), (48, 2048, 256, "empty", 8), (64, 4096, 512, "one", None), (20, 4096, 384, "two", 3),
    (65, 512, 192, "two", None), (129, 384, 320, "one", 3), (200, 2048, 128, "one", 4), (256, 640, 448, "two", 1),
    (250, 4096, 64, "one", 8)])
def test_decode_kernel_nvfp4(B, oracle, env, M, K, N, kind, split):
    """NVFP4 / G = 16 on the few-row kernel (four 64-channel scale blocks per stage, E4M3 scales, power-of-two output
    scale), forced for every M <= 256 and every cluster size, against the oracle and against the pair kernel."""
    c = synth.osc16_linear_case(M + K + 3, M, K, N)
    rng = np.random.default_rng(N + M)
    lut16 = {"one": c["lut16"], "empty": np.full((K // 16, 1), -1, np.int8),
             "two": np.stack([rng.permutation(16)[:2] for _ in range(K // 16)]).astype(np.int8)}[kind]
    ex, ew = synth.nvfp4_tensor_exponent(c["X"]), synth.nvfp4_tensor_exponent(c["W"])
    Yref, T, *_ = oracle.nvfp4_linear(c["X"], c["W"], lut16, ex, ew)
    w = B.osc_nvfp4_prepare_weights(dev_bf16(c["W"]), lut16, ew)
    sz = B.osc_nvfp4_act_sizes(w, M)
    X = dev_bf16(c["X"])
    for mode in (2, 0):
        env(mode, split if mode else None)
        ws = poison(sz.workspace_bytes)
        big = torch.full((M + 2, N + 8), 7.0, dtype=torch.bfloat16, device="cuda")
        B.osc_nvfp4_linear(w, X, ex, big[1:M + 1, :N], ws)
        B.osc_sync_check()
        assert_within_tolerance(host_f64(big[1:M + 1, :N]), Yref, T, f"nvfp4 decode={mode} M={M} K={K} N={N} S={split}")
        guard = big.clone()
        guard[1:M + 1, :N] = 7.0
        assert (guard == 7.0).all(), "wrote outside Y"


@pytest.mark.parametrize("side_stream", [False, True], ids=["default_stream", "side_stream"])
@pytest.mark.parametrize("kind", ["osc", "fp8", "mxfp8", "nvfp4"])
def test_linear_right_after_prepare(B, oracle, kind, side_stream):
    """A few-row linear issued on the same stream directly behind its weight preparation, with nothing in between:
    the few-row kernel streams weights ahead of its dependency wait, so the preparation has to be complete before
    any later launch may begin.  The buffers the preparation allocates are made to reuse memory full of 0xFF, so
    weights read too early would show.  Checked against the oracle and against the same call after a sync."""
    M, K, N = 16, 4096, 2048
    if kind in ("osc", "nvfp4"):
        c = synth.osc_linear_case(5, M, K, N, 2) if kind == "osc" else synth.osc16_linear_case(5, M, K, N)
    else:
        c = synth.fp8_linear_case(5, M, K, N)
    X, W = dev_bf16(c["X"]), dev_bf16(c["W"])
    Y1 = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    Y2 = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    ws = poison(64 << 20)
    # blocks of the sizes the preparation will ask for, filled with 0xFF and handed back to the caching allocator
    for nbytes in (N * K, N * K // 2, N * 4, N * 512 * 2, N * K // 32, N * K // 16, 1 << 20):
        poison(nbytes)
    torch.cuda.synchronize()
    if side_stream:   # a stream of its own (non-blocking): programmatic launches overlap for certain
        with torch.cuda.stream(torch.cuda.Stream()):
            _right_after_prepare(B, oracle, kind, c, X, W, Y1, Y2, ws, M)
    else:
        _right_after_prepare(B, oracle, kind, c, X, W, Y1, Y2, ws, M)


def _right_after_prepare(B, oracle, kind, c, X, W, Y1, Y2, ws, M):
    if kind == "osc":
        w = B.osc_prepare_weights(W, c["lut"])
        B.osc_linear(w, X, Y1, ws)
        torch.cuda.synchronize()
        B.osc_linear(w, X, Y2, ws)
        Yref, T, *_ = oracle.linear(c["X"], c["W"], c["lut"])
    elif kind == "fp8":
        w = B.osc_fp8_prepare_weights(W)
        B.osc_fp8_linear(w, X, Y1, ws)
        torch.cuda.synchronize()
        B.osc_fp8_linear(w, X, Y2, ws)
        Yref, T, *_ = oracle.fp8_linear(c["X"], c["W"])
    elif kind == "mxfp8":
        w = B.osc_mxfp8_prepare_weights(W)
        B.osc_mxfp8_linear(w, X, Y1, ws)
        torch.cuda.synchronize()
        B.osc_mxfp8_linear(w, X, Y2, ws)
        Yref, T, *_ = oracle.mxfp8_linear(c["X"], c["W"])
    else:
        ex, ew = synth.nvfp4_tensor_exponent(c["X"]), synth.nvfp4_tensor_exponent(c["W"])
        w = B.osc_nvfp4_prepare_weights(W, c["lut16"], ew)
        B.osc_nvfp4_linear(w, X, ex, Y1, ws)
        torch.cuda.synchronize()
        B.osc_nvfp4_linear(w, X, ex, Y2, ws)
        Yref, T, *_ = oracle.nvfp4_linear(c["X"], c["W"], c["lut16"], ex, ew)
    B.osc_sync_check()
    assert_within_tolerance(host_f64(Y1), Yref, T, f"{kind}: linear directly behind prepare")
    assert torch.equal(Y1.view(torch.int16), Y2.view(torch.int16)), "the call behind the preparation differs from the call after a sync"
