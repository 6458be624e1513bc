"""GPU parity: the CUDA library (through the C ABI) against the CPU oracle on the same seeded inputs.

Bit-exact for packed codes, scale bytes, gathered channels and FP8 codes/scales; the GEMM outputs
within |err| <= 2^-7 |ref| + 1e-3 sum_k |a_k b_k| per element.
"""
import numpy as np
import pytest
import torch

from paper_2604_12782_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_12782_b200 import binding
    return binding


from gpu_util import (assert_within_tolerance, dev_bf16, host_bf16_bits, host_f64, host_u8, poison,  # noqa: E402
                      valid_sf_bytes)


def rand_lut(rng, K, C, p_none=0.2):
    lut = np.full((K // 32, C), -1, np.int8)
    for k in range(K // 32):
        ch = rng.permutation(32)[:C]
        for c in range(C):
            if rng.random() > p_none:
                lut[k, c] = ch[c]
    return lut


def run_quantize(B, w, X_bits):
    M = X_bits.shape[0]
    sz = B.osc_act_sizes(w, M)
    xq, sfa, xo = poison(sz.xq_bytes), poison(sz.sfa_bytes), poison(sz.xo_bytes)
    X = dev_bf16(X_bits)
    B.osc_quantize_extract(w, X, xq, sfa, xo)
    B.osc_sync_check()
    return sz, xq, sfa, xo


def compare_quantized(oracle, ref, xq, sf, xo, rows, K, sizes):
    xq_h = host_u8(xq)[:sizes[0]].reshape(rows, K // 2)
    assert np.array_equal(xq_h, ref["xq"]), f"packed codes differ in {np.count_nonzero(xq_h != ref['xq'])} bytes"
    sf_h = host_u8(sf)[:sizes[1]]
    assert sf_h.size == ref["sf"].size
    valid = valid_sf_bytes(oracle, rows, K)
    assert np.array_equal(sf_h[valid], ref["sf"][valid]), "scale bytes differ"
    pad = np.ones(sf_h.size, bool)
    pad[valid] = False
    assert not sf_h[pad].any(), "scale bytes of rows beyond the row count must be 0"
    if ref["K_o_pad"]:
        xo_h = host_u8(xo)[:sizes[2]].view(np.uint16).reshape(rows, ref["K_o_pad"])
        assert np.array_equal(xo_h, ref["xo"]), "gathered channels differ"


QUANT_CASES = [
    # (M, K, lut kind)
    (64, 512, "tiny"),
    (300, 1024, "rand2"),     # ragged last row tile, several column blocks, some groups without a channel
    (1, 128, "rand1"),
    (129, 256, "empty"),
    (40, 128, "full"),
    (257, 384, "rand4"),
]


@pytest.mark.parametrize("M,K,kind", QUANT_CASES)
def test_quantize_extract_bit_exact(B, oracle, M, K, kind):
    rng = np.random.default_rng(M * 7 + K)
    if kind == "tiny":
        case = synth.tiny_case()
        X_bits, lut = case["X"], case["lut"]
    else:
        Xf, _ = synth.planted_activations(rng, M, K, 2)
        Xf[rng.random((M, K)) < 0.02] = 0.0
        Xf[0, :32] = 0.0                      # an all-zero group
        Xf[M - 1, -32:] *= 2.0 ** -60          # tiny magnitudes
        Xf[0, 33] = -0.0
        X_bits = synth.f32_to_bf16_bits(Xf.astype(np.float32))
        lut = {"rand1": lambda: rand_lut(rng, K, 1), "rand2": lambda: rand_lut(rng, K, 2),
               "rand4": lambda: rand_lut(rng, K, 4), "empty": lambda: np.full((K // 32, 1), -1, np.int8),
               "full": lambda: np.tile(np.arange(32, dtype=np.int8), (K // 32, 1))}[kind]()
    W = dev_bf16(np.zeros((64, K), np.uint16))
    w = B.osc_prepare_weights(W, lut)
    sz, xq, sfa, xo = run_quantize(B, w, X_bits)
    ref = oracle.quantize_extract(X_bits, lut)
    assert (w.K_o, w.K_o_pad) == (ref["K_o"], ref["K_o_pad"])
    compare_quantized(oracle, ref, xq, sfa, xo, M, K, (sz.xq_bytes, sz.sfa_bytes, sz.xo_bytes))
    # the device copy of the table
    meta = host_u8(w.keep["meta"])
    Kg = K // 32
    assert np.array_equal(meta[:Kg * 4].view(np.uint32), ref["mask"])
    assert np.array_equal(meta[Kg * 4:Kg * 8].view(np.int32), ref["prefix"])
    assert np.array_equal(meta[Kg * 8:Kg * 8 + ref["K_o"] * 4].view(np.int32), ref["idx_o"])


def test_strided_input_rows(B, oracle):
    rng = np.random.default_rng(5)
    M, K = 70, 256
    big = synth.f32_to_bf16_bits(rng.standard_normal((M, K + 64)).astype(np.float32))
    lut = rand_lut(rng, K, 1)
    w = B.osc_prepare_weights(dev_bf16(np.zeros((64, K), np.uint16)), lut)
    Xd = dev_bf16(big)[:, :K]
    sz = B.osc_act_sizes(w, M)
    xq, sfa, xo = poison(sz.xq_bytes), poison(sz.sfa_bytes), poison(sz.xo_bytes)
    B.osc_quantize_extract(w, Xd, xq, sfa, xo)
    B.osc_sync_check()
    ref = oracle.quantize_extract(big[:, :K], lut)
    compare_quantized(oracle, ref, xq, sfa, xo, M, K, (sz.xq_bytes, sz.sfa_bytes, sz.xo_bytes))


def test_prepare_weights_bit_exact(B, oracle):
    case = synth.osc_linear_case(3, 0, 512, 320, 2)
    w = B.osc_prepare_weights(dev_bf16(case["W"]), case["lut"])
    B.osc_sync_check()
    ref = oracle.prepare_weights(case["W"], case["lut"])
    compare_quantized(oracle, ref, w.keep["wq"], w.keep["sfw"], w.keep["wo"], 320, 512,
                      (w.sizes.wq_bytes, w.sizes.sfw_bytes, w.sizes.wo_bytes))


@pytest.mark.parametrize("M,K", [(37, 12288), (5, 128), (130, 768), (3, 16384 + 256)])
def test_fp8_quantize_bit_exact(B, oracle, M, K):
    case = synth.fp8_linear_case(M, M, K, 8)
    Xb = case["X"].copy()
    Xb[0, :] = 0                                  # all-zero row: scale floors at 2^-40/448
    Xb[M - 1, 3] = 0x8000                         # -0.0
    x8, sx = poison(M * K), torch.full((M,), float("nan"), device="cuda")
    B.osc_fp8_quantize(dev_bf16(Xb), x8, sx)
    B.osc_sync_check()
    r8, rs = oracle.fp8_quantize(Xb)
    assert np.array_equal(sx.cpu().numpy().view(np.uint32), rs.view(np.uint32)), "row scales differ"
    got = host_u8(x8)[:M * K].reshape(M, K)
    assert np.array_equal(got, r8), f"{np.count_nonzero(got != r8)} E4M3 codes differ"


def oracle_weights(oracle, W_bits, lut):
    return oracle.prepare_weights(W_bits, lut)


GEMM_CASES = [
    # (M, N, K, lut kind, seed)
    (64, 512, 512, "tiny", 0),
    (128, 256, 256, "empty", 1),       # one tile, plain W4A4
    (200, 320, 1024, "rand2", 2),      # ragged M, N tail inside a tile
    (128, 128, 128, "full", 3),        # every channel protected: a BF16 GEMM
    (385, 704, 384, "rand1", 4),       # K = 1.5 x 256: half FP4 block; several tiles both ways
    (1, 64, 128, "rand1", 5),
    (1300, 1536, 2048, "rand1", 6),    # > 148 tiles with BLOCK_N = 128: CTAs loop over tiles
]


def make_case(kind, M, N, K, seed):
    rng = np.random.default_rng(seed)
    if kind == "tiny":
        c = synth.tiny_case()
        return c["X"], c["W"], c["lut"]
    c = synth.osc_linear_case(seed, M, K, N, 2)
    lut = {"rand1": lambda: rand_lut(rng, K, 1), "rand2": lambda: rand_lut(rng, K, 2),
           "empty": lambda: np.full((K // 32, 1), -1, np.int8),
           "full": lambda: np.tile(np.arange(32, dtype=np.int8), (K // 32, 1))}[kind]()
    return c["X"], c["W"], lut


@pytest.mark.parametrize("M,N,K,kind,seed", GEMM_CASES)
def test_gemm_dual_within_tolerance(B, oracle, M, N, K, kind, seed):
    X_bits, W_bits, lut = make_case(kind, M, N, K, seed)
    w = B.osc_prepare_weights(dev_bf16(W_bits), lut)
    sz, xq, sfa, xo = run_quantize(B, w, X_bits)
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_gemm_dual(w, xq, sfa, xo, M, Y)
    B.osc_sync_check()
    Yref, T, act, wts = oracle.linear(X_bits, W_bits, lut)
    # the operands the GPU multiplied are the oracle's own, bit for bit
    compare_quantized(oracle, act, xq, sfa, xo, M, K, (sz.xq_bytes, sz.sfa_bytes, sz.xo_bytes))
    assert_within_tolerance(host_f64(Y), Yref, T, f"gemm_dual {M}x{N}x{K} {kind}")


def test_osc_linear_matches_two_step_path_and_padding_is_untouched(B, oracle):
    X_bits, W_bits, lut = make_case("rand2", 200, 320, 1024, 2)
    M, N, K = 200, 320, 1024
    w = B.osc_prepare_weights(dev_bf16(W_bits), lut)
    sz = B.osc_act_sizes(w, M)
    ws = poison(sz.workspace_bytes)
    Ybig = torch.full((M + 2, N + 64), 7.0, dtype=torch.bfloat16, device="cuda")   # guard band around Y
    Y = Ybig[1:M + 1, :N]
    B.osc_linear(w, dev_bf16(X_bits), Y, ws)
    B.osc_sync_check()
    Yref, T, *_ = oracle.linear(X_bits, W_bits, lut)
    assert_within_tolerance(host_f64(Y), Yref, T, "osc_linear")
    guard = Ybig.clone()
    guard[1:M + 1, :N] = 7.0
    assert (guard == 7.0).all(), "osc_linear wrote outside Y"
    # M == 0 is a successful no-op
    B.osc_linear(w, dev_bf16(X_bits)[:0], Y[:0], ws)
    # too small a workspace is refused before any launch
    with pytest.raises(B.OscError) as e:
        B.osc_linear(w, dev_bf16(X_bits), Y, ws[:1024])
    assert e.value.status == -5


FP8_CASES = [(48, 128, 256, 0), (200, 320, 768, 1), (1, 64, 128, 2), (700, 1280, 1536, 3)]


@pytest.mark.parametrize("M,N,K,seed", FP8_CASES)
def test_fp8_linear_within_tolerance(B, oracle, M, N, K, seed):
    c = synth.fp8_linear_case(seed, M, K, N)
    w = B.osc_fp8_prepare_weights(dev_bf16(c["W"]))
    sz = B.osc_fp8_act_sizes(w, M)
    ws = poison(sz.workspace_bytes)
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_fp8_linear(w, dev_bf16(c["X"]), Y, ws)
    B.osc_sync_check()
    Yref, T, (x8, sx), (w8, sw) = oracle.fp8_linear(c["X"], c["W"])
    assert np.array_equal(host_u8(w.keep["w8"])[:N * K].reshape(N, K), w8)
    assert np.array_equal(w.keep["sw"].cpu().numpy().view(np.uint32), sw.view(np.uint32))
    got8 = host_u8(ws)[sz.x8_offset:sz.x8_offset + M * K].reshape(M, K)
    assert np.array_equal(got8, x8)
    assert_within_tolerance(host_f64(Y), Yref, T, f"fp8_linear {M}x{N}x{K}")
    # GEMM-only entry point on the same operands
    Y2 = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_fp8_gemm(w, ws[sz.x8_offset:], ws[sz.sx_offset:], M, Y2)
    B.osc_sync_check()
    assert torch.equal(Y, Y2)


def grouped_counts(kind):
    """"small" averages under 96 rows per expert (128-row tiles, single-CTA kernel); "mid" and "zipf" run on the
    CTA-pair kernel with 256-row tiles: experts ending inside the first / second half of a tile, on a tile edge,
    empty experts, one-row experts."""
    if kind == "small":
        return np.array([3, 0, 130, 1, 257, 128])
    if kind == "mid":
        return np.array([300, 0, 5, 256, 129, 511, 1, 385])
    return synth.zipf_expert_rows(E=16, T=512, top_k=4, seed=1)


@pytest.mark.parametrize("kind", ["small", "mid", "zipf"])
def test_grouped_osc_linear(B, oracle, kind):
    counts = grouped_counts(kind)
    E, K, N = counts.size, 256, (320 if kind == "mid" else 192)
    c = synth.moe_gate_up_case(E, counts, K=K, N=N, seed=3)
    M = c["M"]
    w = B.osc_prepare_weights_grouped(dev_bf16(c["W"].reshape(E * N, K)).view(E, N, K), c["lut"])
    sz = B.osc_act_sizes(w, M)
    ws = poison(sz.workspace_bytes)
    off = torch.from_numpy(c["off"]).cuda()
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_linear_grouped(w, dev_bf16(c["X"]), off, Y, ws)
    B.osc_sync_check()
    # quantized operands, expert by expert
    gq = oracle.quantize_extract_grouped(c["X"], c["off"], c["lut"])
    ws_h = host_u8(ws)
    assert np.array_equal(ws_h[sz.xq_offset:sz.xq_offset + sz.xq_bytes].reshape(M, K // 2), gq["xq"])
    sf_h = ws_h[sz.sfa_offset:sz.sfa_offset + gq["sf"].size]
    for e in range(E):
        if counts[e]:
            v = valid_sf_bytes(oracle, int(counts[e]), K, int(gq["sf_row_base"][e]))
            assert np.array_equal(sf_h[v], gq["sf"][v]), f"scales of expert {e}"
    if gq["K_o_pad"]:
        xo_h = ws_h[sz.xo_offset:sz.xo_offset + sz.xo_bytes].view(np.uint16).reshape(M, gq["K_o_pad"])
        assert np.array_equal(xo_h, gq["xo"])
    # outputs, expert by expert with that expert's weights
    Yh = host_f64(Y)
    for e in range(E):
        r0, r1 = int(c["off"][e]), int(c["off"][e + 1])
        if r1 == r0:
            continue
        Yref, T, *_ = oracle.linear(c["X"][r0:r1], c["W"][e], c["lut"])
        assert_within_tolerance(Yh[r0:r1], Yref, T, f"grouped expert {e}")


@pytest.mark.parametrize("kind", ["small", "mid"])
def test_grouped_fp8_linear(B, oracle, kind):
    counts = grouped_counts(kind)
    E, K, N = counts.size, 384, (320 if kind == "mid" else 128)
    c = synth.moe_down_case(E, counts, K=K, N=N, seed=4)
    M = c["M"]
    w = B.osc_fp8_prepare_weights_grouped(dev_bf16(c["W"].reshape(E * N, K)).view(E, N, K))
    sz = B.osc_fp8_act_sizes(w, M)
    ws = poison(sz.workspace_bytes)
    off = torch.from_numpy(c["off"]).cuda()
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_fp8_linear_grouped(w, dev_bf16(c["X"]), off, Y, ws)
    B.osc_sync_check()
    Yh = host_f64(Y)
    for e in range(E):
        r0, r1 = int(c["off"][e]), int(c["off"][e + 1])
        if r1 == r0:
            continue
        Yref, T, *_ = oracle.fp8_linear(c["X"][r0:r1], c["W"][e])
        assert_within_tolerance(Yh[r0:r1], Yref, T, f"grouped fp8 expert {e}")


def test_error_ordering_on_device(B, oracle):
    """OSC output is closer to the exact product than unprotected MXFP4 on outlier-planted inputs."""
    c = synth.tiny_case()
    exact = synth.bf16_bits_to_f64(c["X"]) @ synth.bf16_bits_to_f64(c["W"]).T

    def run(lut):
        w = B.osc_prepare_weights(dev_bf16(c["W"]), lut)
        sz = B.osc_act_sizes(w, 64)
        ws = poison(sz.workspace_bytes)
        Y = torch.empty(64, 512, dtype=torch.bfloat16, device="cuda")
        B.osc_linear(w, dev_bf16(c["X"]), Y, ws)
        B.osc_sync_check()
        return np.linalg.norm(host_f64(Y) - exact) / np.linalg.norm(exact)

    assert run(c["lut"]) < 0.3 * run(np.full((16, 1), -1, np.int8))


def test_calls_can_be_captured_in_a_cuda_graph(B, oracle):
    """The calls allocate nothing and never synchronise, so a sequence of them can be captured once and replayed:
    the replay must give the bytes of a plain launch, for the dual-path, the few-row and the FP8 paths."""
    outs = {}
    for M in (24, 300):
        X_bits, W_bits, lut = make_case("rand1", M, 320, 512, 5)
        w = B.osc_prepare_weights(dev_bf16(W_bits), lut)
        w8 = B.osc_fp8_prepare_weights(dev_bf16(W_bits))
        sz, sz8 = B.osc_act_sizes(w, M), B.osc_fp8_act_sizes(w8, M)
        ws, ws8 = poison(sz.workspace_bytes), poison(sz8.workspace_bytes)
        X = dev_bf16(X_bits)
        Y = torch.zeros((M, 320), dtype=torch.bfloat16, device="cuda")
        Y8 = torch.zeros((M, 320), dtype=torch.bfloat16, device="cuda")
        B.osc_linear(w, X, Y, ws)
        B.osc_fp8_linear(w8, X, Y8, ws8)
        B.osc_sync_check()
        want, want8 = Y.clone(), Y8.clone()
        st = torch.cuda.Stream()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(st):
            with torch.cuda.graph(g, stream=st):
                B.osc_linear(w, X, Y, ws, stream=st)
                B.osc_fp8_linear(w8, X, Y8, ws8, stream=st)
        for _ in range(2):
            Y.zero_()
            Y8.zero_()
            g.replay()
            torch.cuda.synchronize()
            assert torch.equal(Y, want) and torch.equal(Y8, want8)
        B.osc_sync_check()
        outs[M] = want
    assert outs[24].shape[0] == 24


@pytest.mark.parametrize("M", [16, 64, 300, 1500])
def test_back_to_back_calls_on_a_stream_of_their_own(B, M):
    """Every kernel is launched as a programmatic dependent of the one in front; on a non-blocking stream of its own
    the launches really overlap.  A chain of calls that reuse one workspace and feed each other (the output of a
    linear is the input of the next) must give the bytes of the same calls with a synchronisation between them."""
    K = N = 512
    X_bits, W_bits, lut = make_case("rand2", M, N, K, 3)
    X = dev_bf16(X_bits)
    w = B.osc_prepare_weights(dev_bf16(W_bits), lut)
    w8 = B.osc_fp8_prepare_weights(dev_bf16(W_bits))
    ws = poison(max(B.osc_act_sizes(w, M).workspace_bytes, B.osc_fp8_act_sizes(w8, M).workspace_bytes))
    torch.cuda.synchronize()

    def chain(sync):
        a, b = (torch.zeros((M, N), dtype=torch.bfloat16, device="cuda") for _ in range(2))
        src = X
        for i in range(6):
            dst = a if i % 2 == 0 else b
            if i % 3 == 2:
                B.osc_fp8_linear(w8, src, dst, ws)
            else:
                B.osc_linear(w, src, dst, ws)
            if sync:
                torch.cuda.synchronize()
            src = dst
        torch.cuda.synchronize()
        return src.clone()
    want = chain(True)
    with torch.cuda.stream(torch.cuda.Stream()):
        got = chain(False)
    B.osc_sync_check()
    assert torch.isfinite(want.float()).all()
    assert torch.equal(got.view(torch.int16), want.view(torch.int16))


@pytest.mark.parametrize("kind", ["small", "mid"])
def test_grouped_gather_equals_grouped_on_permuted_rows(B, oracle, kind):
    """Dispatch fused behind the quantizer: tokens quantized once, quantized rows gathered per expert.  Must equal the
    grouped linear on X[row_token] byte for byte (same kernels on identical operands), and the oracle within tolerance."""
    counts = grouped_counts(kind)
    E, K, N, T = counts.size, 384, (320 if kind == "mid" else 192), 200
    c = synth.moe_gate_up_case(E, counts, K=K, N=N, seed=5)
    M = c["M"]
    rng = np.random.default_rng(11)
    Xtok, _ = synth.osc_activations_only(9, T, K, 1)
    row_token = rng.integers(0, T, size=M).astype(np.int32)
    row_token[:3] = [0, T - 1, 0]                      # repeated and extreme tokens
    Xperm = Xtok[row_token]
    w = B.osc_prepare_weights_grouped(dev_bf16(c["W"].reshape(E * N, K)).view(E, N, K), c["lut"])
    off = torch.from_numpy(c["off"]).cuda()
    sz = B.osc_act_sizes(w, M)
    ws_a = poison(sz.workspace_bytes)
    Ya = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_linear_grouped(w, dev_bf16(Xperm), off, Ya, ws_a)
    nbytes = B.osc_gather_workspace_bytes(w, T, M)
    assert nbytes > sz.workspace_bytes
    ws_b = poison(nbytes)
    Yb = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_linear_grouped_gather(w, dev_bf16(Xtok), torch.from_numpy(row_token).cuda(), off, Yb, ws_b)
    B.osc_sync_check()
    assert torch.equal(Ya.view(torch.int16), Yb.view(torch.int16))
    for o, n in ((sz.xq_offset, sz.xq_bytes), (sz.xo_offset, sz.xo_bytes)):
        assert torch.equal(ws_a[o:o + n], ws_b[o:o + n])
    # scale bytes: every block either side wrote (the blocks of the schedule's tiles) agrees; compare on the valid rows
    gq = oracle.quantize_extract_grouped(Xperm, c["off"], c["lut"])
    sfa, sfb = host_u8(ws_a)[sz.sfa_offset:], host_u8(ws_b)[sz.sfa_offset:]
    for e in range(E):
        if counts[e]:
            v = valid_sf_bytes(oracle, int(counts[e]), K, int(gq["sf_row_base"][e]))
            assert np.array_equal(sfa[v], sfb[v]) and np.array_equal(sfb[v], gq["sf"][v])
    Yh = host_f64(Yb)
    for e in range(E):
        r0, r1 = int(c["off"][e]), int(c["off"][e + 1])
        if r1 > r0:
            Yref, Tb, *_ = oracle.linear(Xperm[r0:r1], c["W"][e], c["lut"])
            assert_within_tolerance(Yh[r0:r1], Yref, Tb, f"gathered grouped expert {e}")
    # too small a workspace is refused before any launch
    with pytest.raises(B.OscError) as err:
        B.osc_linear_grouped_gather(w, dev_bf16(Xtok), torch.from_numpy(row_token).cuda(), off, Yb, ws_b[:sz.workspace_bytes])
    assert err.value.status == -5


@pytest.mark.parametrize("kind", ["small", "mid"])
def test_rmsnorm_grouped_gather(B, oracle, kind):
    """The dispatch-fused grouped linear behind an RMSNorm: equals the gather call on the separately normalized tokens
    bit for bit, and the oracle (RMSNorm, Algorithm 2, Eq. 5 per expert) within tolerance."""
    counts = grouped_counts(kind)
    E, K, N, T = counts.size, 512, (320 if kind == "mid" else 192), 150
    c = synth.moe_gate_up_case(E, counts, K=K, N=N, seed=6)
    M = c["M"]
    rng = np.random.default_rng(12)
    Hb, _ = synth.osc_activations_only(10, T, K, 1)
    gb = synth.f32_to_bf16_bits(rng.uniform(0.3, 2.0, K).astype(np.float32) * rng.choice([-1.0, 1.0], K).astype(np.float32))
    row_token = rng.integers(0, T, size=M).astype(np.int32)
    w = B.osc_prepare_weights_grouped(dev_bf16(c["W"].reshape(E * N, K)).view(E, N, K), c["lut"])
    off, rt = torch.from_numpy(c["off"]).cuda(), torch.from_numpy(row_token).cuda()
    nbytes = B.osc_gather_workspace_bytes(w, T, M)
    H, g = dev_bf16(Hb), dev_bf16(gb)
    Xn = torch.empty((T, K), dtype=torch.bfloat16, device="cuda")
    B.osc_rmsnorm(H, g, 1e-5, Xn)
    Ya = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_linear_grouped_gather(w, Xn, rt, off, Ya, poison(nbytes))
    Yb = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_rmsnorm_linear_grouped_gather(w, H, g, 1e-5, rt, off, Yb, poison(nbytes))
    B.osc_sync_check()
    assert torch.equal(Ya.view(torch.int16), Yb.view(torch.int16))
    Xperm = oracle.rmsnorm(Hb, gb, 1e-5)[row_token]
    Yh = host_f64(Yb)
    for e in range(E):
        r0, r1 = int(c["off"][e]), int(c["off"][e + 1])
        if r1 > r0:
            Yref, Tb, *_ = oracle.linear(Xperm[r0:r1], c["W"][e], c["lut"])
            assert_within_tolerance(Yh[r0:r1], Yref, Tb, f"rmsnorm + gathered grouped, expert {e}")
    with pytest.raises(B.OscError) as err:      # dense handle
        wd = B.osc_prepare_weights(dev_bf16(c["W"][0]), c["lut"])
        B.osc_rmsnorm_linear_grouped_gather(wd, H, g, 1e-5, rt, off, Yb, poison(nbytes))
    assert err.value.status == -1


@pytest.mark.parametrize("kind", ["small", "mid"])
def test_swiglu_fp8_grouped(B, oracle, kind):
    """Grouped FP8 down projection on the experts' gate|up rows: equals the grouped FP8 linear on the separately
    computed activation bit for bit, and the oracle (SwiGLU, per-token FP8, GEMM per expert) within tolerance."""
    counts = grouped_counts(kind)
    E, I, N = counts.size, 384, (320 if kind == "mid" else 128)
    d = synth.moe_down_case(E, counts, K=I, N=N, seed=7)
    M = d["M"]
    rng = np.random.default_rng(13)
    GUb = synth.f32_to_bf16_bits(rng.normal(0.0, 1.5, (M, 2 * I)).astype(np.float32))
    w = B.osc_fp8_prepare_weights_grouped(dev_bf16(d["W"].reshape(E * N, I)).view(E, N, I))
    off = torch.from_numpy(d["off"]).cuda()
    nbytes = B.osc_fp8_act_sizes(w, M).workspace_bytes
    GU = dev_bf16(GUb)
    Hh = torch.empty((M, I), dtype=torch.bfloat16, device="cuda")
    B.osc_swiglu(GU, I, Hh)
    Ya = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_fp8_linear_grouped(w, Hh, off, Ya, poison(nbytes))
    Yb = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_swiglu_fp8_linear_grouped(w, GU, off, Yb, poison(nbytes))
    B.osc_sync_check()
    assert torch.equal(Ya.view(torch.int16), Yb.view(torch.int16))
    hb = oracle.swiglu(GUb, I)
    Yh = host_f64(Yb)
    for e in range(E):
        r0, r1 = int(d["off"][e]), int(d["off"][e + 1])
        if r1 > r0:
            Yref, Tb, *_ = oracle.fp8_linear(hb[r0:r1], d["W"][e])
            assert_within_tolerance(Yh[r0:r1], Yref, Tb, f"swiglu + grouped fp8, expert {e}")
    with pytest.raises(B.OscError) as err:      # dense handle
        wd = B.osc_fp8_prepare_weights(dev_bf16(d["W"][0]))
        B.osc_swiglu_fp8_linear_grouped(wd, GU, off, Yb, poison(nbytes))
    assert err.value.status == -1
