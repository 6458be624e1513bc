"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

Every (M, K, N) the benchmark configurations name goes through the public call with the library's own kernel
routing (no environment override), so the kernel that is timed for a shape is the kernel that is checked:
  QKV 4096 -> 6144 (two protected channels per group) at M = 16, 128, 2048, 8192 and, as part of a decoder
  layer, 4096;  gate_up 4096 -> 24576 (one channel per group) at M = 128, 2048, 8192 and 4096;  o_proj
  4096 -> 4096 at M = 4096;  the down projection 12288 -> 4096 through the FP8 fallback at M = 128, 2048,
  8192 and 4096;  the grouped (MoE) pair with the Zipf expert load.

The quantizer outputs (codes, scale bytes, gathered channels, FP8 codes and scales) are compared in
full, bit for bit.  GEMM outputs are compared on sampled rows (all N columns of each) that include
every kind of tile position: first/last rows of 128- and 256-row tiles, the last row, and for the
grouped case the first and last row of several experts.
"""
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


def sample_rows(M, n=40, seed=0):
    if M <= 64:
        return np.arange(M, dtype=np.int32)
    edge = [0, 1, 127, 128, 129, 255, 256, 257, M - 257, M - 256, M - 129, M - 128, M - 1]
    rng = np.random.default_rng(seed)
    rows = sorted(set(int(r) for r in edge if 0 <= r < M) | set(int(r) for r in rng.integers(0, M, size=n)))
    return np.array(rows, np.int32)


OSC_SHAPES = ([("qkv", M, 6144, 2) for M in (16, 128, 2048, 4096, 8192)] +
              [("gate_up", M, 24576, 1) for M in (128, 2048, 4096, 8192)] +
              [("o_proj", 4096, 4096, 1)])


@pytest.mark.parametrize("name,M,N,cpg", OSC_SHAPES, ids=[f"{n}-M{m}" for n, m, _, _ in OSC_SHAPES])
def test_osc_linear_full_size(B, oracle, name, M, N, cpg):
    K = 4096
    c = synth.osc_linear_case(0, M, K, N, cpg)
    w = B.osc_prepare_weights(dev_bf16(c["W"]), c["lut"])
    sz = B.osc_act_sizes(w, M)
    ws = poison(sz.workspace_bytes)
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    before = ws.clone()
    B.osc_linear(w, dev_bf16(c["X"]), Y, ws)
    B.osc_sync_check()
    if torch.equal(ws, before):
        # sixteen rows or fewer: the few-row kernel quantized its activations itself and left the workspace alone;
        # Algorithm 2's outputs at this shape then come from the stand-alone call, the product from both routes
        assert M <= 16
        B.osc_quantize_extract(w, dev_bf16(c["X"]), ws[sz.xq_offset:], ws[sz.sfa_offset:], ws[sz.xo_offset:])
        Y2 = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        B.osc_gemm_dual(w, ws[sz.xq_offset:], ws[sz.sfa_offset:], ws[sz.xo_offset:], M, Y2)
        B.osc_sync_check()
        assert torch.equal(Y.view(torch.int16), Y2.view(torch.int16))
    else:
        assert M > 16
    # Algorithm 2 outputs: everything, bit for bit
    act = oracle.quantize_extract(c["X"], c["lut"])
    ws_h = host_u8(ws)
    assert np.array_equal(ws_h[sz.xq_offset:sz.xq_offset + sz.xq_bytes].reshape(M, K // 2), act["xq"])
    assert np.array_equal(ws_h[sz.sfa_offset:sz.sfa_offset + sz.sfa_bytes], act["sf"])
    assert np.array_equal(ws_h[sz.xo_offset:sz.xo_offset + sz.xo_bytes].view(np.uint16).reshape(M, -1), act["xo"])
    # weight split: everything, bit for bit
    wts = oracle.prepare_weights(c["W"], c["lut"])
    assert np.array_equal(host_u8(w.keep["wq"])[:w.sizes.wq_bytes].reshape(N, K // 2), wts["xq"])
    assert np.array_equal(host_u8(w.keep["sfw"])[:w.sizes.sfw_bytes], wts["sf"])
    assert np.array_equal(host_u8(w.keep["wo"])[:w.sizes.wo_bytes].view(np.uint16).reshape(N, -1), wts["xo"])
    # Eq. 5 on sampled rows
    rows = sample_rows(M)
    Yref, T = oracle.gemm_dual(act, wts, rows)
    Yh = host_f64(Y[torch.from_numpy(rows.astype(np.int64)).cuda()])
    assert_within_tolerance(Yh, Yref, T, f"{name} M={M}")
    assert not torch.isnan(Y.float()).any()


@pytest.mark.parametrize("M", [128, 2048, 4096, 8192])
def test_fp8_down_projection_full_size(B, oracle, M):
    K, N = 12288, 4096
    c = synth.fp8_linear_case(0, M, K, N)
    w = B.osc_fp8_prepare_weights(dev_bf16(c["W"]))
    sz = B.osc_fp8_act_sizes(w, M)
    ws = poison(sz.workspace_bytes)
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_fp8_linear(w, dev_bf16(c["X"]), Y, ws)
    B.osc_sync_check()
    x8, sx = oracle.fp8_quantize(c["X"])
    w8, sw = oracle.fp8_quantize(c["W"])
    ws_h = host_u8(ws)
    assert np.array_equal(ws_h[sz.x8_offset:sz.x8_offset + M * K].reshape(M, K), x8)
    assert np.array_equal(ws_h[sz.sx_offset:sz.sx_offset + 4 * M].view(np.uint32), sx.view(np.uint32))
    assert np.array_equal(host_u8(w.keep["w8"])[:N * K].reshape(N, K), w8)
    rows = sample_rows(M)
    Yref, T = oracle.fp8_gemm(x8, sx, w8, sw, rows)
    assert_within_tolerance(host_f64(Y[torch.from_numpy(rows.astype(np.int64)).cuda()]), Yref, T, f"down fp8 M={M}")
    assert not torch.isnan(Y.float()).any()


def moe_sample_rows(off, per_expert_edges=12, n_random=24):
    E = off.size - 1
    rows = []
    big = np.argsort(-(off[1:] - off[:-1]))
    for e in list(big[:4]) + list(big[-4:]) + [0, E - 1, E // 2, E // 3]:
        r0, r1 = int(off[e]), int(off[e + 1])
        if r1 > r0:
            rows += [r0, r1 - 1, min(r0 + 127, r1 - 1), min(r0 + 128, r1 - 1)]
    rng = np.random.default_rng(1)
    rows += [int(r) for r in rng.integers(0, int(off[-1]), size=n_random)]
    return np.array(sorted(set(rows)), np.int32)


def test_moe_grouped_full_size(B, oracle):
    counts = synth.zipf_expert_rows()
    E = counts.size
    off_h = synth.offsets_from_counts(counts)
    off = torch.from_numpy(off_h).cuda()
    # gate_up through the OSC path: one table for all experts
    c = synth.moe_gate_up_case(E, counts, weight_pool=4)
    M, K, N = c["M"], c["K"], c["N"]
    w = B.osc_prepare_weights_grouped(dev_bf16(c["W"].reshape(E * N, K)).view(E, N, K), c["lut"])
    sz = B.osc_act_sizes(w, M)
    ws = poison(sz.workspace_bytes)
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_linear_grouped(w, dev_bf16(c["X"]), off, Y, ws)
    B.osc_sync_check()
    gq = oracle.quantize_extract_grouped(c["X"], off_h, c["lut"])
    ws_h = host_u8(ws)
    assert np.array_equal(ws_h[sz.xq_offset:sz.xq_offset + sz.xq_bytes].reshape(M, K // 2), gq["xq"])
    assert np.array_equal(ws_h[sz.xo_offset:sz.xo_offset + sz.xo_bytes].view(np.uint16).reshape(M, -1), gq["xo"])
    sf_h = ws_h[sz.sfa_offset:sz.sfa_offset + gq["sf"].size]
    for e in (0, 1, E // 2, E - 1):
        v = valid_sf_bytes(oracle, int(counts[e]), K, int(gq["sf_row_base"][e]))
        assert np.array_equal(sf_h[v], gq["sf"][v]), f"scales of expert {e}"
    rows = moe_sample_rows(off_h)
    Yh = host_f64(Y[torch.from_numpy(rows.astype(np.int64)).cuda()])
    expert_of = np.searchsorted(off_h, rows, side="right") - 1
    prepared = {}
    for i, (r, e) in enumerate(zip(rows, expert_of)):
        key = int(e) % 4                       # weight_pool = 4 distinct matrices
        if key not in prepared:
            prepared[key] = oracle.prepare_weights(c["W"][int(e)], c["lut"])
        sfr = int(gq["sf_row_base"][e]) + int(r) - int(off_h[e])
        Yref, T = oracle.gemm_dual({"xq": gq["xq"], "sf": gq["sf"], "xo": gq["xo"]}, prepared[key],
                                   np.array([r], np.int32), np.array([sfr], np.int32))
        assert_within_tolerance(Yh[i:i + 1], Yref, T, f"moe gate_up row {r} expert {e}")
    assert not torch.isnan(Y.float()).any()

    # down projection through the FP8 fallback
    d = synth.moe_down_case(E, counts, weight_pool=4)
    K2, N2 = d["K"], d["N"]
    w2 = B.osc_fp8_prepare_weights_grouped(dev_bf16(d["W"].reshape(E * N2, K2)).view(E, N2, K2))
    sz2 = B.osc_fp8_act_sizes(w2, M)
    ws2 = poison(sz2.workspace_bytes)
    Y2 = torch.full((M, N2), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_fp8_linear_grouped(w2, dev_bf16(d["X"]), off, Y2, ws2)
    B.osc_sync_check()
    x8, sx = oracle.fp8_quantize(d["X"])
    assert np.array_equal(host_u8(ws2)[sz2.x8_offset:sz2.x8_offset + M * K2].reshape(M, K2), x8)
    Y2h = host_f64(Y2[torch.from_numpy(rows.astype(np.int64)).cuda()])
    q = {}
    for i, (r, e) in enumerate(zip(rows, expert_of)):
        key = int(e) % 4
        if key not in q:
            q[key] = oracle.fp8_quantize(d["W"][int(e)])
        Yref, T = oracle.fp8_gemm(x8, sx, q[key][0], q[key][1], np.array([r], np.int32))
        assert_within_tolerance(Y2h[i:i + 1], Yref, T, f"moe down row {r} expert {e}")
    assert not torch.isnan(Y2.float()).any()


# ---- more than 2^31 elements in one activation matrix --------------------------------------------------------

BIG_K = 4096
BIG_M = (1 << 19) + 77            # M * K = 2^31 + 315392 elements; the FP8 code matrix alone exceeds 2^31 bytes
BIG_BASE = 5000                   # distinct rows, repeated: 2^31 / K = 524288 is not a multiple of 5000, so a row
                                  # offset that wrapped at 32 bits would land on a different base row


def big_rows():
    wrap = (1 << 31) // BIG_K
    edge = [0, 127, 128, BIG_BASE - 1, BIG_BASE, wrap - 1, wrap, wrap + 1, BIG_M - 78, BIG_M - 77, BIG_M - 1]
    rng = np.random.default_rng(7)
    return np.array(sorted(set(edge) | set(int(r) for r in rng.integers(0, BIG_M, size=28))), np.int64)


def sf_positions(rows, K):
    r = np.asarray(rows)[:, None]
    g = np.arange(K // 32)[None, :]
    return ((r // 128) * (K // 128) + g // 4) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + (g % 4)


def repeated_rows(base_bits):
    Xb = dev_bf16(base_bits)
    return Xb.repeat((BIG_M + BIG_BASE - 1) // BIG_BASE, 1)[:BIG_M]


@pytest.mark.parametrize("which", ["osc", "fp8", "mxfp8"])
def test_more_than_2_31_elements(B, oracle, which):
    """Row offsets are 64-bit everywhere: sampled rows on both sides of the 2^31-element mark, and the ragged
    last tile, match the oracle (quantizer outputs bit for bit, GEMM rows within the tolerance)."""
    K, N, M = BIG_K, 128, BIG_M
    rows = big_rows()
    src = rows % BIG_BASE
    rows_d = torch.from_numpy(rows).cuda()
    local = np.arange(rows.size)
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    if which == "osc":
        c = synth.osc_linear_case(3, BIG_BASE, K, N, 2)
        X = repeated_rows(c["X"])
        w = B.osc_prepare_weights(dev_bf16(c["W"]), c["lut"])
        sz = B.osc_act_sizes(w, M)
        ws = poison(sz.workspace_bytes)
        B.osc_linear(w, X, Y, ws)
        B.osc_sync_check()
        act = oracle.quantize_extract(c["X"][src], c["lut"])
        xq = ws[sz.xq_offset:sz.xq_offset + sz.xq_bytes].view(M, K // 2)[rows_d]
        assert np.array_equal(host_u8(xq), act["xq"])
        xo = ws[sz.xo_offset:sz.xo_offset + sz.xo_bytes].view(torch.int16).view(M, -1)[rows_d]
        assert np.array_equal(host_u8(xo).view(np.uint16), act["xo"])
        sf = ws[sz.sfa_offset:sz.sfa_offset + sz.sfa_bytes][torch.from_numpy(sf_positions(rows, K)).cuda()]
        assert np.array_equal(host_u8(sf), act["sf"][sf_positions(local, K)])
        Yref, T, *_ = oracle.linear(c["X"][src], c["W"], c["lut"])
    elif which == "fp8":
        c = synth.fp8_linear_case(3, BIG_BASE, K, N)
        X = repeated_rows(c["X"])
        w = B.osc_fp8_prepare_weights(dev_bf16(c["W"]))
        sz = B.osc_fp8_act_sizes(w, M)
        ws = poison(sz.workspace_bytes)
        B.osc_fp8_linear(w, X, Y, ws)
        B.osc_sync_check()
        Yref, T, (x8, sx), _ = oracle.fp8_linear(c["X"][src], c["W"])
        got8 = ws[sz.x8_offset:sz.x8_offset + M * K].view(M, K)[rows_d]
        assert np.array_equal(host_u8(got8), x8)
        gots = ws[sz.sx_offset:sz.sx_offset + 4 * M].view(torch.int32)[rows_d]
        assert np.array_equal(host_u8(gots).view(np.uint32), sx.view(np.uint32))
    else:
        c = synth.fp8_linear_case(4, BIG_BASE, K, N)
        X = repeated_rows(c["X"])
        w = B.osc_mxfp8_prepare_weights(dev_bf16(c["W"]))
        sz = B.osc_mxfp8_act_sizes(w, M)
        ws = poison(sz.workspace_bytes)
        B.osc_mxfp8_linear(w, X, Y, ws)
        B.osc_sync_check()
        Yref, T, (x8, sfa), _ = oracle.mxfp8_linear(c["X"][src], c["W"])
        got8 = ws[sz.x8_offset:sz.x8_offset + M * K].view(M, K)[rows_d]
        assert np.array_equal(host_u8(got8), x8)
        sf = ws[sz.sfa_offset:sz.sfa_offset + sz.sfa_bytes][torch.from_numpy(sf_positions(rows, K)).cuda()]
        assert np.array_equal(host_u8(sf), sfa[sf_positions(local, K)])
    assert_within_tolerance(host_f64(Y[rows_d]), Yref, T, f"{which} M={M}")
    assert not torch.isnan(Y.float()).any()


@pytest.mark.parametrize("which", ["rmsnorm", "swiglu"])
def test_more_than_2_31_elements_behind_a_producer(B, oracle, which):
    """The same for the quantizers fused into their producers (the residual stream, the gate|up matrix)."""
    M, N = BIG_M, 128
    rows = big_rows()
    src = rows % BIG_BASE
    rows_d = torch.from_numpy(rows).cuda()
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    rng = np.random.default_rng(11)
    if which == "rmsnorm":
        K = BIG_K
        c = synth.osc_linear_case(5, BIG_BASE, K, N, 2)
        gb = synth.f32_to_bf16_bits(rng.uniform(0.5, 2.0, K).astype(np.float32))
        w = B.osc_prepare_weights(dev_bf16(c["W"]), c["lut"])
        ws = poison(B.osc_act_sizes(w, M).workspace_bytes)
        B.osc_rmsnorm_linear(w, repeated_rows(c["X"]), dev_bf16(gb), 1e-6, Y, ws)
        B.osc_sync_check()
        Yref, T, *_ = oracle.linear(oracle.rmsnorm(c["X"][src], gb, 1e-6), c["W"], c["lut"])
    else:
        I = BIG_K // 2                                 # gate|up rows of 4096 columns
        GUb = synth.f32_to_bf16_bits(rng.normal(0.0, 1.5, (BIG_BASE, 2 * I)).astype(np.float32))
        W = synth.fp8_linear_case(3, 1, I, N)["W"]
        w = B.osc_fp8_prepare_weights(dev_bf16(W))
        ws = poison(B.osc_fp8_act_sizes(w, M).workspace_bytes)
        B.osc_swiglu_fp8_linear(w, repeated_rows(GUb), Y, ws)
        B.osc_sync_check()
        Yref, T, *_ = oracle.fp8_linear(oracle.swiglu(GUb[src], I), W)
    assert_within_tolerance(host_f64(Y[rows_d]), Yref, T, f"{which} M={M}")
    assert not torch.isnan(Y.float()).any()
