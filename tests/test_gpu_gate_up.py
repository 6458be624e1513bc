"""The SwiGLU applied in the epilogue of the gate|up projection (Section 3.3: the operator sits where its input is
produced).  H = silu(gate) * up comes out of the GEMM itself; checked
  - against the oracle: its linear (Algorithm 2 + Eq. 5) followed by its SwiGLU.  The GEMM is compared within a
    tolerance, not bit for bit, so the bound on h is that tolerance pushed through h = silu(g) * u: with
    |silu'(g)| <= 1.1 and |silu(g)| <= |g|,  |dh| <= 1.1 |u| dg + |g| du (+ the bf16 roundings of g, u and h, which
    the 2^-7 relative part of dg, du covers with room to spare: 2^-9 each);
  - against the library's own unfused path: osc_swiglu on osc_linear's output for the same handle, bit for bit
    (same kernel family, same operands, same accumulation order, same activation arithmetic)."""
import numpy as np
import pytest
import torch

from paper_2604_12782_b200 import synth

pytestmark = pytest.mark.gpu

from gpu_util import dev_bf16, host_bf16_bits, host_f64, poison  # noqa: E402


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_12782_b200 import binding
    return binding


def h_bound(Yref, T, I):
    g, u = Yref[:, :I], Yref[:, I:]
    dg = 2.0 ** -7 * np.abs(g) + 1e-3 * T[:, :I]
    du = 2.0 ** -7 * np.abs(u) + 1e-3 * T[:, I:]
    with np.errstate(over="ignore"):
        href = g / (1.0 + np.exp(-g)) * u
    return href, 1.1 * np.abs(u) * dg + np.abs(g) * du + 1.1 * dg * du + 2.0 ** -7 * np.abs(href) + 1e-30


# rows x K x I x channels per group: the pair kernel's gate|up form (more than 256 rows; a ragged last feature tile
# when I is not a multiple of 120; a ragged last row tile), and the small-M route through a scratch Y
CASES = [(300, 256, 128, 1), (513, 512, 320, 2), (1000, 384, 896, 1), (257, 128, 64, 0), (2048, 1024, 1536, 1),
         (16, 512, 256, 1), (200, 256, 192, 2)]


@pytest.mark.parametrize("M,K,I,cpg", CASES)
def test_linear_swiglu(B, oracle, M, K, I, cpg):
    c = synth.osc_linear_case(M + I, M, K, 2 * I, max(cpg, 1))
    lut = c["lut"] if cpg else np.full((K // 32, 1), -1, np.int8)
    # weights large enough that the gates leave the linear range of silu
    Wb = synth.f32_to_bf16_bits((synth.bf16_bits_to_f64(c["W"]) * 4.0).astype(np.float32))
    w = B.osc_prepare_weights_gate_up(dev_bf16(Wb), lut)
    X = dev_bf16(c["X"])
    ws = poison(B.osc_linear_swiglu_workspace_bytes(w, M))
    big = torch.full((M + 2, I + 8), 7.0, dtype=torch.bfloat16, device="cuda")
    H = big[1:M + 1, :I]
    B.osc_linear_swiglu(w, X, H, ws)
    B.osc_sync_check()
    guard = big.clone()
    guard[1:M + 1, :I] = 7.0
    assert (guard == 7.0).all(), "wrote outside H"
    # the library's own unfused path on the same handle (the stand-alone activation wants I to be a multiple of 128)
    if I % 128 == 0:
        sz = B.osc_act_sizes(w, M)
        Y = torch.full((M, 2 * I), float("nan"), dtype=torch.bfloat16, device="cuda")
        B.osc_linear(w, X, Y, poison(sz.workspace_bytes))
        H2 = torch.full((M, I), float("nan"), dtype=torch.bfloat16, device="cuda")
        B.osc_swiglu(Y, I, H2)
        B.osc_sync_check()
        got, two = host_bf16_bits(H.contiguous()), host_bf16_bits(H2)
        assert np.array_equal(got, two), f"{np.count_nonzero(got != two)} of {got.size} elements differ from the unfused path"
    # the oracle
    Yref, T, *_ = oracle.linear(c["X"], Wb, lut)
    href, bound = h_bound(Yref, T, I)
    err = np.abs(host_f64(H) - href)
    assert (err <= bound).all(), f"worst err/bound {np.max(err / bound):.3f}"
    assert not torch.isnan(H.float()).any()


def test_rmsnorm_linear_swiglu_and_errors(B, oracle):
    from producer_inputs import gamma_bits, residual_rows
    M, K, I = 700, 512, 384
    rng = np.random.default_rng(3)
    Hb, gb = residual_rows(rng, M, K), gamma_bits(rng, K)
    c = synth.osc_linear_case(9, 1, K, 2 * I, 1)
    Wb = synth.f32_to_bf16_bits((synth.bf16_bits_to_f64(c["W"]) * 4.0).astype(np.float32))
    w = B.osc_prepare_weights_gate_up(dev_bf16(Wb), c["lut"])
    ws = poison(B.osc_linear_swiglu_workspace_bytes(w, M))
    H = torch.full((M, I), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_rmsnorm_linear_swiglu(w, dev_bf16(Hb), dev_bf16(gb), 1e-6, H, ws)
    B.osc_sync_check()
    Yref, T, *_ = oracle.linear(oracle.rmsnorm(Hb, gb, 1e-6), Wb, c["lut"])
    href, bound = h_bound(Yref, T, I)
    assert (np.abs(host_f64(H) - href) <= bound).all()
    B.osc_linear_swiglu(w, dev_bf16(Hb)[:0], H[:0], ws)                       # M == 0: a no-op
    plain = B.osc_prepare_weights(dev_bf16(Wb), c["lut"])
    with pytest.raises(B.OscError) as e:                                     # a plain handle has no gate|up scale copy
        B.osc_linear_swiglu(plain, dev_bf16(Hb), H, ws)
    assert e.value.status == -1
    with pytest.raises(B.OscError) as e:
        B.osc_linear_swiglu(w, dev_bf16(Hb), H, ws[:64])
    assert e.value.status == -5


# experts: large ones (the pair kernel's gate|up form: experts that end inside a 256-row tile, inside a 16-row store pass,
# empty and one-row experts) and small ones (the route through a scratch Y)
@pytest.mark.parametrize("counts,mode", [([300, 0, 5, 256, 129, 511, 1, 385], "perm"), ([700, 64, 0, 900], "perm"),
                                         ([3, 0, 130, 1, 257, 128], "gather"), ([17, 40, 3, 0, 25], "perm"),
                                         ([300, 0, 5, 256, 129, 511, 1, 385], "norm_gather")])
def test_linear_swiglu_grouped(B, oracle, counts, mode):
    """Grouped (MoE) gate|up projection with the SwiGLU in the epilogue: per expert the dense call on that expert's rows
    and weights (bit for bit where both take the CTA-pair kernel), nothing written outside H, and within the
    pushed-through tolerance of the oracle."""
    from producer_inputs import gamma_bits
    counts = np.array(counts)
    E, K, I = counts.size, 384, 256
    M = int(counts.sum())
    off_h = synth.offsets_from_counts(counts)
    off = torch.from_numpy(off_h).cuda()
    rng = np.random.default_rng(E + M)
    T = max(1, M // 3)
    c = synth.osc_linear_case(70 + E, T if mode != "perm" else M, K, 64, 1)
    Wb = synth.f32_to_bf16_bits((0.08 * rng.standard_normal((E, 2 * I, K))).astype(np.float32))
    gb = gamma_bits(rng, K)
    w = B.osc_prepare_weights_gate_up_grouped(dev_bf16(Wb.reshape(E * 2 * I, K)).view(E, 2 * I, K), c["lut"])
    big = torch.full((M + 2, I + 8), 7.0, dtype=torch.bfloat16, device="cuda")
    H = big[1:M + 1, :I]
    if mode == "perm":
        Xp = c["X"]
        ws = poison(B.osc_linear_swiglu_workspace_bytes(w, M))
        B.osc_linear_swiglu_grouped(w, dev_bf16(Xp), off, H, ws)
    else:
        row_token_h = rng.integers(0, T, size=M).astype(np.int32)
        src = oracle.rmsnorm(c["X"], gb, 1e-6) if mode == "norm_gather" else c["X"]
        Xp = np.ascontiguousarray(src[row_token_h])
        ws = poison(B.osc_swiglu_gather_workspace_bytes(w, T, M))
        row_token = torch.from_numpy(row_token_h).cuda()
        if mode == "norm_gather":
            B.osc_rmsnorm_linear_swiglu_grouped_gather(w, dev_bf16(c["X"]), dev_bf16(gb), 1e-6, row_token, off, H, ws)
        else:
            B.osc_linear_swiglu_grouped_gather(w, dev_bf16(c["X"]), row_token, off, H, ws)
    B.osc_sync_check()
    guard = big.clone()
    guard[1:M + 1, :I] = 7.0
    assert (guard == 7.0).all(), "wrote outside H"
    got = host_bf16_bits(H.contiguous())
    Hf = host_f64(H)
    for e in range(E):
        r0, r1 = int(off_h[e]), int(off_h[e + 1])
        if r1 == r0:
            continue
        Yref, T_, *_ = oracle.linear(Xp[r0:r1], Wb[e], c["lut"])
        href, bound = h_bound(Yref, T_, I)
        err = np.abs(Hf[r0:r1] - href)
        assert (err <= bound).all(), f"expert {e}: worst err/bound {np.max(err / bound):.3f}"
        # the dense fused call on the expert's own rows and weights
        wd = B.osc_prepare_weights_gate_up(dev_bf16(Wb[e]), c["lut"])
        Hd = torch.full((r1 - r0, I), float("nan"), dtype=torch.bfloat16, device="cuda")
        B.osc_linear_swiglu(wd, dev_bf16(Xp[r0:r1]), Hd, poison(B.osc_linear_swiglu_workspace_bytes(wd, r1 - r0)))
        B.osc_sync_check()
        if r1 - r0 > 256 and M >= 96 * E:   # both on the CTA-pair kernel's gate|up form: the same accumulation order
            assert np.array_equal(got[r0:r1], host_bf16_bits(Hd)), f"expert {e} differs from the dense call"
        else:                               # another kernel for the dense call: equal up to the rounding of the fp32 sums
            assert (np.abs(Hf[r0:r1] - host_f64(Hd)) <= 2.0 * bound).all()
    assert not torch.isnan(H.float()).any()
