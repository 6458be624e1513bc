"""Seeded random shapes through every linear entry point, against the oracle.

The fixed cases elsewhere pick their shapes by hand; here the shapes are drawn (M from one row to a few
thousand, K any multiple of 128 up to 2048, N any multiple of 64 up to 2048, tables with one to three
channels per group and any share of groups without one, output rows with a padded leading dimension), so
that every kernel the dispatcher can choose meets tails it was not written around.  Outputs within the
stated tolerance, and nothing written outside the [M, N] window of Y.
"""
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


def draw_rows(rng):
    r = rng.random()
    if r < 0.3:
        return int(rng.integers(1, 70))
    if r < 0.6:
        return int(rng.integers(70, 400))
    if r < 0.9:
        return int(rng.integers(400, 1500))
    return int(rng.integers(1500, 4000))


def draw_lut(rng, K, C, p_none):
    lut = np.full((K // 32, C), -1, np.int8)
    for k in range(K // 32):
        ch = rng.permutation(32)[:C]
        for c in range(C):
            if rng.random() > p_none:
                lut[k, c] = ch[c]
    return lut


def run_in_window(rng, M, N, call, Yref, T, what):
    """Y is a window of a larger buffer: rows above and below, columns to the right, stay as they were."""
    ldy = N + 8 * int(rng.integers(0, 3))
    big = torch.full((M + 2, ldy), 7.0, dtype=torch.bfloat16, device="cuda")
    Y = big[1:M + 1, :N]
    call(Y)
    assert_within_tolerance(host_f64(Y), Yref, T, what)
    guard = big.clone()
    guard[1:M + 1, :N] = 7.0
    assert (guard == 7.0).all(), f"{what}: wrote outside Y"


KINDS = ["osc", "osc", "fp8", "mxfp8", "nvfp4", "dyn"]


@pytest.mark.parametrize("seed", range(36))
def test_random_dense_shape(B, oracle, seed):
    rng = np.random.default_rng(1000 + seed)
    kind = KINDS[seed % len(KINDS)]
    M, K, N = draw_rows(rng), 128 * int(rng.integers(1, 17)), 64 * int(rng.integers(1, 33))
    cap = 1.5e9 if kind == "dyn" else 4e9           # keeps the oracle's part of a case under a second
    if M * N * K > cap:
        M = max(1, int(cap / (N * K)))
    what = f"{kind} M={M} N={N} K={K}"
    if kind == "osc":
        C = int(rng.integers(1, 4))
        c = synth.osc_linear_case(seed, M, K, N, 2)
        lut = draw_lut(rng, K, C, float(rng.choice([0.0, 0.3, 0.9, 1.0])))
        w = B.osc_prepare_weights(dev_bf16(c["W"]), lut)
        ws = poison(B.osc_act_sizes(w, M).workspace_bytes)
        X = dev_bf16(c["X"])
        Yref, T, *_ = oracle.linear(c["X"], c["W"], lut)
        run_in_window(rng, M, N, lambda Y: B.osc_linear(w, X, Y, ws), Yref, T, f"{what} C={C} K_o={w.K_o}")
    elif kind == "fp8":
        c = synth.fp8_linear_case(seed, M, K, N)
        w = B.osc_fp8_prepare_weights(dev_bf16(c["W"]))
        ws = poison(B.osc_fp8_act_sizes(w, M).workspace_bytes)
        X = dev_bf16(c["X"])
        Yref, T, *_ = oracle.fp8_linear(c["X"], c["W"])
        run_in_window(rng, M, N, lambda Y: B.osc_fp8_linear(w, X, Y, ws), Yref, T, what)
    elif kind == "mxfp8":
        c = synth.fp8_linear_case(seed, M, K, N)
        w = B.osc_mxfp8_prepare_weights(dev_bf16(c["W"]))
        ws = poison(B.osc_mxfp8_act_sizes(w, M).workspace_bytes)
        X = dev_bf16(c["X"])
        Yref, T, *_ = oracle.mxfp8_linear(c["X"], c["W"])
        run_in_window(rng, M, N, lambda Y: B.osc_mxfp8_linear(w, X, Y, ws), Yref, T, what)
    elif kind == "nvfp4":
        c = synth.osc16_linear_case(seed, M, K, N)
        ex, ew = synth.nvfp4_tensor_exponent(c["X"]), synth.nvfp4_tensor_exponent(c["W"])
        w = B.osc_nvfp4_prepare_weights(dev_bf16(c["W"]), c["lut16"], ew)
        ws = poison(B.osc_nvfp4_act_sizes(w, M).workspace_bytes)
        X = dev_bf16(c["X"])
        Yref, T, *_ = oracle.nvfp4_linear(c["X"], c["W"], c["lut16"], ex, ew)
        run_in_window(rng, M, N, lambda Y: B.osc_nvfp4_linear(w, X, ex, Y, ws), Yref, T, what)
    else:
        c = synth.osc_linear_case(seed, M, K, N, 2)
        w = B.osc_dyn_prepare_weights(dev_bf16(c["W"]))
        ws = poison(B.osc_dyn_act_sizes(w, M).workspace_bytes)
        X = dev_bf16(c["X"])
        Yref, T, *_ = oracle.dyn_linear(c["X"], c["W"])
        run_in_window(rng, M, N, lambda Y: B.osc_dyn_linear(w, X, Y, ws), Yref, T, what)
    B.osc_sync_check()


@pytest.mark.parametrize("seed", range(16))
def test_random_grouped_shape(B, oracle, seed):
    """Expert row counts drawn from {0, 1, under one tile, several tiles}: both tile schedules, experts that end
    anywhere inside a tile, runs of empty experts."""
    rng = np.random.default_rng(2000 + seed)
    E = int(rng.integers(1, 12))
    top = 700 if seed % 2 else 200
    counts = np.array([int(rng.choice([0, 1, int(rng.integers(1, 130)), int(rng.integers(130, top))])) for _ in range(E)])
    if counts.sum() == 0:
        counts[0] = 5
    K, N = 128 * int(rng.integers(1, 7)), 64 * int(rng.integers(1, 9))
    which = ["osc", "fp8", "mxfp8", "nvfp4"][seed % 4]
    what = f"grouped {which} counts={counts.tolist()} K={K} N={N}"
    if which == "osc":
        c = synth.moe_gate_up_case(E, counts, K=K, N=N, seed=seed)
        w = B.osc_prepare_weights_grouped(dev_bf16(c["W"].reshape(E * N, K)).view(E, N, K), c["lut"])
        ws = poison(B.osc_act_sizes(w, c["M"]).workspace_bytes)
        run = B.osc_linear_grouped

        def ref(x, wt):
            return oracle.linear(x, wt, c["lut"])[:2]
    elif which == "fp8":
        c = synth.moe_down_case(E, counts, K=K, N=N, seed=seed)
        w = B.osc_fp8_prepare_weights_grouped(dev_bf16(c["W"].reshape(E * N, K)).view(E, N, K))
        ws = poison(B.osc_fp8_act_sizes(w, c["M"]).workspace_bytes)
        run = B.osc_fp8_linear_grouped

        def ref(x, wt):
            return oracle.fp8_linear(x, wt)[:2]
    elif which == "nvfp4":
        c = synth.moe_gate_up_case(E, counts, K=K, N=N, seed=seed)
        lut16 = np.stack([rng.permutation(16)[:1] for _ in range(K // 16)]).astype(np.int8)
        ex, ew = synth.nvfp4_tensor_exponent(c["X"]), synth.nvfp4_tensor_exponent(c["W"])
        w = B.osc_nvfp4_prepare_weights_grouped(dev_bf16(c["W"].reshape(E * N, K)).view(E, N, K), lut16, ew)
        ws = poison(B.osc_nvfp4_act_sizes(w, c["M"]).workspace_bytes)

        def run(w_, X_, off_, Y_, ws_):
            B.osc_nvfp4_linear_grouped(w_, X_, off_, ex, Y_, ws_)

        def ref(x, wt):
            return oracle.nvfp4_linear(x, wt, lut16, ex, ew)[:2]
    else:
        c = synth.moe_down_case(E, counts, K=K, N=N, seed=seed)
        w = B.osc_mxfp8_prepare_weights_grouped(dev_bf16(c["W"].reshape(E * N, K)).view(E, N, K))
        ws = poison(B.osc_mxfp8_act_sizes(w, c["M"]).workspace_bytes)
        run = B.osc_mxfp8_linear_grouped

        def ref(x, wt):
            return oracle.mxfp8_linear(x, wt)[:2]
    M = c["M"]
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    run(w, dev_bf16(c["X"]), torch.from_numpy(c["off"]).cuda(), Y, ws)
    B.osc_sync_check()
    Yh = host_f64(Y)
    for e in range(E):
        r0, r1 = int(c["off"][e]), int(c["off"][e + 1])
        if r1 > r0:
            Yref, T = ref(c["X"][r0:r1], c["W"][e])
            assert_within_tolerance(Yh[r0:r1], Yref, T, f"{what}, expert {e}")
