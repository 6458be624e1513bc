"""Pins for the oracle's offline profiling (Eq. 1-4, Algorithm 1) and, on a GPU, bit-exact parity of
osc_profile_lut with it."""
import os

import numpy as np
import pytest

from paper_2604_12782_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def numpy_profile(Xf, alpha):
    """Independent restatement with library routines (np.argmax takes the first maximum, np.bincount + argmax
    the smallest most frequent index)."""
    S, H = Xf.shape
    A = np.abs(Xf)
    T = alpha * A.mean()
    g = A.reshape(S, H // 32, 32)
    jstar = g.argmax(-1)
    peak = np.take_along_axis(g, jstar[..., None], -1)[..., 0]
    L, nh, nt = [], [], []
    for k in range(H // 32):
        votes = jstar[peak[:, k] > T, k]
        cnt = np.bincount(votes, minlength=32)
        nt.append(int(cnt.sum()))
        nh.append(int(cnt.max()))
        L.append(int(cnt.argmax()) if cnt.sum() else -1)
    return T, np.array(L), np.array(nh), np.array(nt)


def test_worked_example(oracle):
    rows = [l.split() for l in open(os.path.join(GOLD, "profile_indexing_example.txt")) if l.strip() and l[0] != "#"]
    X = np.full((4, 64), 0.5, np.float32)
    exp = {}
    for r in rows:
        if r[0] == "entry":
            X[int(r[1]), int(r[2])] = float(r[3])
        else:
            exp[r[0]] = [float(v) for v in r[1:]]
    Xb = synth.f32_to_bf16_bits(X)
    T = oracle.threshold(Xb, exp["alpha"][0])
    assert T == exp["T"][0]
    L, nh, nt = oracle.profile_indexing(Xb, T)
    assert list(L) == exp["lut"] and list(nt) == exp["n_total"] and list(nh) == exp["n_hit"]
    c, mean = oracle.clustering_density(nh, nt)
    assert np.allclose(c, exp["density"]) and abs(mean - np.mean(exp["density"])) < 1e-15


def test_against_numpy_restatement(oracle):
    rng = np.random.default_rng(7)
    X = rng.standard_normal((96, 256)) * np.exp(rng.standard_normal((1, 256)))
    X[:, 40] *= 30
    X[rng.random(X.shape) < 0.01] *= 25
    X[:, 64:96] = 0.01 * rng.standard_normal((96, 32))          # a group that never exceeds the threshold
    Xb = synth.f32_to_bf16_bits(X.astype(np.float32))
    Xf = synth.bf16_bits_to_f64(Xb)
    for alpha in (5.0, 1.5):
        T = oracle.threshold(Xb, alpha)
        Tn, Ln, nhn, ntn = numpy_profile(Xf, alpha)
        assert abs(T - Tn) <= 1e-12 * Tn
        L, nh, nt = oracle.profile_indexing(Xb, T)
        assert np.array_equal(L, Ln) and np.array_equal(nh, nhn) and np.array_equal(nt, ntn)
    assert L[2] == -1 and nt[2] == 0


def test_threshold_bits(oracle):
    for T in (5.37109375, 1.0, 1.0000001, 0.99999, 3.0e-5, 123456.789):
        tb = oracle.threshold_bits(T)
        lo = synth.bf16_bits_to_f64(np.array([tb], np.uint16))[0]
        hi = synth.bf16_bits_to_f64(np.array([tb + 1], np.uint16))[0]
        assert lo <= T < hi
    assert oracle.threshold_bits(0.0) == 0


def test_planted_channels_are_recovered(oracle):
    Xb, lut = synth.osc_activations_only(3, 1536, 1024, 1)      # 3 x 512 calibration tokens, as in the paper's set-up
    T = oracle.threshold(Xb)
    L, nh, nt = oracle.profile_indexing(Xb, T)
    assert np.array_equal(L, lut[:, 0])
    c, mean = oracle.clustering_density(nh, nt)
    assert mean > 0.9                                            # persistent channels: high clustering density
    Xd = synth.fp8_linear_case(3, 1536, 1024, 8)["X"]           # diffuse heavy tails: low density, as at the W2 input
    Ld, nhd, ntd = oracle.profile_indexing(Xd, oracle.threshold(Xd))
    assert oracle.clustering_density(nhd, ntd)[1] < 0.35


@pytest.mark.gpu
@pytest.mark.parametrize("S,K,kind", [(1536, 4096, "planted"), (96, 256, "mixed"), (7, 128, "zeros"), (300, 1024, "diffuse")])
def test_gpu_profile_bit_exact(oracle, S, K, kind):
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from gpu_util import dev_bf16
    from paper_2604_12782_b200 import binding as B
    rng = np.random.default_rng(S + K)
    if kind == "planted":
        Xb, _ = synth.osc_activations_only(1, S, K, 1)
    elif kind == "diffuse":
        Xb = synth.fp8_linear_case(2, S, K, 8)["X"]
    elif kind == "zeros":
        Xb = np.zeros((S, K), np.uint16)
        Xb[3, 40] = 0x4000
    else:
        X = rng.standard_normal((S, K)) * np.exp(rng.standard_normal((1, K)))
        X[:, 64:96] = 0.001
        Xb = synth.f32_to_bf16_bits(X.astype(np.float32))
    alpha = 5.0
    X = dev_bf16(Xb)
    scratch = torch.full((B.osc_profile_scratch_bytes(K),), 0xFF, dtype=torch.uint8, device="cuda")
    lut = torch.full((K // 32,), 99, dtype=torch.int8, device="cuda")
    nh = torch.full((K // 32,), -7, dtype=torch.int32, device="cuda")
    nt = torch.full((K // 32,), -7, dtype=torch.int32, device="cuda")
    tb = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    B.osc_profile_lut(X, alpha, scratch, lut, nh, nt, tb)
    B.osc_sync_check()
    T = oracle.threshold(Xb, alpha)
    L, rh, rt = oracle.profile_indexing(Xb, T)
    assert int(tb.item()) == oracle.threshold_bits(T)
    assert np.array_equal(lut.cpu().numpy(), L)
    assert np.array_equal(nh.cpu().numpy(), rh) and np.array_equal(nt.cpu().numpy(), rt)
    if kind == "planted":
        # the table the profiler found drives the OSC path
        w = B.osc_prepare_weights(dev_bf16(np.zeros((64, K), np.uint16)), lut.cpu().numpy().reshape(-1, 1))
        assert w.K_o == K // 32
