"""Seeded inputs of the producer tests (RMSNorm rows, gate|up rows), shared by the CPU pins and the GPU parity tests
so that both look at the same values.  Numbers only: no arithmetic of the method."""
import numpy as np

from paper_2604_12782_b200 import synth


def residual_rows(rng, M, K):
    """Residual-stream-like rows: heavy-tailed values, per-row magnitudes over several orders, a few channels
    that are large in every row, plus rows of extreme scale."""
    H = rng.standard_t(4, size=(M, K)) * rng.lognormal(0.0, 1.5, size=(M, 1))
    hot = rng.choice(K, size=max(1, K // 64), replace=False)
    H[:, hot] *= 25.0
    if M > 4:
        H[1] *= 1e-18
        H[2] *= 1e15
        H[3, : K // 2] = 0.0
    return synth.f32_to_bf16_bits(H.astype(np.float32))


def gamma_bits(rng, K):
    return synth.f32_to_bf16_bits(rng.uniform(0.1, 3.0, K).astype(np.float32) * rng.choice([-1.0, 1.0], K).astype(np.float32))


def gate_up(rng, M, I, pad=0):
    """Gate/up projection outputs: gates over the whole range where silu bends, saturates or vanishes, a few extreme
    rows, zeros; `pad` extra columns behind the up half."""
    g = rng.standard_normal((M, I)) * rng.choice([0.3, 3.0, 30.0], size=(M, 1))
    u = rng.standard_t(4, size=(M, I)) * rng.lognormal(0.0, 1.0, size=(M, 1))
    if M > 4:
        g[1] = rng.uniform(-120.0, 120.0, I)     # both clamps of exp32
        g[2, : I // 2] = 0.0
        u[3] *= 1e-30
    GU = np.concatenate([g, u, np.full((M, pad), 7.0)], axis=1)
    return synth.f32_to_bf16_bits(GU.astype(np.float32))


RMSNORM_ROW_CASES = [(1, 128, 1e-6), (37, 384, 1e-5), (130, 1024, 1e-6), (64, 4096, 1e-6),
                     (9, 8192, 1e-6), (5, 4096 + 128, 0.0), (300, 2048, 1e-6)]
SWIGLU_ROW_CASES = [(1, 128), (37, 384), (130, 1024), (20, 12288), (5, 16384), (64, 768)]
