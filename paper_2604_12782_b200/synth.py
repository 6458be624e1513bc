"""Seeded synthetic inputs for the OSC dual-path linear layer.

This module only draws random numbers and formats them as bf16 bit patterns.
It contains none of the method's arithmetic (no quantizer, no lookup-table
processing, no GEMM): the CPU oracle and the CUDA path both receive the byte
buffers produced here, so neither has to re-implement the generator.

The shapes and value distributions stand in for the activations the paper
profiles at the four monitored positions of Qwen3-8B / Qwen3-30B-A3B
(Section 2.1): "vertical stripe" outliers that sit in fixed channels of each
32-channel group for most tokens (Fig. 2, Table 1: 60-80 % density at the
attention / FFN-up inputs) and diffuse heavy-tailed activations at the
down-projection input (Table 1: 20-35 %).  The real activations, weights and
calibration text are not available; these recipes replace them.

All arrays are numpy.  bf16 tensors are returned as uint16 bit patterns
(round-to-nearest-even from float32).
"""
from __future__ import annotations

import numpy as np

G = 32  # micro-scaling group size of MXFP4 (Section 3.2, "G = 32")


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit pattern (uint16), round-to-nearest-even."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    """bf16 bit pattern (uint16) -> float64 (exact)."""
    u = np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def _bf16(a: np.ndarray) -> np.ndarray:
    return f32_to_bf16_bits(a.astype(np.float32))


def lut_from_channels(ch: np.ndarray) -> np.ndarray:
    """[Kg, C] local channel indices -> int8 lookup table (the boundary's format)."""
    ch = np.asarray(ch)
    if ch.ndim == 1:
        ch = ch[:, None]
    return np.ascontiguousarray(ch.astype(np.int8))


def tiny_case(seed: int = 0, M: int = 64, K: int = 512, N: int = 512):
    """Single small OSC linear: one fixed channel per 32-group scaled x50 on every token."""
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((M, K))
    ch = rng.integers(0, G, size=K // G)
    X[:, np.arange(K // G) * G + ch] *= 50.0
    W = 0.02 * rng.standard_normal((N, K))
    return {"X": _bf16(X), "W": _bf16(W), "lut": lut_from_channels(ch), "M": M, "K": K, "N": N}


def planted_activations(rng: np.random.Generator, M: int, K: int, ch_per_group: int,
                        hit_prob: float = 0.9, spike_prob: float = 0.001):
    """Activations with `ch_per_group` persistent outlier channels in every 32-group.

    Per outlier channel a fixed factor ~U[20,100]; applied to a token with
    probability `hit_prob`; afterwards every element is independently multiplied
    by 30 with probability `spike_prob` (diffuse spikes the static table misses).
    Returns (X float64 [M,K], local channel table [Kg, ch_per_group]).
    """
    Kg = K // G
    X = rng.standard_normal((M, K))
    ch = np.stack([rng.permutation(G)[:ch_per_group] for _ in range(Kg)])  # [Kg, C]
    cols = (np.arange(Kg)[:, None] * G + ch).reshape(-1)
    factor = rng.uniform(20.0, 100.0, size=cols.size)
    if M > 0:
        hit = rng.random((M, cols.size)) < hit_prob
        X[:, cols] *= np.where(hit, factor[None, :], 1.0)
        spikes = rng.random((M, K)) < spike_prob
        X[spikes] *= 30.0
    return X, ch


def osc_linear_case(seed: int, M: int, K: int, N: int, ch_per_group: int):
    """One OSC-path linear (QKV / o_proj / gate_up shaped)."""
    rng = np.random.default_rng(seed)
    X, ch = planted_activations(rng, M, K, ch_per_group)
    W = 0.02 * rng.standard_normal((N, K))
    return {"X": _bf16(X), "W": _bf16(W), "lut": lut_from_channels(ch), "M": M, "K": K, "N": N}


def osc_weights_only(seed: int, K: int, N: int, ch_per_group: int):
    """Weights + lookup table of an OSC linear (same draw order as osc_linear_case with M=0)."""
    return osc_linear_case(seed, 0, K, N, ch_per_group)


def osc_activations_only(seed: int, M: int, K: int, ch_per_group: int):
    rng = np.random.default_rng(seed)
    X, ch = planted_activations(rng, M, K, ch_per_group)
    return _bf16(X), lut_from_channels(ch)


def fp8_linear_case(seed: int, M: int, K: int, N: int):
    """Down-projection shaped FP8 fallback linear: diffuse Student-t(3) activations."""
    rng = np.random.default_rng(seed)
    X = rng.standard_t(3.0, size=(M, K))
    W = 0.02 * rng.standard_normal((N, K))
    return {"X": _bf16(X), "W": _bf16(W), "M": M, "K": K, "N": N}


def qkv_case(M: int, seed: int = 0):
    """Qwen3-8B QKV projection: K=4096, N=6144, two persistent channels per group (K_o=256)."""
    return osc_linear_case(seed, M, 4096, 6144, 2)


def gate_up_case(M: int, seed: int = 0):
    """Qwen3-8B FFN gate_up: K=4096, N=24576, one channel per group (K_o=128)."""
    return osc_linear_case(seed, M, 4096, 24576, 1)


def o_proj_case(M: int, seed: int = 0):
    return osc_linear_case(seed, M, 4096, 4096, 1)


def down_case(M: int, seed: int = 0):
    """Qwen3-8B FFN down projection through the FP8 fallback: K=12288, N=4096."""
    return fp8_linear_case(seed, M, 12288, 4096)


def zipf_expert_rows(E: int = 128, T: int = 8192, top_k: int = 8, s: float = 1.1, seed: int = 0):
    """Rows per expert for top-k routing with Zipf(s) expert popularity.

    popularity p_e ~ (e+1)^-s; per token the k largest of log p + Gumbel noise.
    Returns int64 counts [E] summing to T*top_k.
    """
    rng = np.random.default_rng(seed)
    p = 1.0 / np.arange(1, E + 1) ** s
    p /= p.sum()
    g = rng.gumbel(size=(T, E)) + np.log(p)[None, :]
    top = np.argsort(-g, axis=1)[:, :top_k]
    return np.bincount(top.ravel(), minlength=E).astype(np.int64)


def offsets_from_counts(counts: np.ndarray) -> np.ndarray:
    off = np.zeros(counts.size + 1, dtype=np.int32)
    off[1:] = np.cumsum(counts)
    return off


def moe_gate_up_case(E: int, counts: np.ndarray, K: int = 2048, N: int = 1536, seed: int = 0,
                     weight_pool: int | None = None):
    """Grouped OSC linear: token rows sorted by expert, one lookup table for all experts.

    `weight_pool`: draw only that many distinct expert weight matrices and tile
    them (keeps host generation time bounded at E=128; values stay N(0,0.02)).
    """
    rng = np.random.default_rng(seed)
    Mtot = int(counts.sum())
    X, ch = planted_activations(rng, Mtot, K, 1)
    pool = E if weight_pool is None else min(E, weight_pool)
    Wp = _bf16(0.02 * rng.standard_normal((pool, N, K)))
    W = Wp[np.arange(E) % pool]
    return {"X": _bf16(X), "W": np.ascontiguousarray(W), "lut": lut_from_channels(ch),
            "off": offsets_from_counts(counts), "E": E, "K": K, "N": N, "M": Mtot}


def moe_down_case(E: int, counts: np.ndarray, K: int = 768, N: int = 2048, seed: int = 0,
                  weight_pool: int | None = None):
    """Grouped FP8 fallback linear with diffuse Student-t(3) inputs."""
    rng = np.random.default_rng(seed)
    Mtot = int(counts.sum())
    X = rng.standard_t(3.0, size=(Mtot, K))
    pool = E if weight_pool is None else min(E, weight_pool)
    Wp = _bf16(0.02 * rng.standard_normal((pool, N, K)))
    W = Wp[np.arange(E) % pool]
    return {"X": _bf16(X), "W": np.ascontiguousarray(W), "off": offsets_from_counts(counts),
            "E": E, "K": K, "N": N, "M": Mtot}


def nvfp4_tensor_exponent(bits: np.ndarray) -> int:
    """Power-of-two tensor-level scale for an NVFP4 tensor: the smallest e with amax * 2^-e <= 6 * 448, so that
    every block scale amax_b * 2^-e / 6 fits the E4M3 range.  An input recipe (calibration), handed to the oracle
    and to the library alike."""
    a = float(np.abs(bf16_bits_to_f64(bits)).max())
    if a == 0.0:
        return 0
    return int(np.ceil(np.log2(a / (6.0 * 448.0))))


def osc16_linear_case(seed: int, M: int, K: int, N: int):
    """OSC inputs for 16-channel groups: one planted channel per 16-group (same recipe as osc_linear_case)."""
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((M, K)).astype(np.float32)
    Kg = K // 16
    ch = rng.integers(0, 16, size=Kg)
    cols = np.arange(Kg) * 16 + ch
    factor = rng.uniform(20.0, 100.0, size=Kg).astype(np.float32)
    hit = rng.random((M, Kg)) < 0.9
    X[:, cols] *= np.where(hit, factor[None, :], 1.0).astype(np.float32)
    X *= np.where(rng.random((M, K)) < 0.001, 30.0, 1.0).astype(np.float32)
    W = (0.02 * rng.standard_normal((N, K))).astype(np.float32)
    return {"X": f32_to_bf16_bits(X), "W": f32_to_bf16_bits(W), "lut16": ch.astype(np.int8).reshape(-1, 1),
            "M": M, "K": K, "N": N}


# ----------------------------------------------------------------------------------------------------------------
# The same recipes drawn on the device (torch generator): for timing-only benchmark rows, where drawing 10^8 values
# with numpy on the host would take longer than everything that is measured.  Values are not bit-identical to the
# numpy recipes above (another generator); shapes, distributions and the planted structure are the same.  Parity
# tests never use these.

def osc_linear_case_torch(torch, seed: int, M: int, K: int, N: int, ch_per_group: int, device="cuda"):
    """osc_linear_case on the device -> {"X": bf16 [M,K], "W": bf16 [N,K], "lut": int8 [Kg,C] (host)}."""
    rng = np.random.default_rng(seed)
    Kg = K // G
    ch = np.stack([rng.permutation(G)[:ch_per_group] for _ in range(Kg)])
    cols = (np.arange(Kg)[:, None] * G + ch).reshape(-1)
    factor = rng.uniform(20.0, 100.0, size=cols.size).astype(np.float32)
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    X = torch.randn(M, K, generator=gen, device=device, dtype=torch.float32)
    cols_d = torch.from_numpy(cols.astype(np.int64)).to(device)
    hit = torch.rand(M, cols.size, generator=gen, device=device) < 0.9
    f = torch.where(hit, torch.from_numpy(factor).to(device)[None, :], torch.ones((), device=device))
    X[:, cols_d] *= f
    spikes = torch.rand(M, K, generator=gen, device=device) < 0.001
    X = torch.where(spikes, X * 30.0, X).to(torch.bfloat16)
    W = (0.02 * torch.randn(N, K, generator=gen, device=device, dtype=torch.float32)).to(torch.bfloat16)
    return {"X": X, "W": W, "lut": lut_from_channels(ch), "M": M, "K": K, "N": N}


def student_t3_torch(torch, gen, shape, device="cuda"):
    """Student-t with 3 degrees of freedom: z / sqrt(chi2_3 / 3), in chunks of rows to bound the scratch."""
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    rows = shape[0]
    step = max(1, (1 << 24) // max(1, shape[1]))
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        z = torch.randn(r1 - r0, shape[1], generator=gen, device=device)
        c = torch.randn(3, r1 - r0, shape[1], generator=gen, device=device).square_().sum(0)
        out[r0:r1] = (z / torch.sqrt(c / 3.0)).to(torch.bfloat16)
    return out


def fp8_linear_case_torch(torch, seed: int, M: int, K: int, N: int, device="cuda"):
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    X = student_t3_torch(torch, gen, (M, K), device)
    W = (0.02 * torch.randn(N, K, generator=gen, device=device, dtype=torch.float32)).to(torch.bfloat16)
    return {"X": X, "W": W, "M": M, "K": K, "N": N}
