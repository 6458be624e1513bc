"""Work, traffic and roofline model of the OSC dual-path linear (host-side arithmetic only).

Path A is a block-scaled FP4 GEMM over all K channels, Path B a dense BF16 GEMM
over the K_o protected channels (Eq. 5).  The paper's efficiency table
(Table 3) assumes matrix-unit peaks in the ratio 1:2:4 for 16-, 8- and 4-bit
operands; with that ratio the compute-bound speed-up over a W8A8 GEMM is
(1/2) / (1/4 + c/G) for c protected channels per group of G.
"""
from __future__ import annotations


def analytic_speedup_vs_w8a8(G: int = 32, channels_per_group: int = 1) -> float:
    """Compute-bound column of Table 3: time per MAC is 1/4 (FP4), 1/2 (FP8), 1 (16-bit)."""
    return 0.5 / (0.25 + channels_per_group / G)


def analytic_cycle_saving_vs_w8a8(G: int = 32, channels_per_group: int = 1) -> float:
    return 1.0 - (0.25 + channels_per_group / G) / 0.5


def analytic_branch_overhead(G: int = 32, channels_per_group: int = 1) -> float:
    """Path-B cycles relative to Path-A cycles (Section 3.3, item 4)."""
    return (channels_per_group / G) / 0.25


def osc_flops(M: int, N: int, K: int, K_o: int):
    """(FP4 flops, BF16 flops): useful work only, pad columns not counted."""
    return 2.0 * M * N * K, 2.0 * M * N * K_o


def osc_bytes(M: int, N: int, K: int, K_o: int) -> float:
    """Algorithmic HBM bytes of one OSC linear: X in, prepared weights in, Y out."""
    return 2.0 * M * K + (N * K / 2 + N * K / 32 + 2.0 * N * K_o) + 2.0 * M * N


def osc_intermediate_bytes(M: int, K: int, K_o_pad: int) -> float:
    """Bytes of Xq + SFA + X_o (written by the quantizer, read by the GEMM)."""
    return M * K / 2 + M * K / 32 + 2.0 * M * K_o_pad


def quantize_extract_bytes(M: int, K: int, K_o_pad: int) -> float:
    return 2.0 * M * K + osc_intermediate_bytes(M, K, K_o_pad)


def fp8_flops(M: int, N: int, K: int) -> float:
    return 2.0 * M * N * K


def fp8_bytes(M: int, N: int, K: int) -> float:
    return 2.0 * M * K + N * K + 4.0 * N + 2.0 * M * N


def fp8_quantize_bytes(M: int, K: int) -> float:
    return 2.0 * M * K + M * K + 4.0 * M


def peaks(bf16_tflops: float, hbm_gbs: float):
    """Tensor peaks by operand width from the measured BF16 figure, 1:2:4 as in Table 3."""
    return {"bf16": bf16_tflops * 1e12, "fp8": 2 * bf16_tflops * 1e12, "fp4": 4 * bf16_tflops * 1e12,
            "hbm": hbm_gbs * 1e9}


def osc_roofline_seconds(M, N, K, K_o, pk) -> float:
    f4, f16 = osc_flops(M, N, K, K_o)
    return max(f4 / pk["fp4"] + f16 / pk["bf16"], osc_bytes(M, N, K, K_o) / pk["hbm"])


def fp8_roofline_seconds(M, N, K, pk) -> float:
    return max(fp8_flops(M, N, K) / pk["fp8"], fp8_bytes(M, N, K) / pk["hbm"])
