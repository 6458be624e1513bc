"""Helpers for the GPU parity tests: numpy <-> torch marshalling and the tolerance check."""
import numpy as np
import torch


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> cuda bf16 tensor with the same bits."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


def host_u8(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().numpy()


def host_bf16_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().view(torch.int16).cpu().numpy().view(np.uint16)


def host_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def poison(nbytes: int) -> torch.Tensor:
    """0xFF-filled device buffer: unwritten bytes show up in the comparisons."""
    return torch.full((max(int(nbytes), 16),), 0xFF, dtype=torch.uint8, device="cuda")


def assert_within_tolerance(Y, Yref, T, what=""):
    """|err| <= 2^-7 |ref| + 1e-3 * sum_k |a_k b_k| per element (the bound the task states)."""
    err = np.abs(Y - Yref)
    bound = 2.0 ** -7 * np.abs(Yref) + 1e-3 * T
    bad = err > bound
    if bad.any():
        i = np.unravel_index(np.argmax(err - bound), err.shape)
        raise AssertionError(f"{what}: {bad.sum()} of {bad.size} outside tolerance; worst at {i}: "
                             f"got {Y[i]!r} ref {Yref[i]!r} bound {bound[i]!r}; "
                             f"bad rows {np.unique(np.nonzero(bad)[0])[:8]} cols {np.unique(np.nonzero(bad)[1])[:8]}")


def valid_sf_bytes(oracle, rows: int, K: int, row_base: int = 0) -> np.ndarray:
    r = np.arange(rows)[:, None] + row_base
    g = np.arange(K // 32)[None, :]
    idx = ((r // 128) * (K // 128) + g // 4) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + (g % 4)
    assert idx[0, 0] == oracle.sf_index(row_base, 0, K)
    return idx.ravel()
