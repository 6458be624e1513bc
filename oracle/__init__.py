"""ctypes front-end of the CPU oracle (oracle/osc_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, the smoke check and the bench's
cpu-baseline leg.  The CUDA package never imports this module and this module
never imports the CUDA package.  All arguments and results are numpy arrays in
host memory; bf16 tensors are uint16 bit patterns.

Function-to-paper map (details in the C file):
  quantize_extract / prepare_weights  Algorithm 2 (+ Section 3.3 weight split)
  gemm_dual / linear                   Eq. 5
  fp8_quantize / fp8_gemm / fp8_linear Section 3.4 fallback (per-token E4M3)
  mxfp8_quantize / mxfp8_gemm / mxfp8_linear   Section 3.4 fallback in its 8-bit micro-scaling form (MXFP8)
  dyn_quantize_extract / dyn_prepare_weights / dyn_linear   the dynamic-protection control group of Section 4.2
  nvfp4_quantize_extract / nvfp4_gemm / nvfp4_linear         the NVFP4 / G = 16 variant (efficiency table, G = 16)
  threshold / profile_indexing / clustering_density   Eq. 1-4, Algorithm 1 (offline profiling)
  rmsnorm (oracle/rmsnorm.py)          the normalization in front of Algorithm 2 when the two are fused (Section 3.3)
  swiglu / silu32 / exp32              the activation in front of the FP8 quantizer of the down projection (Sections 3.3, 3.4)
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "osc_oracle.c")
_LIB = os.path.join(_HERE, "libosc_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
                               "-o", _LIB, _SRC, "-lm"])
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.osc_ref_e2m1_decode.restype = C.c_double
        _lib.osc_ref_e2m1_decode.argtypes = [C.c_int]
        _lib.osc_ref_e2m1_encode.argtypes = [C.c_double]
        _lib.osc_ref_e4m3_decode.restype = C.c_double
        _lib.osc_ref_e4m3_decode.argtypes = [C.c_int]
        _lib.osc_ref_e4m3_encode.argtypes = [C.c_double]
        _lib.osc_ref_e8m0_from_amax.argtypes = [C.c_double]
        _lib.osc_ref_sf_index.restype = C.c_int64
        _lib.osc_ref_sf_index.argtypes = [C.c_int64, C.c_int64, C.c_int64]
        _lib.osc_ref_sf_bytes.restype = C.c_int64
        _lib.osc_ref_sf_bytes.argtypes = [C.c_int64, C.c_int64]
        _lib.osc_ref_sf_row_base.restype = C.c_int64
        _lib.osc_ref_e8m0_from_amax_emax.argtypes = [C.c_double, C.c_int]
        _lib.osc_ref_sf16_index.restype = C.c_int64
        _lib.osc_ref_sf16_index.argtypes = [C.c_int64, C.c_int64, C.c_int64]
        _lib.osc_ref_sf16_bytes.restype = C.c_int64
        _lib.osc_ref_sf16_bytes.argtypes = [C.c_int64, C.c_int64]
        _lib.osc_ref_threshold.restype = C.c_double
        _lib.osc_ref_threshold.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_int, C.c_double]
        _lib.osc_ref_threshold_bits.restype = C.c_uint32
        _lib.osc_ref_threshold_bits.argtypes = [C.c_double]
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def num_threads() -> int:
    return int(lib().osc_ref_num_threads())


def e2m1_encode(v: float) -> int:
    return int(lib().osc_ref_e2m1_encode(float(v)))


def e2m1_decode(n: int) -> float:
    return float(lib().osc_ref_e2m1_decode(int(n)))


def e4m3_encode(v: float) -> int:
    return int(lib().osc_ref_e4m3_encode(float(v)))


def e4m3_decode(b: int) -> float:
    return float(lib().osc_ref_e4m3_decode(int(b)))


def e8m0_from_amax(a: float) -> int:
    return int(lib().osc_ref_e8m0_from_amax(float(a)))


def sf_index(r: int, g: int, K: int) -> int:
    return int(lib().osc_ref_sf_index(r, g, K))


def sf_bytes(rows: int, K: int) -> int:
    return int(lib().osc_ref_sf_bytes(rows, K))


def lut_normalize(lut: np.ndarray, K: int):
    """-> (K_o, K_o_pad, mask u32[Kg], prefix i32[Kg], idx_o i32[K_o]); raises on a bad table."""
    lut = np.ascontiguousarray(lut, dtype=np.int8)
    Kg = K // 32
    if lut.ndim == 1:
        lut = lut.reshape(Kg, -1)
    assert lut.shape[0] == Kg
    mask = np.zeros(Kg, np.uint32)
    prefix = np.zeros(Kg, np.int32)
    idx = np.zeros(max(K, 1), np.int32)
    ko = lib().osc_ref_lut_normalize(_p(lut), Kg, lut.shape[1], _p(mask), _p(prefix), _p(idx))
    if ko < 0:
        raise ValueError({-1: "lookup-table entry outside -1..31", -2: "duplicate channel in a group"}[ko])
    return ko, int(lib().osc_ref_ko_pad(ko)), mask, prefix, idx[:ko].copy()


def quantize_extract(X: np.ndarray, lut: np.ndarray):
    """Algorithm 2 on bf16 rows X [M,K] -> dict(xq [M,K/2] u8, sf u8 (block layout), xo [M,K_o_pad] u16)."""
    X = np.ascontiguousarray(X, dtype=np.uint16)
    M, K = X.shape
    lut = np.ascontiguousarray(lut, dtype=np.int8).reshape(K // 32, -1)
    ko, kop, mask, prefix, idx = lut_normalize(lut, K)
    xq = np.zeros((M, K // 2), np.uint8)
    sf = np.zeros(sf_bytes(M, K), np.uint8)
    xo = np.zeros((M, kop), np.uint16)
    rc = lib().osc_ref_quantize_extract(_p(X), C.c_int64(K), M, K, _p(lut), lut.shape[1], _p(xq), _p(sf), _p(xo))
    assert rc == ko
    return {"xq": xq, "sf": sf, "xo": xo, "K_o": ko, "K_o_pad": kop, "mask": mask, "prefix": prefix, "idx_o": idx}


def prepare_weights(W: np.ndarray, lut: np.ndarray):
    """Offline weight split (Section 3.3): the same routine on the rows of W [N,K]."""
    return quantize_extract(W, lut)


def sf_row_base(off: np.ndarray):
    off = np.ascontiguousarray(off, dtype=np.int32)
    E = off.size - 1
    base = np.zeros(max(E, 1), np.int64)
    total = lib().osc_ref_sf_row_base(_p(off), E, _p(base))
    return base[:E], int(total)


def quantize_extract_grouped(X: np.ndarray, off: np.ndarray, lut: np.ndarray):
    X = np.ascontiguousarray(X, dtype=np.uint16)
    off = np.ascontiguousarray(off, dtype=np.int32)
    M, K = X.shape
    E = off.size - 1
    lut = np.ascontiguousarray(lut, dtype=np.int8).reshape(K // 32, -1)
    ko, kop, mask, prefix, idx = lut_normalize(lut, K)
    base, total = sf_row_base(off)
    xq = np.zeros((M, K // 2), np.uint8)
    sf = np.zeros(sf_bytes(total, K), np.uint8)
    xo = np.zeros((M, kop), np.uint16)
    rc = lib().osc_ref_quantize_extract_grouped(_p(X), C.c_int64(K), _p(off), E, K, _p(lut), lut.shape[1],
                                                _p(xq), _p(sf), _p(xo), kop)
    assert rc >= 0
    return {"xq": xq, "sf": sf, "xo": xo, "K_o": ko, "K_o_pad": kop, "sf_row_base": base, "sf_rows": total}


def gemm_dual(act: dict, wts: dict, rows=None, sf_rows=None):
    """Eq. 5 for the listed activation rows (all rows if None) -> (Y, T) float64 [nrows, N]."""
    xq, sfa, xo = act["xq"], act["sf"], act["xo"]
    wq, sfw, wo = wts["xq"], wts["sf"], wts["xo"]
    M, K2 = xq.shape
    K = 2 * K2
    N = wq.shape[0]
    kop = xo.shape[1]
    assert wq.shape[1] == K2 and wo.shape[1] == kop
    if rows is None:
        rows = np.arange(M, dtype=np.int32)
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    sf_rows = rows if sf_rows is None else np.ascontiguousarray(sf_rows, dtype=np.int32)
    Y = np.zeros((rows.size, N), np.float64)
    T = np.zeros((rows.size, N), np.float64)
    lib().osc_ref_gemm_dual_rows(_p(xq), _p(sfa), _p(xo), _p(rows), _p(sf_rows), rows.size,
                                 _p(wq), _p(sfw), _p(wo), N, K, kop, _p(Y), _p(T))
    return Y, T


def linear(X: np.ndarray, W: np.ndarray, lut: np.ndarray, rows=None):
    """The whole OSC linear: Algorithm 2 on X, weight split on W, Eq. 5."""
    act = quantize_extract(X, lut)
    wts = prepare_weights(W, lut)
    Y, T = gemm_dual(act, wts, rows)
    return Y, T, act, wts


def fp8_quantize(X: np.ndarray):
    X = np.ascontiguousarray(X, dtype=np.uint16)
    M, K = X.shape
    x8 = np.zeros((M, K), np.uint8)
    sx = np.zeros(M, np.float32)
    lib().osc_ref_fp8_quantize(_p(X), C.c_int64(K), M, K, _p(x8), _p(sx))
    return x8, sx


def fp8_gemm(x8, sx, w8, sw, rows=None):
    M, K = x8.shape
    N = w8.shape[0]
    if rows is None:
        rows = np.arange(M, dtype=np.int32)
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    Y = np.zeros((rows.size, N), np.float64)
    T = np.zeros((rows.size, N), np.float64)
    lib().osc_ref_fp8_gemm_rows(_p(np.ascontiguousarray(x8)), _p(np.ascontiguousarray(sx, dtype=np.float32)),
                                _p(rows), rows.size, _p(np.ascontiguousarray(w8)),
                                _p(np.ascontiguousarray(sw, dtype=np.float32)), N, K, _p(Y), _p(T))
    return Y, T


def fp8_linear(X: np.ndarray, W: np.ndarray, rows=None):
    x8, sx = fp8_quantize(X)
    w8, sw = fp8_quantize(W)
    Y, T = fp8_gemm(x8, sx, w8, sw, rows)
    return Y, T, (x8, sx), (w8, sw)


def e8m0_from_amax_emax(a: float, emax: int) -> int:
    return int(lib().osc_ref_e8m0_from_amax_emax(float(a), int(emax)))


def mxfp8_quantize(X: np.ndarray):
    """MXFP8 (E4M3 elements, E8M0 scale per 32) of bf16 rows X [M,K] -> (x8 [M,K] u8, sf u8 in block layout)."""
    X = np.ascontiguousarray(X, dtype=np.uint16)
    M, K = X.shape
    x8 = np.zeros((M, K), np.uint8)
    sf = np.zeros(sf_bytes(M, K), np.uint8)
    lib().osc_ref_mxfp8_quantize(_p(X), C.c_int64(K), M, K, _p(x8), _p(sf))
    return x8, sf


def mxfp8_gemm(x8, sfa, w8, sfw, rows=None):
    M, K = x8.shape
    N = w8.shape[0]
    if rows is None:
        rows = np.arange(M, dtype=np.int32)
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    Y = np.zeros((rows.size, N), np.float64)
    T = np.zeros((rows.size, N), np.float64)
    lib().osc_ref_mxfp8_gemm_rows(_p(np.ascontiguousarray(x8)), _p(np.ascontiguousarray(sfa)), _p(rows), rows.size,
                                  _p(np.ascontiguousarray(w8)), _p(np.ascontiguousarray(sfw)), N, K, _p(Y), _p(T))
    return Y, T


def mxfp8_quantize_grouped(X: np.ndarray, off: np.ndarray):
    """Rows sorted by expert: every expert is quantized on its own and its scale blocks (whole 128-row blocks,
    rows numbered from 0 inside the expert) are laid end to end, so expert e starts at scale row
    sum_{e'<e} roundup(m_e', 128).  -> (x8 [M,K], sf, per-expert (x8, sf) list)."""
    X = np.ascontiguousarray(X, dtype=np.uint16)
    parts, sfs = [], []
    for e in range(off.size - 1):
        x8e, sfe = mxfp8_quantize(X[int(off[e]):int(off[e + 1])])
        parts.append((x8e, sfe))
        sfs.append(sfe)
    x8 = np.concatenate([p[0] for p in parts], axis=0) if parts else np.zeros((0, X.shape[1]), np.uint8)
    return x8, (np.concatenate(sfs) if sfs else np.zeros(0, np.uint8)), parts


def mxfp8_linear(X: np.ndarray, W: np.ndarray, rows=None):
    x8, sfa = mxfp8_quantize(X)
    w8, sfw = mxfp8_quantize(W)
    Y, T = mxfp8_gemm(x8, sfa, w8, sfw, rows)
    return Y, T, (x8, sfa), (w8, sfw)


def dyn_quantize_extract(X: np.ndarray):
    """Dynamic protection: per token and 32-group the run-time largest element is extracted (Section 4.2 control
    group).  -> dict(xq, sf, idx u8 [M,K/32], val u16 [M,K/32], xo u16 [M,K] = the extracted elements scattered
    back to their channels, zero elsewhere)."""
    X = np.ascontiguousarray(X, dtype=np.uint16)
    M, K = X.shape
    Kg = K // 32
    xq = np.zeros((M, K // 2), np.uint8)
    sf = np.zeros(sf_bytes(M, K), np.uint8)
    idx = np.zeros((M, Kg), np.uint8)
    val = np.zeros((M, Kg), np.uint16)
    lib().osc_ref_dyn_quantize_extract(_p(X), C.c_int64(K), M, K, _p(xq), _p(sf), _p(idx), _p(val))
    xo = np.zeros((M, K), np.uint16)
    cols = (np.arange(Kg, dtype=np.int64) * 32)[None, :] + idx
    np.put_along_axis(xo, cols, val, axis=1)
    return {"xq": xq, "sf": sf, "idx": idx, "val": val, "xo": xo, "K_o": K, "K_o_pad": K}


def dyn_prepare_weights(W: np.ndarray):
    """Weights of the dynamic baseline: MXFP4 of the whole matrix (no column zeroed) + the bf16 matrix itself
    as the high-precision operand (any column can be picked by some token)."""
    W = np.ascontiguousarray(W, dtype=np.uint16)
    K = W.shape[1]
    q = quantize_extract(W, np.full((K // 32, 1), -1, np.int8))
    return {"xq": q["xq"], "sf": q["sf"], "xo": W.copy()}


def dyn_linear(X: np.ndarray, W: np.ndarray, rows=None):
    act = dyn_quantize_extract(X)
    wts = dyn_prepare_weights(W)
    Y, T = gemm_dual(act, wts, rows)
    return Y, T, act, wts


def sf16_index(r: int, b: int, K: int) -> int:
    return int(lib().osc_ref_sf16_index(r, b, K))


def nvfp4_quantize_extract(X: np.ndarray, lut16: np.ndarray, e: int):
    """NVFP4 / G = 16 form of Algorithm 2 with tensor-level scale 2^e: X bf16 [M,K], lut16 [K/16, C] entries -1..15
    -> dict(xq [M,K/2], sf (E4M3 block scales, 128 x 4 block layout per 64 channels), xo [M,K_o_pad] scaled by 2^-e)."""
    X = np.ascontiguousarray(X, dtype=np.uint16)
    M, K = X.shape
    lut16 = np.ascontiguousarray(lut16, dtype=np.int8).reshape(K // 16, -1)
    Kg = K // 16
    mask = np.zeros(Kg, np.uint32)
    prefix = np.zeros(Kg, np.int32)
    idx = np.zeros(max(K, 1), np.int32)
    ko = lib().osc_ref_lut16_normalize(_p(lut16), Kg, lut16.shape[1], _p(mask), _p(prefix), _p(idx))
    if ko < 0:
        raise ValueError({-1: "lookup-table entry outside -1..15", -2: "duplicate channel in a group"}[ko])
    kop = int(lib().osc_ref_ko_pad(ko))
    xq = np.zeros((M, K // 2), np.uint8)
    sf = np.zeros(int(lib().osc_ref_sf16_bytes(M, K)), np.uint8)
    xo = np.zeros((M, kop), np.uint16)
    rc = lib().osc_ref_nvfp4_quantize_extract(_p(X), C.c_int64(K), M, K, _p(lut16), lut16.shape[1], int(e), _p(xq),
                                              _p(sf), _p(xo))
    assert rc == ko
    return {"xq": xq, "sf": sf, "xo": xo, "K_o": ko, "K_o_pad": kop, "idx_o": idx[:ko].copy(), "e": int(e)}


def nvfp4_gemm(act: dict, wts: dict, rows=None):
    xq, sfa, xo = act["xq"], act["sf"], act["xo"]
    wq, sfw, wo = wts["xq"], wts["sf"], wts["xo"]
    M, K2 = xq.shape
    N = wq.shape[0]
    if rows is None:
        rows = np.arange(M, dtype=np.int32)
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    Y = np.zeros((rows.size, N), np.float64)
    T = np.zeros((rows.size, N), np.float64)
    lib().osc_ref_nvfp4_gemm_rows(_p(xq), _p(sfa), _p(xo), _p(rows), rows.size, _p(wq), _p(sfw), _p(wo), N, 2 * K2,
                                  xo.shape[1], act["e"] + wts["e"], _p(Y), _p(T))
    return Y, T


def nvfp4_linear(X, W, lut16, ex: int, ew: int, rows=None):
    act = nvfp4_quantize_extract(X, lut16, ex)
    wts = nvfp4_quantize_extract(W, lut16, ew)
    Y, T = nvfp4_gemm(act, wts, rows)
    return Y, T, act, wts


def threshold(X: np.ndarray, alpha: float = 5.0) -> float:
    """Eq. 1: T_l = alpha * mean|X|."""
    X = np.ascontiguousarray(X, dtype=np.uint16)
    S, H = X.shape
    return float(lib().osc_ref_threshold(_p(X), H, S, H, float(alpha)))


def threshold_bits(T: float) -> int:
    return int(lib().osc_ref_threshold_bits(float(T)))


def profile_indexing(X: np.ndarray, T: float):
    """Algorithm 1 for one (position, layer) -> (L int8 [K], n_hit i32 [K], n_total i32 [K])."""
    X = np.ascontiguousarray(X, dtype=np.uint16)
    S, H = X.shape
    K = H // 32
    L = np.zeros(K, np.int8)
    nh = np.zeros(K, np.int32)
    nt = np.zeros(K, np.int32)
    rc = lib().osc_ref_profile_indexing(_p(X), C.c_int64(H), S, H, C.c_double(T), _p(L), _p(nh), _p(nt))
    assert rc == 0
    return L, nh, nt


def clustering_density(n_hit: np.ndarray, n_total: np.ndarray):
    """Eq. 4 and the block mean: C_k = n_hit/n_total (0 for groups without outlier tokens), mean over all K groups."""
    c = np.where(n_total > 0, n_hit / np.maximum(n_total, 1), 0.0)
    return c, float(c.mean())


def exp32(z: float) -> float:
    """The fp32 exponential the SwiGLU definition uses (see the C file)."""
    f = lib().osc_ref_exp32
    f.restype, f.argtypes = C.c_float, [C.c_float]
    return float(f(C.c_float(z)))


def silu32(g: float) -> float:
    f = lib().osc_ref_silu32
    f.restype, f.argtypes = C.c_float, [C.c_float]
    return float(f(C.c_float(g)))


def swiglu(GU: np.ndarray, I: int) -> np.ndarray:
    """GU [M, >= 2I] bf16 bits (gate columns [0, I), up columns [I, 2I)) -> h = bf16(silu32(gate) * up) [M, I]."""
    GU = np.ascontiguousarray(GU, dtype=np.uint16)
    M = GU.shape[0]
    H = np.zeros((M, I), np.uint16)
    rc = lib().osc_ref_swiglu(_p(GU), C.c_int64(GU.shape[1]), M, I, _p(H))
    assert rc == 0
    return H


from .rmsnorm import add_rmsnorm, f64_to_bf16_bits, residual_add, rmsnorm  # noqa: E402,F401
