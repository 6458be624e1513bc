"""Thin ctypes binding of the C ABI in include/osc.h (argument marshalling only).

Every function here has the name of the C entry point it calls.  torch is used
for device memory and streams; all arithmetic happens in the CUDA library.
Importing this module loads `libosc_b200.so` from the package directory and
raises if it is missing: there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libosc_b200.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} not found: build it with `python -c 'import __graft_entry__ as g; g.build()'` "
                      "(nvcc, sm_100a). The OSC path has no CPU fallback.")
_lib = C.CDLL(LIB_PATH)

OSC_OK = 0
STATUS = {0: "OSC_OK", -1: "OSC_ERR_INVALID_ARG", -2: "OSC_ERR_SHAPE", -3: "OSC_ERR_LUT", -4: "OSC_ERR_ALIGN",
          -5: "OSC_ERR_WORKSPACE", -6: "OSC_ERR_ARCH", -7: "OSC_ERR_CUDA", -8: "OSC_ERR_TIMEOUT"}


class OscError(RuntimeError):
    def __init__(self, status: int, detail: str):
        super().__init__(f"{STATUS.get(status, status)}: {detail}")
        self.status = status


class WeightSizes(C.Structure):
    _fields_ = [("K_o", C.c_int32), ("K_o_pad", C.c_int32), ("wq_bytes", C.c_size_t), ("sfw_bytes", C.c_size_t),
                ("wo_bytes", C.c_size_t), ("meta_bytes", C.c_size_t)]


class ActSizes(C.Structure):
    _fields_ = [(n, C.c_size_t) for n in ("xq_bytes", "sfa_bytes", "xo_bytes", "sched_bytes", "xq_offset",
                                          "sfa_offset", "xo_offset", "sched_offset", "workspace_bytes")]


class Fp8ActSizes(C.Structure):
    _fields_ = [(n, C.c_size_t) for n in ("x8_bytes", "sx_bytes", "sched_bytes", "x8_offset", "sx_offset",
                                          "sched_offset", "workspace_bytes")]


class DynActSizes(C.Structure):
    _fields_ = [(n, C.c_size_t) for n in ("xq_bytes", "sfa_bytes", "xo_bytes", "idx_bytes", "val_bytes", "xq_offset",
                                          "sfa_offset", "xo_offset", "idx_offset", "val_offset", "workspace_bytes")]


class Mxfp8WeightSizes(C.Structure):
    _fields_ = [("w8_bytes", C.c_size_t), ("sfw_bytes", C.c_size_t)]


class Mxfp8ActSizes(C.Structure):
    _fields_ = [(n, C.c_size_t) for n in ("x8_bytes", "sfa_bytes", "sched_bytes", "x8_offset", "sfa_offset",
                                          "sched_offset", "workspace_bytes")]


_vp, _i, _i64, _sz = C.c_void_p, C.c_int, C.c_int64, C.c_size_t
_SIGS = {
    "osc_status_string": (C.c_char_p, [_i]),
    "osc_last_error": (C.c_char_p, []),
    "osc_sync_check": (_i, [_vp]),
    "osc_weight_sizes": (_i, [_i, _i, _i, _vp, _i, C.POINTER(WeightSizes)]),
    "osc_prepare_weights": (_i, [_vp, _i, _i, _i64, _vp, _i, _vp, _vp, _vp, _vp, _vp, C.POINTER(_vp)]),
    "osc_prepare_weights_grouped": (_i, [_vp, _i, _i, _i, _vp, _i, _vp, _vp, _vp, _vp, _vp, C.POINTER(_vp)]),
    "osc_weights_destroy": (_i, [_vp]),
    "osc_act_sizes": (_i, [_vp, _i, C.POINTER(ActSizes)]),
    "osc_quantize_extract": (_i, [_vp, _vp, _i, _i64, _vp, _vp, _vp, _vp]),
    "osc_gemm_dual": (_i, [_vp, _vp, _vp, _vp, _i, _vp, _i64, _vp]),
    "osc_linear": (_i, [_vp, _vp, _i, _i64, _vp, _i64, _vp, _sz, _vp]),
    "osc_linear_static": (_i, [_vp, _vp, _i, _i64, _vp, _i64, _vp]),
    "osc_linear_grouped": (_i, [_vp, _vp, _vp, _i, _i64, _vp, _i64, _vp, _sz, _vp]),
    "osc_gather_workspace_bytes": (_i, [_vp, _i, _i, C.POINTER(_sz)]),
    "osc_linear_grouped_gather": (_i, [_vp, _vp, _i, _i64, _vp, _vp, _i, _vp, _i64, _vp, _sz, _vp]),
    "osc_rmsnorm_linear_grouped_gather": (_i, [_vp, _vp, _i, _i64, _vp, C.c_float, _vp, _vp, _i, _vp, _i64, _vp, _sz, _vp]),
    "osc_swiglu_fp8_linear_grouped": (_i, [_vp, _vp, _vp, _i, _i64, _vp, _i64, _vp, _sz, _vp]),
    "osc_add_rmsnorm": (_i, [_vp, _vp, _i, _i, _i64, _i64, _vp, C.c_float, _vp, _i64, _vp, _i64, _vp]),
    "osc_add_rmsnorm_quantize_extract": (_i, [_vp, _vp, _vp, _i, _i64, _i64, _vp, C.c_float, _vp, _i64, _vp, _vp, _vp, _vp]),
    "osc_add_rmsnorm_linear": (_i, [_vp, _vp, _vp, _i, _i64, _i64, _vp, C.c_float, _vp, _i64, _vp, _i64, _vp, _sz, _vp]),
    "osc_rmsnorm": (_i, [_vp, _i, _i, _i64, _vp, C.c_float, _vp, _i64, _vp]),
    "osc_swiglu": (_i, [_vp, _i, _i, _i64, _vp, _i64, _vp]),
    "osc_swiglu_fp8_quantize": (_i, [_vp, _i, _i, _i64, _vp, _vp, _vp]),
    "osc_swiglu_fp8_linear": (_i, [_vp, _vp, _i, _i64, _vp, _i64, _vp, _sz, _vp]),
    "osc_rmsnorm_quantize_extract": (_i, [_vp, _vp, _i, _i64, _vp, C.c_float, _vp, _vp, _vp, _vp]),
    "osc_rmsnorm_linear": (_i, [_vp, _vp, _i, _i64, _vp, C.c_float, _vp, _i64, _vp, _sz, _vp]),
    "osc_profile_scratch_bytes": (_i, [_i, C.POINTER(_sz)]),
    "osc_profile_lut": (_i, [_vp, _i, _i, _i64, C.c_float, _vp, _sz, _vp, _vp, _vp, _vp, _vp]),
    "osc_fp8_prepare_weights": (_i, [_vp, _i, _i, _i64, _vp, _vp, _vp, C.POINTER(_vp)]),
    "osc_fp8_prepare_weights_grouped": (_i, [_vp, _i, _i, _i, _vp, _vp, _vp, C.POINTER(_vp)]),
    "osc_fp8_weights_destroy": (_i, [_vp]),
    "osc_fp8_act_sizes": (_i, [_vp, _i, C.POINTER(Fp8ActSizes)]),
    "osc_fp8_quantize": (_i, [_vp, _i, _i, _i64, _vp, _vp, _vp]),
    "osc_fp8_gemm": (_i, [_vp, _vp, _vp, _i, _vp, _i64, _vp]),
    "osc_fp8_linear": (_i, [_vp, _vp, _i, _i64, _vp, _i64, _vp, _sz, _vp]),
    "osc_fp8_linear_grouped": (_i, [_vp, _vp, _vp, _i, _i64, _vp, _i64, _vp, _sz, _vp]),
    "osc_dyn_weight_sizes": (_i, [_i, _i, C.POINTER(WeightSizes)]),
    "osc_dyn_prepare_weights": (_i, [_vp, _i, _i, _i64, _vp, _vp, _vp, _vp, _vp, C.POINTER(_vp)]),
    "osc_dyn_act_sizes": (_i, [_vp, _i, C.POINTER(DynActSizes)]),
    "osc_dyn_quantize_extract": (_i, [_vp, _vp, _i, _i64, _vp, _vp, _vp, _vp, _vp, _vp]),
    "osc_dyn_linear": (_i, [_vp, _vp, _i, _i64, _vp, _i64, _vp, _sz, _vp]),
    "osc_nvfp4_weight_sizes": (_i, [_i, _i, _vp, _i, C.POINTER(WeightSizes)]),
    "osc_nvfp4_prepare_weights": (_i, [_vp, _i, _i, _i64, _vp, _i, _i, _vp, _vp, _vp, _vp, _vp, C.POINTER(_vp)]),
    "osc_nvfp4_weight_sizes_grouped": (_i, [_i, _i, _i, _vp, _i, C.POINTER(WeightSizes)]),
    "osc_nvfp4_prepare_weights_grouped": (_i, [_vp, _i, _i, _i, _vp, _i, _i, _vp, _vp, _vp, _vp, _vp, C.POINTER(_vp)]),
    "osc_nvfp4_linear_grouped": (_i, [_vp, _vp, _vp, _i, _i64, _i, _vp, _i64, _vp, _sz, _vp]),
    "osc_nvfp4_act_sizes": (_i, [_vp, _i, C.POINTER(ActSizes)]),
    "osc_nvfp4_quantize_extract": (_i, [_vp, _vp, _i, _i64, _i, _vp, _vp, _vp, _vp]),
    "osc_nvfp4_gemm": (_i, [_vp, _vp, _vp, _vp, _i, _i, _vp, _i64, _vp]),
    "osc_nvfp4_linear": (_i, [_vp, _vp, _i, _i64, _i, _vp, _i64, _vp, _sz, _vp]),
    "osc_gate_up_weight_sizes": (_i, [_i, _i, _vp, _i, C.POINTER(WeightSizes)]),
    "osc_prepare_weights_gate_up": (_i, [_vp, _i, _i, _i64, _vp, _i, _vp, _vp, _vp, _vp, _vp, C.POINTER(_vp)]),
    "osc_linear_swiglu_workspace_bytes": (_i, [_vp, _i, C.POINTER(_sz)]),
    "osc_linear_swiglu": (_i, [_vp, _vp, _i, _i64, _vp, _i64, _vp, _sz, _vp]),
    "osc_rmsnorm_linear_swiglu": (_i, [_vp, _vp, _i, _i64, _vp, C.c_float, _vp, _i64, _vp, _sz, _vp]),
    "osc_gate_up_weight_sizes_grouped": (_i, [_i, _i, _i, _vp, _i, C.POINTER(WeightSizes)]),
    "osc_prepare_weights_gate_up_grouped": (_i, [_vp, _i, _i, _i, _vp, _i, _vp, _vp, _vp, _vp, _vp, C.POINTER(_vp)]),
    "osc_linear_swiglu_grouped": (_i, [_vp, _vp, _vp, _i, _i64, _vp, _i64, _vp, _sz, _vp]),
    "osc_swiglu_gather_workspace_bytes": (_i, [_vp, _i, _i, C.POINTER(_sz)]),
    "osc_linear_swiglu_grouped_gather": (_i, [_vp, _vp, _i, _i64, _vp, _vp, _i, _vp, _i64, _vp, _sz, _vp]),
    "osc_rmsnorm_linear_swiglu_grouped_gather": (_i, [_vp, _vp, _i, _i64, _vp, C.c_float, _vp, _vp, _i, _vp, _i64, _vp, _sz, _vp]),
    "osc_nvfp4_rmsnorm_quantize_extract": (_i, [_vp, _vp, _i, _i64, _vp, C.c_float, _i, _vp, _vp, _vp, _vp]),
    "osc_nvfp4_rmsnorm_linear": (_i, [_vp, _vp, _i, _i64, _vp, C.c_float, _i, _vp, _i64, _vp, _sz, _vp]),
    "osc_nvfp4_gather_workspace_bytes": (_i, [_vp, _i, _i, C.POINTER(_sz)]),
    "osc_nvfp4_linear_grouped_gather": (_i, [_vp, _vp, _i, _i64, _vp, _vp, _i, _i, _vp, _i64, _vp, _sz, _vp]),
    "osc_nvfp4_rmsnorm_linear_grouped_gather": (_i, [_vp, _vp, _i, _i64, _vp, C.c_float, _vp, _vp, _i, _i, _vp, _i64, _vp, _sz,
                                                     _vp]),
    "osc_mxfp8_weight_sizes": (_i, [_i, _i, _i, C.POINTER(Mxfp8WeightSizes)]),
    "osc_mxfp8_prepare_weights_grouped": (_i, [_vp, _i, _i, _i, _vp, _vp, _vp, C.POINTER(_vp)]),
    "osc_mxfp8_linear_grouped": (_i, [_vp, _vp, _vp, _i, _i64, _vp, _i64, _vp, _sz, _vp]),
    "osc_mxfp8_prepare_weights": (_i, [_vp, _i, _i, _i64, _vp, _vp, _vp, C.POINTER(_vp)]),
    "osc_mxfp8_weights_destroy": (_i, [_vp]),
    "osc_mxfp8_act_sizes": (_i, [_vp, _i, C.POINTER(Mxfp8ActSizes)]),
    "osc_mxfp8_quantize": (_i, [_vp, _i, _i, _i64, _vp, _vp, _vp]),
    "osc_mxfp8_gemm": (_i, [_vp, _vp, _vp, _i, _vp, _i64, _vp]),
    "osc_mxfp8_linear": (_i, [_vp, _vp, _i, _i64, _vp, _i64, _vp, _sz, _vp]),
}
for _name, (_res, _args) in _SIGS.items():
    _f = getattr(_lib, _name)
    _f.restype = _res
    _f.argtypes = _args

EXPORTS = tuple(_SIGS)


def osc_last_error() -> str:
    return _lib.osc_last_error().decode()


def osc_status_string(s: int) -> str:
    return _lib.osc_status_string(s).decode()


def _check(status: int):
    if status != OSC_OK:
        raise OscError(status, osc_last_error())


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        return t.data_ptr() if t.numel() > 0 else None
    return int(t)


_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)
_raw_device = getattr(torch._C, "_cuda_getDevice", None)


def _stream(stream=None):
    """cudaStream_t of `stream`, or of torch's current stream.  Building a torch.cuda.Stream object for the current
    stream costs ~3 us per call, a third of a few-row linear; torch's raw accessor gives the handle directly."""
    if stream is not None:
        return stream.cuda_stream
    if _raw_stream is not None and _raw_device is not None:
        return _raw_stream(_raw_device())
    return torch.cuda.current_stream().cuda_stream


def _lut(lut):
    lut = np.ascontiguousarray(lut, dtype=np.int8)
    if lut.ndim == 1:
        lut = lut.reshape(-1, 1)
    return lut


def osc_sync_check(stream=None):
    _check(_lib.osc_sync_check(_stream(stream)))


def osc_weight_sizes(E: int, N: int, K: int, lut) -> WeightSizes:
    lut = _lut(lut)
    out = WeightSizes()
    _check(_lib.osc_weight_sizes(E, N, K, lut.ctypes.data, lut.shape[1], C.byref(out)))
    return out


class _Handle:
    _destroy = None

    def __init__(self, ptr, keep):
        self.ptr = ptr
        self.keep = keep  # device buffers the handle borrows

    def close(self):
        if self.ptr:
            self._destroy(self.ptr)
            self.ptr = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class OscWeights(_Handle):
    _destroy = staticmethod(_lib.osc_weights_destroy)


class Fp8Weights(_Handle):
    _destroy = staticmethod(_lib.osc_fp8_weights_destroy)


class Mxfp8Weights(_Handle):
    _destroy = staticmethod(_lib.osc_mxfp8_weights_destroy)


def _alloc(nbytes, dev):
    return torch.empty(max(int(nbytes), 16), dtype=torch.uint8, device=dev)


def osc_prepare_weights(W: torch.Tensor, lut, stream=None) -> OscWeights:
    """W: cuda bf16 [N, K] (row stride = ldw). Returns a handle owning wq/sfw/wo/meta."""
    N, K = W.shape
    lut = _lut(lut)
    sz = osc_weight_sizes(1, N, K, lut)
    dev = W.device
    bufs = {k: _alloc(getattr(sz, k + "_bytes"), dev) for k in ("wq", "sfw", "wo", "meta")}
    h = _vp()
    _check(_lib.osc_prepare_weights(_ptr(W), N, K, W.stride(0), lut.ctypes.data, lut.shape[1], _ptr(bufs["wq"]),
                                    _ptr(bufs["sfw"]), _ptr(bufs["wo"]) if sz.wo_bytes else None, _ptr(bufs["meta"]),
                                    _stream(stream), C.byref(h)))
    w = OscWeights(h.value, bufs)
    w.E, w.N, w.K, w.K_o, w.K_o_pad, w.sizes = 1, N, K, sz.K_o, sz.K_o_pad, sz
    return w


def osc_prepare_weights_grouped(W: torch.Tensor, lut, stream=None) -> OscWeights:
    """W: cuda bf16 [E, N, K] contiguous."""
    E, N, K = W.shape
    assert W.is_contiguous()
    lut = _lut(lut)
    sz = osc_weight_sizes(E, N, K, lut)
    dev = W.device
    bufs = {k: _alloc(getattr(sz, k + "_bytes"), dev) for k in ("wq", "sfw", "wo", "meta")}
    h = _vp()
    _check(_lib.osc_prepare_weights_grouped(_ptr(W), E, N, K, lut.ctypes.data, lut.shape[1], _ptr(bufs["wq"]),
                                            _ptr(bufs["sfw"]), _ptr(bufs["wo"]) if sz.wo_bytes else None,
                                            _ptr(bufs["meta"]), _stream(stream), C.byref(h)))
    w = OscWeights(h.value, bufs)
    w.E, w.N, w.K, w.K_o, w.K_o_pad, w.sizes = E, N, K, sz.K_o, sz.K_o_pad, sz
    return w


def osc_weights_destroy(w: OscWeights):
    w.close()


def osc_act_sizes(w: OscWeights, M: int) -> ActSizes:
    out = ActSizes()
    _check(_lib.osc_act_sizes(w.ptr, M, C.byref(out)))
    return out


def osc_quantize_extract(w: OscWeights, X: torch.Tensor, xq, sfa, xo, stream=None):
    M = X.shape[0]
    _check(_lib.osc_quantize_extract(w.ptr, _ptr(X), M, X.stride(0) if M else w.K, _ptr(xq), _ptr(sfa),
                                     _ptr(xo) if w.K_o_pad else None, _stream(stream)))


def osc_gemm_dual(w: OscWeights, xq, sfa, xo, M: int, Y: torch.Tensor, stream=None):
    _check(_lib.osc_gemm_dual(w.ptr, _ptr(xq), _ptr(sfa), _ptr(xo) if w.K_o_pad else None, M, _ptr(Y),
                              Y.stride(0) if M else w.N, _stream(stream)))


def osc_linear(w: OscWeights, X: torch.Tensor, Y: torch.Tensor, workspace: torch.Tensor, stream=None):
    M = X.shape[0]
    _check(_lib.osc_linear(w.ptr, _ptr(X), M, X.stride(0) if M else w.K, _ptr(Y), Y.stride(0) if M else w.N,
                           _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)))


def osc_linear_static(w: OscWeights, X: torch.Tensor, Y: torch.Tensor, stream=None):
    """osc_linear for callers that cannot provide a workspace: the scratch is a fixed array inside the
    library (limited size, shared by all calls on a device); nothing is allocated here or in the library."""
    M = X.shape[0]
    _check(_lib.osc_linear_static(w.ptr, _ptr(X), M, X.stride(0) if M else w.K, _ptr(Y), Y.stride(0) if M else w.N,
                                  _stream(stream)))


def osc_gather_workspace_bytes(w: OscWeights, T: int, M_total: int) -> int:
    out = _sz()
    _check(_lib.osc_gather_workspace_bytes(w.ptr, T, M_total, C.byref(out)))
    return int(out.value)


def osc_linear_grouped_gather(w: OscWeights, X: torch.Tensor, row_token: torch.Tensor, off: torch.Tensor, Y: torch.Tensor,
                              workspace: torch.Tensor, stream=None):
    """Grouped linear on X[row_token] without materialising it: tokens quantized once, quantized rows gathered."""
    T, M = X.shape[0], row_token.shape[0]
    _check(_lib.osc_linear_grouped_gather(w.ptr, _ptr(X), T, X.stride(0) if T else w.K, _ptr(row_token), _ptr(off), M,
                                          _ptr(Y), Y.stride(0) if M else w.N, _ptr(workspace),
                                          workspace.numel() * workspace.element_size(), _stream(stream)))


def osc_rmsnorm_linear_grouped_gather(w: OscWeights, H: torch.Tensor, gamma: torch.Tensor, eps: float, row_token: torch.Tensor,
                                      off: torch.Tensor, Y: torch.Tensor, workspace: torch.Tensor, stream=None):
    """osc_linear_grouped_gather with the RMSNorm of the residual stream H fused into the quantizer."""
    T, M = H.shape[0], row_token.shape[0]
    _check(_lib.osc_rmsnorm_linear_grouped_gather(w.ptr, _ptr(H), T, H.stride(0) if T else w.K, _ptr(gamma), float(eps),
                                                  _ptr(row_token), _ptr(off), M, _ptr(Y), Y.stride(0) if M else w.N,
                                                  _ptr(workspace), workspace.numel() * workspace.element_size(),
                                                  _stream(stream)))


def osc_rmsnorm(H: torch.Tensor, gamma: torch.Tensor, eps: float, X: torch.Tensor, stream=None):
    """X = bf16(RMSNorm(H) * gamma) (statistic in double, element-wise part in fp32, one rounding to bf16):
    the unfused reference point."""
    M, K = H.shape
    _check(_lib.osc_rmsnorm(_ptr(H), M, K, H.stride(0) if M else K, _ptr(gamma), float(eps), _ptr(X),
                            X.stride(0) if M else K, _stream(stream)))


def osc_add_rmsnorm(H: torch.Tensor, R: torch.Tensor, gamma: torch.Tensor, eps: float, Hout: torch.Tensor, X: torch.Tensor,
                    stream=None):
    """Hout = bf16(H + R), X = RMSNorm(Hout) * gamma: the unfused reference point of the residual form."""
    M, K = H.shape
    _check(_lib.osc_add_rmsnorm(_ptr(H), _ptr(R), M, K, H.stride(0) if M else K, R.stride(0) if M else K, _ptr(gamma),
                                float(eps), _ptr(Hout), Hout.stride(0) if M else K, _ptr(X), X.stride(0) if M else K,
                                _stream(stream)))


def osc_add_rmsnorm_quantize_extract(w: OscWeights, H: torch.Tensor, R: torch.Tensor, gamma: torch.Tensor, eps: float,
                                     Hout: torch.Tensor, xq, sfa, xo, stream=None):
    """Residual update, RMSNorm and Algorithm 2 in one pass: Hout = bf16(H + R) is the only full-width tensor written."""
    M = H.shape[0]
    _check(_lib.osc_add_rmsnorm_quantize_extract(w.ptr, _ptr(H), _ptr(R), M, H.stride(0) if M else w.K,
                                                 R.stride(0) if M else w.K, _ptr(gamma), float(eps), _ptr(Hout),
                                                 Hout.stride(0) if M else w.K, _ptr(xq), _ptr(sfa),
                                                 _ptr(xo) if w.K_o_pad else None, _stream(stream)))


def osc_add_rmsnorm_linear(w: OscWeights, H: torch.Tensor, R: torch.Tensor, gamma: torch.Tensor, eps: float,
                           Hout: torch.Tensor, Y: torch.Tensor, workspace: torch.Tensor, stream=None):
    M = H.shape[0]
    _check(_lib.osc_add_rmsnorm_linear(w.ptr, _ptr(H), _ptr(R), M, H.stride(0) if M else w.K, R.stride(0) if M else w.K,
                                       _ptr(gamma), float(eps), _ptr(Hout), Hout.stride(0) if M else w.K, _ptr(Y),
                                       Y.stride(0) if M else w.N, _ptr(workspace),
                                       workspace.numel() * workspace.element_size(), _stream(stream)))


def osc_rmsnorm_quantize_extract(w: OscWeights, H: torch.Tensor, gamma: torch.Tensor, eps: float, xq, sfa, xo, stream=None):
    """RMSNorm fused in front of Algorithm 2: H is read once, the normalized tensor is never written."""
    M = H.shape[0]
    _check(_lib.osc_rmsnorm_quantize_extract(w.ptr, _ptr(H), M, H.stride(0) if M else w.K, _ptr(gamma), float(eps),
                                             _ptr(xq), _ptr(sfa), _ptr(xo) if w.K_o_pad else None, _stream(stream)))


def osc_rmsnorm_linear(w: OscWeights, H: torch.Tensor, gamma: torch.Tensor, eps: float, Y: torch.Tensor,
                       workspace: torch.Tensor, stream=None):
    M = H.shape[0]
    _check(_lib.osc_rmsnorm_linear(w.ptr, _ptr(H), M, H.stride(0) if M else w.K, _ptr(gamma), float(eps), _ptr(Y),
                                   Y.stride(0) if M else w.N, _ptr(workspace),
                                   workspace.numel() * workspace.element_size(), _stream(stream)))


def osc_swiglu(GU: torch.Tensor, I: int, H: torch.Tensor, stream=None):
    """H = bf16(silu(GU[:, :I]) * GU[:, I:2I]) in the library's fixed fp32 arithmetic: the unfused reference point."""
    M = GU.shape[0]
    _check(_lib.osc_swiglu(_ptr(GU), M, I, GU.stride(0) if M else 2 * I, _ptr(H), H.stride(0) if M else I, _stream(stream)))


def osc_swiglu_fp8_quantize(GU: torch.Tensor, I: int, x8, sx, stream=None):
    """SwiGLU fused in front of the per-token FP8 quantizer: the activation h is never written."""
    M = GU.shape[0]
    _check(_lib.osc_swiglu_fp8_quantize(_ptr(GU), M, I, GU.stride(0) if M else 2 * I, _ptr(x8), _ptr(sx), _stream(stream)))


def osc_swiglu_fp8_linear(w: "Fp8Weights", GU: torch.Tensor, Y: torch.Tensor, workspace: torch.Tensor, stream=None):
    M = GU.shape[0]
    _check(_lib.osc_swiglu_fp8_linear(w.ptr, _ptr(GU), M, GU.stride(0) if M else 2 * w.K, _ptr(Y),
                                      Y.stride(0) if M else w.N, _ptr(workspace),
                                      workspace.numel() * workspace.element_size(), _stream(stream)))


def osc_swiglu_fp8_linear_grouped(w: "Fp8Weights", GU: torch.Tensor, off: torch.Tensor, Y: torch.Tensor,
                                  workspace: torch.Tensor, stream=None):
    """Grouped FP8 linear on silu(gate) * up of the experts' gate|up rows, the activation never written."""
    M = GU.shape[0]
    _check(_lib.osc_swiglu_fp8_linear_grouped(w.ptr, _ptr(GU), _ptr(off), M, GU.stride(0) if M else 2 * w.K, _ptr(Y),
                                              Y.stride(0) if M else w.N, _ptr(workspace),
                                              workspace.numel() * workspace.element_size(), _stream(stream)))


def osc_linear_grouped(w: OscWeights, X: torch.Tensor, off: torch.Tensor, Y: torch.Tensor, workspace: torch.Tensor,
                       stream=None):
    M = X.shape[0]
    _check(_lib.osc_linear_grouped(w.ptr, _ptr(X), _ptr(off), M, X.stride(0) if M else w.K, _ptr(Y),
                                   Y.stride(0) if M else w.N, _ptr(workspace),
                                   workspace.numel() * workspace.element_size(), _stream(stream)))


def osc_profile_scratch_bytes(K: int) -> int:
    out = _sz()
    _check(_lib.osc_profile_scratch_bytes(K, C.byref(out)))
    return int(out.value)


def osc_profile_lut(X: torch.Tensor, alpha: float, scratch, lut, n_hit, n_total, threshold_bits, stream=None):
    """X: cuda bf16 [S, K]; outputs are cuda tensors (int8 [K/32], int32 [K/32] x2, int32/uint32 [1])."""
    S, K = X.shape
    _check(_lib.osc_profile_lut(_ptr(X), S, K, X.stride(0), float(alpha), _ptr(scratch),
                                scratch.numel() * scratch.element_size(), _ptr(lut), _ptr(n_hit), _ptr(n_total),
                                _ptr(threshold_bits), _stream(stream)))


def osc_fp8_prepare_weights(W: torch.Tensor, stream=None) -> Fp8Weights:
    N, K = W.shape
    dev = W.device
    bufs = {"w8": _alloc(N * K, dev), "sw": torch.empty(N, dtype=torch.float32, device=dev)}
    h = _vp()
    _check(_lib.osc_fp8_prepare_weights(_ptr(W), N, K, W.stride(0), _ptr(bufs["w8"]), _ptr(bufs["sw"]),
                                        _stream(stream), C.byref(h)))
    w = Fp8Weights(h.value, bufs)
    w.E, w.N, w.K = 1, N, K
    return w


def osc_fp8_prepare_weights_grouped(W: torch.Tensor, stream=None) -> Fp8Weights:
    E, N, K = W.shape
    assert W.is_contiguous()
    dev = W.device
    bufs = {"w8": _alloc(E * N * K, dev), "sw": torch.empty(E * N, dtype=torch.float32, device=dev)}
    h = _vp()
    _check(_lib.osc_fp8_prepare_weights_grouped(_ptr(W), E, N, K, _ptr(bufs["w8"]), _ptr(bufs["sw"]),
                                                _stream(stream), C.byref(h)))
    w = Fp8Weights(h.value, bufs)
    w.E, w.N, w.K = E, N, K
    return w


def osc_fp8_weights_destroy(w: Fp8Weights):
    w.close()


def osc_fp8_act_sizes(w: Fp8Weights, M: int) -> Fp8ActSizes:
    out = Fp8ActSizes()
    _check(_lib.osc_fp8_act_sizes(w.ptr, M, C.byref(out)))
    return out


def osc_fp8_quantize(X: torch.Tensor, x8, sx, stream=None):
    M, K = X.shape
    _check(_lib.osc_fp8_quantize(_ptr(X), M, K, X.stride(0) if M else K, _ptr(x8), _ptr(sx), _stream(stream)))


def osc_fp8_gemm(w: Fp8Weights, x8, sx, M: int, Y: torch.Tensor, stream=None):
    _check(_lib.osc_fp8_gemm(w.ptr, _ptr(x8), _ptr(sx), M, _ptr(Y), Y.stride(0) if M else w.N, _stream(stream)))


def osc_fp8_linear(w: Fp8Weights, X: torch.Tensor, Y: torch.Tensor, workspace: torch.Tensor, stream=None):
    M = X.shape[0]
    _check(_lib.osc_fp8_linear(w.ptr, _ptr(X), M, X.stride(0) if M else w.K, _ptr(Y), Y.stride(0) if M else w.N,
                               _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)))


def osc_fp8_linear_grouped(w: Fp8Weights, X: torch.Tensor, off: torch.Tensor, Y: torch.Tensor,
                           workspace: torch.Tensor, stream=None):
    M = X.shape[0]
    _check(_lib.osc_fp8_linear_grouped(w.ptr, _ptr(X), _ptr(off), M, X.stride(0) if M else w.K, _ptr(Y),
                                       Y.stride(0) if M else w.N, _ptr(workspace),
                                       workspace.numel() * workspace.element_size(), _stream(stream)))


# ------------------------------------------------------------- MXFP8 form of the fallback

def osc_mxfp8_weight_sizes(E: int, N: int, K: int) -> Mxfp8WeightSizes:
    out = Mxfp8WeightSizes()
    _check(_lib.osc_mxfp8_weight_sizes(E, N, K, C.byref(out)))
    return out


def osc_mxfp8_prepare_weights(W: torch.Tensor, stream=None) -> Mxfp8Weights:
    N, K = W.shape
    sz = osc_mxfp8_weight_sizes(1, N, K)
    bufs = {"w8": _alloc(sz.w8_bytes, W.device), "sfw": _alloc(sz.sfw_bytes, W.device)}
    h = _vp()
    _check(_lib.osc_mxfp8_prepare_weights(_ptr(W), N, K, W.stride(0), _ptr(bufs["w8"]), _ptr(bufs["sfw"]),
                                          _stream(stream), C.byref(h)))
    w = Mxfp8Weights(h.value, bufs)
    w.E, w.N, w.K, w.sizes = 1, N, K, sz
    return w


def osc_mxfp8_prepare_weights_grouped(W: torch.Tensor, stream=None) -> Mxfp8Weights:
    E, N, K = W.shape
    assert W.is_contiguous()
    sz = osc_mxfp8_weight_sizes(E, N, K)
    bufs = {"w8": _alloc(sz.w8_bytes, W.device), "sfw": _alloc(sz.sfw_bytes, W.device)}
    h = _vp()
    _check(_lib.osc_mxfp8_prepare_weights_grouped(_ptr(W), E, N, K, _ptr(bufs["w8"]), _ptr(bufs["sfw"]),
                                                  _stream(stream), C.byref(h)))
    w = Mxfp8Weights(h.value, bufs)
    w.E, w.N, w.K, w.sizes = E, N, K, sz
    return w


def osc_mxfp8_linear_grouped(w: Mxfp8Weights, X: torch.Tensor, off: torch.Tensor, Y: torch.Tensor,
                             workspace: torch.Tensor, stream=None):
    M = X.shape[0]
    _check(_lib.osc_mxfp8_linear_grouped(w.ptr, _ptr(X), _ptr(off), M, X.stride(0) if M else w.K, _ptr(Y),
                                         Y.stride(0) if M else w.N, _ptr(workspace),
                                         workspace.numel() * workspace.element_size(), _stream(stream)))


def osc_mxfp8_weights_destroy(w: Mxfp8Weights):
    w.close()


def osc_mxfp8_act_sizes(w: Mxfp8Weights, M: int) -> Mxfp8ActSizes:
    out = Mxfp8ActSizes()
    _check(_lib.osc_mxfp8_act_sizes(w.ptr, M, C.byref(out)))
    return out


def osc_mxfp8_quantize(X: torch.Tensor, x8, sfa, stream=None):
    M, K = X.shape
    _check(_lib.osc_mxfp8_quantize(_ptr(X), M, K, X.stride(0) if M else K, _ptr(x8), _ptr(sfa), _stream(stream)))


def osc_mxfp8_gemm(w: Mxfp8Weights, x8, sfa, M: int, Y: torch.Tensor, stream=None):
    _check(_lib.osc_mxfp8_gemm(w.ptr, _ptr(x8), _ptr(sfa), M, _ptr(Y), Y.stride(0) if M else w.N, _stream(stream)))


def osc_mxfp8_linear(w: Mxfp8Weights, X: torch.Tensor, Y: torch.Tensor, workspace: torch.Tensor, stream=None):
    M = X.shape[0]
    _check(_lib.osc_mxfp8_linear(w.ptr, _ptr(X), M, X.stride(0) if M else w.K, _ptr(Y), Y.stride(0) if M else w.N,
                                 _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)))


# ------------------------------------------- dynamic-protection control group (a baseline)

def osc_dyn_weight_sizes(N: int, K: int) -> WeightSizes:
    out = WeightSizes()
    _check(_lib.osc_dyn_weight_sizes(N, K, C.byref(out)))
    return out


def osc_dyn_prepare_weights(W: torch.Tensor, stream=None) -> OscWeights:
    N, K = W.shape
    sz = osc_dyn_weight_sizes(N, K)
    bufs = {k: _alloc(getattr(sz, k + "_bytes"), W.device) for k in ("wq", "sfw", "wo", "meta")}
    h = _vp()
    _check(_lib.osc_dyn_prepare_weights(_ptr(W), N, K, W.stride(0), _ptr(bufs["wq"]), _ptr(bufs["sfw"]),
                                        _ptr(bufs["wo"]), _ptr(bufs["meta"]), _stream(stream), C.byref(h)))
    w = OscWeights(h.value, bufs)
    w.E, w.N, w.K, w.K_o, w.K_o_pad, w.sizes = 1, N, K, K, K, sz
    return w


def osc_dyn_act_sizes(w: OscWeights, M: int) -> DynActSizes:
    out = DynActSizes()
    _check(_lib.osc_dyn_act_sizes(w.ptr, M, C.byref(out)))
    return out


def osc_dyn_quantize_extract(w: OscWeights, X: torch.Tensor, xq, sfa, xo, idx, val, stream=None):
    M = X.shape[0]
    _check(_lib.osc_dyn_quantize_extract(w.ptr, _ptr(X), M, X.stride(0) if M else w.K, _ptr(xq), _ptr(sfa), _ptr(xo),
                                         _ptr(idx), _ptr(val), _stream(stream)))


def osc_dyn_linear(w: OscWeights, X: torch.Tensor, Y: torch.Tensor, workspace: torch.Tensor, stream=None):
    M = X.shape[0]
    _check(_lib.osc_dyn_linear(w.ptr, _ptr(X), M, X.stride(0) if M else w.K, _ptr(Y), Y.stride(0) if M else w.N,
                               _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)))


# --------------------------------------------------------------- NVFP4 / G = 16 variant

def _lut16(lut, K):
    lut = np.ascontiguousarray(lut, dtype=np.int8)
    return lut.reshape(K // 16, -1)


def osc_nvfp4_weight_sizes(N: int, K: int, lut16) -> WeightSizes:
    lut16 = _lut16(lut16, K)
    out = WeightSizes()
    _check(_lib.osc_nvfp4_weight_sizes(N, K, lut16.ctypes.data, lut16.shape[1], C.byref(out)))
    return out


def osc_nvfp4_prepare_weights(W: torch.Tensor, lut16, ew: int, stream=None) -> OscWeights:
    N, K = W.shape
    lut16 = _lut16(lut16, K)
    sz = osc_nvfp4_weight_sizes(N, K, lut16)
    bufs = {k: _alloc(getattr(sz, k + "_bytes"), W.device) for k in ("wq", "sfw", "wo", "meta")}
    h = _vp()
    _check(_lib.osc_nvfp4_prepare_weights(_ptr(W), N, K, W.stride(0), lut16.ctypes.data, lut16.shape[1], int(ew),
                                          _ptr(bufs["wq"]), _ptr(bufs["sfw"]), _ptr(bufs["wo"]) if sz.wo_bytes else None,
                                          _ptr(bufs["meta"]), _stream(stream), C.byref(h)))
    w = OscWeights(h.value, bufs)
    w.E, w.N, w.K, w.K_o, w.K_o_pad, w.sizes, w.ew = 1, N, K, sz.K_o, sz.K_o_pad, sz, int(ew)
    return w


def osc_nvfp4_prepare_weights_grouped(W: torch.Tensor, lut16, ew: int, stream=None) -> OscWeights:
    """W: cuda bf16 [E, N, K] contiguous; one table and one tensor exponent for all experts."""
    E, N, K = W.shape
    assert W.is_contiguous()
    lut16 = _lut16(lut16, K)
    sz = WeightSizes()
    _check(_lib.osc_nvfp4_weight_sizes_grouped(E, N, K, lut16.ctypes.data, lut16.shape[1], C.byref(sz)))
    bufs = {k: _alloc(getattr(sz, k + "_bytes"), W.device) for k in ("wq", "sfw", "wo", "meta")}
    h = _vp()
    _check(_lib.osc_nvfp4_prepare_weights_grouped(_ptr(W), E, N, K, lut16.ctypes.data, lut16.shape[1], int(ew),
                                                  _ptr(bufs["wq"]), _ptr(bufs["sfw"]),
                                                  _ptr(bufs["wo"]) if sz.wo_bytes else None, _ptr(bufs["meta"]),
                                                  _stream(stream), C.byref(h)))
    w = OscWeights(h.value, bufs)
    w.E, w.N, w.K, w.K_o, w.K_o_pad, w.sizes, w.ew = E, N, K, sz.K_o, sz.K_o_pad, sz, int(ew)
    return w


def osc_nvfp4_linear_grouped(w: OscWeights, X: torch.Tensor, off: torch.Tensor, ex: int, Y: torch.Tensor,
                             workspace: torch.Tensor, stream=None):
    M = X.shape[0]
    _check(_lib.osc_nvfp4_linear_grouped(w.ptr, _ptr(X), _ptr(off), M, X.stride(0) if M else w.K, int(ex), _ptr(Y),
                                         Y.stride(0) if M else w.N, _ptr(workspace),
                                         workspace.numel() * workspace.element_size(), _stream(stream)))


def osc_nvfp4_act_sizes(w: OscWeights, M: int) -> ActSizes:
    out = ActSizes()
    _check(_lib.osc_nvfp4_act_sizes(w.ptr, M, C.byref(out)))
    return out


def osc_nvfp4_quantize_extract(w: OscWeights, X: torch.Tensor, ex: int, xq, sfa, xo, stream=None):
    M = X.shape[0]
    _check(_lib.osc_nvfp4_quantize_extract(w.ptr, _ptr(X), M, X.stride(0) if M else w.K, int(ex), _ptr(xq), _ptr(sfa),
                                           _ptr(xo) if w.K_o_pad else None, _stream(stream)))


def osc_nvfp4_gemm(w: OscWeights, xq, sfa, xo, M: int, ex: int, Y: torch.Tensor, stream=None):
    _check(_lib.osc_nvfp4_gemm(w.ptr, _ptr(xq), _ptr(sfa), _ptr(xo) if w.K_o_pad else None, M, int(ex), _ptr(Y),
                               Y.stride(0) if M else w.N, _stream(stream)))


def osc_nvfp4_linear(w: OscWeights, X: torch.Tensor, ex: int, Y: torch.Tensor, workspace: torch.Tensor, stream=None):
    M = X.shape[0]
    _check(_lib.osc_nvfp4_linear(w.ptr, _ptr(X), M, X.stride(0) if M else w.K, int(ex), _ptr(Y),
                                 Y.stride(0) if M else w.N, _ptr(workspace),
                                 workspace.numel() * workspace.element_size(), _stream(stream)))


def osc_nvfp4_rmsnorm_quantize_extract(w: OscWeights, H: torch.Tensor, gamma: torch.Tensor, eps: float, ex: int, xq, sfa, xo,
                                       stream=None):
    M = H.shape[0]
    _check(_lib.osc_nvfp4_rmsnorm_quantize_extract(w.ptr, _ptr(H), M, H.stride(0) if M else w.K, _ptr(gamma), float(eps),
                                                   int(ex), _ptr(xq), _ptr(sfa), _ptr(xo) if w.K_o_pad else None,
                                                   _stream(stream)))


def osc_nvfp4_rmsnorm_linear(w: OscWeights, H: torch.Tensor, gamma: torch.Tensor, eps: float, ex: int, Y: torch.Tensor,
                             workspace: torch.Tensor, stream=None):
    M = H.shape[0]
    _check(_lib.osc_nvfp4_rmsnorm_linear(w.ptr, _ptr(H), M, H.stride(0) if M else w.K, _ptr(gamma), float(eps), int(ex),
                                         _ptr(Y), Y.stride(0) if M else w.N, _ptr(workspace),
                                         workspace.numel() * workspace.element_size(), _stream(stream)))


def osc_nvfp4_gather_workspace_bytes(w: OscWeights, T: int, M_total: int) -> int:
    out = _sz()
    _check(_lib.osc_nvfp4_gather_workspace_bytes(w.ptr, T, M_total, C.byref(out)))
    return int(out.value)


def osc_nvfp4_linear_grouped_gather(w: OscWeights, X: torch.Tensor, row_token: torch.Tensor, off: torch.Tensor, ex: int,
                                    Y: torch.Tensor, workspace: torch.Tensor, stream=None):
    T, M = X.shape[0], row_token.shape[0]
    _check(_lib.osc_nvfp4_linear_grouped_gather(w.ptr, _ptr(X), T, X.stride(0) if T else w.K, _ptr(row_token), _ptr(off), M,
                                                int(ex), _ptr(Y), Y.stride(0) if M else w.N, _ptr(workspace),
                                                workspace.numel() * workspace.element_size(), _stream(stream)))


def osc_nvfp4_rmsnorm_linear_grouped_gather(w: OscWeights, H: torch.Tensor, gamma: torch.Tensor, eps: float,
                                            row_token: torch.Tensor, off: torch.Tensor, ex: int, Y: torch.Tensor,
                                            workspace: torch.Tensor, stream=None):
    T, M = H.shape[0], row_token.shape[0]
    _check(_lib.osc_nvfp4_rmsnorm_linear_grouped_gather(w.ptr, _ptr(H), T, H.stride(0) if T else w.K, _ptr(gamma), float(eps),
                                                        _ptr(row_token), _ptr(off), M, int(ex), _ptr(Y),
                                                        Y.stride(0) if M else w.N, _ptr(workspace),
                                                        workspace.numel() * workspace.element_size(), _stream(stream)))


def osc_prepare_weights_gate_up(W: torch.Tensor, lut, stream=None) -> OscWeights:
    """W: cuda bf16 [2I, K], gate rows above up rows.  A dense OSC handle that also serves osc_linear_swiglu."""
    N, K = W.shape
    I = N // 2
    lut = _lut(lut)
    sz = WeightSizes()
    _check(_lib.osc_gate_up_weight_sizes(I, K, lut.ctypes.data, lut.shape[1], C.byref(sz)))
    bufs = {k: _alloc(getattr(sz, k + "_bytes"), W.device) for k in ("wq", "sfw", "wo", "meta")}
    h = _vp()
    _check(_lib.osc_prepare_weights_gate_up(_ptr(W), I, K, W.stride(0), lut.ctypes.data, lut.shape[1], _ptr(bufs["wq"]),
                                            _ptr(bufs["sfw"]), _ptr(bufs["wo"]) if sz.wo_bytes else None, _ptr(bufs["meta"]),
                                            _stream(stream), C.byref(h)))
    w = OscWeights(h.value, bufs)
    w.E, w.N, w.K, w.K_o, w.K_o_pad, w.sizes = 1, N, K, sz.K_o, sz.K_o_pad, sz
    return w


def osc_linear_swiglu_workspace_bytes(w: OscWeights, M: int) -> int:
    out = _sz()
    _check(_lib.osc_linear_swiglu_workspace_bytes(w.ptr, M, C.byref(out)))
    return int(out.value)


def osc_linear_swiglu(w: OscWeights, X: torch.Tensor, H: torch.Tensor, workspace: torch.Tensor, stream=None):
    """H [M, I] = silu(gate) * up of the gate|up projection of X, the activation applied in the GEMM epilogue."""
    M = X.shape[0]
    _check(_lib.osc_linear_swiglu(w.ptr, _ptr(X), M, X.stride(0) if M else w.K, _ptr(H), H.stride(0) if M else w.N // 2,
                                  _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)))


def osc_rmsnorm_linear_swiglu(w: OscWeights, Hin: torch.Tensor, gamma: torch.Tensor, eps: float, H: torch.Tensor,
                              workspace: torch.Tensor, stream=None):
    M = Hin.shape[0]
    _check(_lib.osc_rmsnorm_linear_swiglu(w.ptr, _ptr(Hin), M, Hin.stride(0) if M else w.K, _ptr(gamma), float(eps), _ptr(H),
                                          H.stride(0) if M else w.N // 2, _ptr(workspace),
                                          workspace.numel() * workspace.element_size(), _stream(stream)))


def osc_prepare_weights_gate_up_grouped(W: torch.Tensor, lut, stream=None) -> OscWeights:
    """W: cuda bf16 [E, 2I, K] contiguous, every expert's gate rows above its up rows."""
    E, N, K = W.shape
    assert W.is_contiguous()
    lut = _lut(lut)
    sz = WeightSizes()
    _check(_lib.osc_gate_up_weight_sizes_grouped(E, N // 2, K, lut.ctypes.data, lut.shape[1], C.byref(sz)))
    bufs = {k: _alloc(getattr(sz, k + "_bytes"), W.device) for k in ("wq", "sfw", "wo", "meta")}
    h = _vp()
    _check(_lib.osc_prepare_weights_gate_up_grouped(_ptr(W), E, N // 2, K, lut.ctypes.data, lut.shape[1], _ptr(bufs["wq"]),
                                                    _ptr(bufs["sfw"]), _ptr(bufs["wo"]) if sz.wo_bytes else None,
                                                    _ptr(bufs["meta"]), _stream(stream), C.byref(h)))
    w = OscWeights(h.value, bufs)
    w.E, w.N, w.K, w.K_o, w.K_o_pad, w.sizes = E, N, K, sz.K_o, sz.K_o_pad, sz
    return w


def osc_linear_swiglu_grouped(w: OscWeights, X: torch.Tensor, off: torch.Tensor, H: torch.Tensor, workspace: torch.Tensor,
                              stream=None):
    M = X.shape[0]
    _check(_lib.osc_linear_swiglu_grouped(w.ptr, _ptr(X), _ptr(off), M, X.stride(0) if M else w.K, _ptr(H),
                                          H.stride(0) if M else w.N // 2, _ptr(workspace),
                                          workspace.numel() * workspace.element_size(), _stream(stream)))


def osc_swiglu_gather_workspace_bytes(w: OscWeights, T: int, M_total: int) -> int:
    out = _sz()
    _check(_lib.osc_swiglu_gather_workspace_bytes(w.ptr, T, M_total, C.byref(out)))
    return int(out.value)


def osc_linear_swiglu_grouped_gather(w: OscWeights, X: torch.Tensor, row_token: torch.Tensor, off: torch.Tensor, H: torch.Tensor,
                                     workspace: torch.Tensor, stream=None):
    T, M = X.shape[0], row_token.shape[0]
    _check(_lib.osc_linear_swiglu_grouped_gather(w.ptr, _ptr(X), T, X.stride(0) if T else w.K, _ptr(row_token), _ptr(off), M,
                                                 _ptr(H), H.stride(0) if M else w.N // 2, _ptr(workspace),
                                                 workspace.numel() * workspace.element_size(), _stream(stream)))


def osc_rmsnorm_linear_swiglu_grouped_gather(w: OscWeights, Hin: torch.Tensor, gamma: torch.Tensor, eps: float,
                                             row_token: torch.Tensor, off: torch.Tensor, H: torch.Tensor, workspace: torch.Tensor,
                                             stream=None):
    T, M = Hin.shape[0], row_token.shape[0]
    _check(_lib.osc_rmsnorm_linear_swiglu_grouped_gather(w.ptr, _ptr(Hin), T, Hin.stride(0) if T else w.K, _ptr(gamma),
                                                         float(eps), _ptr(row_token), _ptr(off), M, _ptr(H),
                                                         H.stride(0) if M else w.N // 2, _ptr(workspace),
                                                         workspace.numel() * workspace.element_size(), _stream(stream)))
