"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, and rejects bad arguments before touching the device."""
import ctypes as C
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    import __graft_entry__ as g
    g.build()
    from paper_2604_12782_b200 import binding
    return binding


def test_library_exports_every_declared_symbol(B):
    with open(os.path.join(ROOT, "include", "osc.h")) as f:
        text = f.read()
    declared = set(re.findall(r"\b(osc_[a-z0-9_]+)\s*\(", text))
    assert len(declared) >= 20
    lib = C.CDLL(B.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(B.EXPORTS), declared ^ set(B.EXPORTS)


def test_status_strings(B):
    assert B.osc_status_string(0) == "OSC_OK"
    assert B.osc_status_string(-3) == "OSC_ERR_LUT"
    assert B.osc_status_string(-8) == "OSC_ERR_TIMEOUT"


def test_weight_sizes_and_table_validation(B):
    lut = np.full((4096 // 32, 2), -1, np.int8)
    lut[:, 0] = 3
    lut[:, 1] = 17
    sz = B.osc_weight_sizes(1, 6144, 4096, lut)
    assert (sz.K_o, sz.K_o_pad) == (256, 256)
    assert sz.wq_bytes == 6144 * 2048 and sz.sfw_bytes == 48 * 32 * 512 and sz.wo_bytes == 6144 * 256 * 2
    lut1 = np.full((16, 1), -1, np.int8)
    lut1[3] = 9
    sz = B.osc_weight_sizes(2, 64, 512, lut1)
    assert (sz.K_o, sz.K_o_pad) == (1, 64) and sz.sfw_bytes == 2 * 1 * 4 * 512
    assert B.osc_weight_sizes(1, 64, 512, np.full((16, 1), -1, np.int8)).wo_bytes == 0

    for bad, status in [((1, 64, 500), -2), ((1, 60, 512), -2), ((0, 64, 512), -1)]:
        with pytest.raises(B.OscError) as e:
            B.osc_weight_sizes(*bad, np.full((16, 1), -1, np.int8))
        assert e.value.status == status
    dup = np.full((16, 2), 5, np.int8)
    with pytest.raises(B.OscError) as e:
        B.osc_weight_sizes(1, 64, 512, dup)
    assert e.value.status == -3 and "twice" in str(e.value)
    oob = np.full((16, 1), 32, np.int8)
    with pytest.raises(B.OscError) as e:
        B.osc_weight_sizes(1, 64, 512, oob)
    assert e.value.status == -3


def test_null_and_misaligned_arguments_launch_nothing(B):
    lib = C.CDLL(B.LIB_PATH)
    lut = np.full((4, 1), -1, np.int8)
    h = C.c_void_p()
    f = lib.osc_prepare_weights
    f.argtypes = B._SIGS["osc_prepare_weights"][1]
    assert f(None, 64, 128, 128, lut.ctypes.data, 1, None, None, None, None, None, C.byref(h)) == -1
    assert h.value is None
    # misaligned device pointer (never dereferenced: validation comes first)
    assert f(0x1008, 64, 128, 128, lut.ctypes.data, 1, 0x2000, 0x3000, None, 0x4000, None, C.byref(h)) == -4
    assert f(0x1000, 64, 128, 100, lut.ctypes.data, 1, 0x2000, 0x3000, None, 0x4000, None, C.byref(h)) == -2
    q = lib.osc_fp8_quantize
    q.argtypes = B._SIGS["osc_fp8_quantize"][1]
    assert q(0x1000, -1, 128, 128, 0x2000, 0x3000, None) == -1
    assert q(0x1000, 4, 100, 128, 0x2000, 0x3000, None) == -2
    assert q(0x1000, 0, 128, 128, None, None, None) == 0          # M == 0 is a no-op
    assert q(0x1000, 4, 128, 132, 0x2000, 0x3000, None) == -4     # ldx not a multiple of 8
    assert lib.osc_linear(None, None, 0, 0, None, 0, None, 0, None) == -1


def test_producer_fusions_validate_before_launching(B):
    """RMSNorm / SwiGLU entry points: shape, range, alignment and null checks come before any device work."""
    lib = C.CDLL(B.LIB_PATH)
    rn = lib.osc_rmsnorm
    rn.argtypes = B._SIGS["osc_rmsnorm"][1]
    assert rn(0x1000, 4, 100, 128, 0x2000, 1e-6, 0x3000, 128, None) == -2       # K not a multiple of 128
    assert rn(0x1000, 4, 8320, 8320, 0x2000, 1e-6, 0x3000, 8320, None) == -2    # a row must fit on chip: K <= 8192
    assert rn(0x1000, -1, 128, 128, 0x2000, 1e-6, 0x3000, 128, None) == -1
    assert rn(0x1000, 0, 128, 128, None, 1e-6, None, 128, None) == 0            # M == 0 is a no-op
    assert rn(0x1000, 4, 128, 128, None, 1e-6, 0x3000, 128, None) == -1         # gamma is null
    assert rn(0x1000, 4, 128, 120, 0x2000, 1e-6, 0x3000, 128, None) == -2       # ldh < K
    assert rn(0x1008, 4, 128, 128, 0x2000, 1e-6, 0x3000, 128, None) == -4
    assert rn(0x1000, 4, 128, 132, 0x2000, 1e-6, 0x3000, 128, None) == -4       # ldh not a multiple of 8
    sg = lib.osc_swiglu
    sg.argtypes = B._SIGS["osc_swiglu"][1]
    assert sg(0x1000, 4, 100, 256, 0x2000, 128, None) == -2                     # I not a multiple of 128
    assert sg(0x1000, 4, 16512, 33024, 0x2000, 16512, None) == -2               # I <= 16384
    assert sg(0x1000, 4, 128, 200, 0x2000, 128, None) == -2                     # ldg < 2 I
    assert sg(0x1000, 4, 128, 256, None, 128, None) == -1
    assert sg(0x1000, 4, 128, 256, 0x2008, 128, None) == -4
    assert sg(0x1000, 0, 128, 256, None, 128, None) == 0
    sq = lib.osc_swiglu_fp8_quantize
    sq.argtypes = B._SIGS["osc_swiglu_fp8_quantize"][1]
    assert sq(0x1000, 4, 128, 256, None, 0x3000, None) == -1
    assert sq(0x1000, 4, 128, 256, 0x2004, 0x3000, None) == -4
    assert lib.osc_rmsnorm_linear(None, None, 0, 0, None, C.c_float(0), None, 0, None, 0, None) == -1
    assert lib.osc_swiglu_fp8_linear(None, None, 0, 0, None, 0, None, 0, None) == -1


def test_grouped_fused_calls_refuse_null_handles():
    from paper_2604_12782_b200 import binding as B
    lib = B._lib
    assert lib.osc_swiglu_fp8_linear_grouped(None, None, None, 0, 0, None, 0, None, 0, None) == -1
    assert lib.osc_rmsnorm_linear_grouped_gather(None, None, 0, 0, None, C.c_float(0), None, None, 0, None, 0, None, 0,
                                                 None) == -1


def test_residual_forms_validate_before_launching():
    from paper_2604_12782_b200 import binding as B
    lib = B._lib
    f = lib.osc_add_rmsnorm
    f.argtypes = B._SIGS["osc_add_rmsnorm"][1]
    f.restype = C.c_int
    ok = dict(H=0x1000, R=0x2000, M=4, K=256, ldh=256, ldr=256, g=0x3000, eps=1e-6, Ho=0x4000, ldo=256, X=0x5000, ldx=256)

    def call(**kw):
        a = {**ok, **kw}
        return f(a["H"], a["R"], a["M"], a["K"], a["ldh"], a["ldr"], a["g"], a["eps"], a["Ho"], a["ldo"], a["X"], a["ldx"], None)
    assert call(M=0) == 0
    assert call(M=-1) == -1
    assert call(K=100) == -2 and call(K=8192 + 128, ldh=8320, ldr=8320, ldo=8320, ldx=8320) == -2
    assert call(R=None) == -1 and call(Ho=None) == -1
    assert call(ldr=128) == -2 and call(ldo=128) == -2
    assert call(ldr=260) == -4 and call(R=0x2008) == -4 and call(Ho=0x4004) == -4
    assert lib.osc_add_rmsnorm_linear(None, None, None, 0, 0, 0, None, C.c_float(0), None, 0, None, 0, None, 0, None) == -1
    assert lib.osc_add_rmsnorm_quantize_extract(None, None, None, 0, 0, 0, None, C.c_float(0), None, 0, None, None, None,
                                                None) == -1


def test_nvfp4_fused_calls_refuse_null_handles():
    from paper_2604_12782_b200 import binding as B
    lib = B._lib
    sz = C.c_size_t()
    assert lib.osc_nvfp4_rmsnorm_quantize_extract(None, None, 0, 0, None, C.c_float(0), 0, None, None, None, None) == -1
    assert lib.osc_nvfp4_rmsnorm_linear(None, None, 0, 0, None, C.c_float(0), 0, None, 0, None, 0, None) == -1
    assert lib.osc_nvfp4_gather_workspace_bytes(None, 0, 0, C.byref(sz)) == -1
    assert lib.osc_nvfp4_linear_grouped_gather(None, None, 0, 0, None, None, 0, 0, None, 0, None, 0, None) == -1
    assert lib.osc_nvfp4_rmsnorm_linear_grouped_gather(None, None, 0, 0, None, C.c_float(0), None, None, 0, 0, None, 0, None, 0,
                                                       None) == -1


def test_gate_up_calls_refuse_null_handles_and_odd_shapes():
    from paper_2604_12782_b200 import binding as B
    lib = B._lib
    sz = C.c_size_t()
    assert lib.osc_linear_swiglu(None, None, 0, 0, None, 0, None, 0, None) == -1
    assert lib.osc_linear_swiglu_grouped(None, None, None, 0, 0, None, 0, None, 0, None) == -1
    assert lib.osc_swiglu_gather_workspace_bytes(None, 0, 0, C.byref(sz)) == -1
    assert lib.osc_linear_swiglu_grouped_gather(None, None, 0, 0, None, None, 0, None, 0, None, 0, None) == -1
    assert lib.osc_rmsnorm_linear_swiglu_grouped_gather(None, None, 0, 0, None, C.c_float(0), None, None, 0, None, 0, None, 0,
                                                        None) == -1
    lut = np.full((16, 1), -1, np.int8)
    ws = B.WeightSizes()
    assert lib.osc_gate_up_weight_sizes_grouped(0, 64, 512, lut.ctypes.data, 1, C.byref(ws)) == -1     # no experts
    assert lib.osc_gate_up_weight_sizes_grouped(2, 60, 512, lut.ctypes.data, 1, C.byref(ws)) == -2     # I not a multiple of 64
    assert lib.osc_gate_up_weight_sizes_grouped(2, 64, 512, lut.ctypes.data, 1, C.byref(ws)) == 0
    assert ws.wq_bytes == 2 * 128 * 256
