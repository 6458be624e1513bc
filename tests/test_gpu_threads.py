"""Host threads: distinct handles on distinct streams, called from several threads at once.

ctypes releases the interpreter lock for the duration of a foreign call, so the calls below do run inside the
library at the same time (validation, kernel selection, tensor-map encoding, launches).  Every thread must get,
bit for bit, what the same call gives when it runs alone.
"""
import threading

import numpy as np
import pytest
import torch

from paper_2604_12782_b200 import synth

pytestmark = pytest.mark.gpu

from gpu_util import assert_within_tolerance, dev_bf16, host_bf16_bits, host_f64, poison  # noqa: E402


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_12782_b200 import binding
    return binding


SHAPES = [(16, 512, 256, "osc"), (200, 1024, 320, "osc"), (700, 512, 512, "fp8"), (1300, 768, 448, "osc"),
          (64, 2048, 128, "mxfp8"), (3000, 256, 192, "fp8")]


def make_job(B, seed, M, K, N, kind):
    if kind == "osc":
        c = synth.osc_linear_case(seed, M, K, N, 2)
        w = B.osc_prepare_weights(dev_bf16(c["W"]), c["lut"])
        ws = poison(B.osc_act_sizes(w, M).workspace_bytes)
        call = B.osc_linear
    elif kind == "fp8":
        c = synth.fp8_linear_case(seed, M, K, N)
        w = B.osc_fp8_prepare_weights(dev_bf16(c["W"]))
        ws = poison(B.osc_fp8_act_sizes(w, M).workspace_bytes)
        call = B.osc_fp8_linear
    else:
        c = synth.fp8_linear_case(seed, M, K, N)
        w = B.osc_mxfp8_prepare_weights(dev_bf16(c["W"]))
        ws = poison(B.osc_mxfp8_act_sizes(w, M).workspace_bytes)
        call = B.osc_mxfp8_linear
    return {"c": c, "w": w, "ws": ws, "call": call, "X": dev_bf16(c["X"]), "kind": kind, "M": M, "N": N}


def test_concurrent_calls_from_host_threads(B, oracle):
    jobs = [make_job(B, 40 + i, *s) for i, s in enumerate(SHAPES)]
    alone = []
    for j in jobs:                       # each call on its own, default stream
        Y = torch.full((j["M"], j["N"]), float("nan"), dtype=torch.bfloat16, device="cuda")
        j["call"](j["w"], j["X"], Y, j["ws"])
        B.osc_sync_check()
        alone.append(host_bf16_bits(Y))
    # the first one also against the oracle, so that "alone" is not only compared with itself
    c = jobs[0]["c"]
    Yref, T, *_ = oracle.linear(c["X"], c["W"], c["lut"])
    assert_within_tolerance(host_f64(dev_bf16(alone[0])), Yref, T, "single call")

    torch.cuda.synchronize()
    rounds = 25
    errors, outs = [], [None] * len(jobs)
    start = threading.Barrier(len(jobs))

    def worker(i):
        try:
            j = jobs[i]
            st = torch.cuda.Stream()
            Ys = [torch.full((j["M"], j["N"]), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(rounds)]
            torch.cuda.synchronize()
            start.wait()
            with torch.cuda.stream(st):
                for Y in Ys:
                    j["call"](j["w"], j["X"], Y, j["ws"], stream=st)
            st.synchronize()
            outs[i] = [host_bf16_bits(Y) for Y in Ys]
        except Exception as e:           # reported by the main thread
            errors.append((i, repr(e)))

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(len(jobs))]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    B.osc_sync_check()
    for i, ys in enumerate(outs):
        for r, y in enumerate(ys):
            assert np.array_equal(y, alone[i]), f"job {i} ({SHAPES[i]}), round {r}: differs from the call made alone"
