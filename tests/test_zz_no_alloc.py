"""osc_linear_static: the workspace-free variant of osc_linear.

Some users of the library cannot hand it scratch memory (a plug-in that only receives input and output
pointers from its host, or a path on which allocating is forbidden because it would synchronise the
device).  For them the library keeps the scratch in a fixed array of its own.  This test calls that entry
point through the C ABI twice in a row - the second time on a smaller, different problem, so that whatever the
first call left in the shared array would show - and checks both results against osc_linear with a caller
workspace.  It is collected last on purpose: a failure here must not hide the other GPU tests in a run that
stops at the first failure.
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


def test_static_scratch_matches_workspace_path_on_two_calls(B, oracle):
    base = synth.osc_linear_case(11, 300, 1024, 320, 2)
    w = B.osc_prepare_weights(dev_bf16(base["W"]), base["lut"])
    for M, seed in ((300, 11), (37, 12)):           # second call: fewer rows, other data, same weights
        Xb, _ = synth.osc_activations_only(seed, M, 1024, 2)
        X = dev_bf16(Xb)
        sz = B.osc_act_sizes(w, M)
        assert sz.workspace_bytes <= 4 * 1024 * 1024
        Y_ref = torch.full((M, 320), float("nan"), dtype=torch.bfloat16, device="cuda")
        B.osc_linear(w, X, Y_ref, poison(sz.workspace_bytes))
        Y = torch.full((M, 320), float("nan"), dtype=torch.bfloat16, device="cuda")
        B.osc_linear_static(w, X, Y)
        B.osc_sync_check()
        # same kernels, same operands: the outputs agree well inside the GEMM tolerance of the other tests
        Yo, T, *_ = oracle.linear(Xb, base["W"], base["lut"])
        assert_within_tolerance(host_f64(Y), Yo, T, f"osc_linear_static M={M} vs oracle")
        assert_within_tolerance(host_f64(Y), host_f64(Y_ref), T, f"osc_linear_static M={M} vs osc_linear")
        assert not torch.isnan(Y.float()).any()


def test_static_scratch_rejects_oversized_problems(B):
    c = synth.osc_linear_case(3, 0, 4096, 64, 2)
    w = B.osc_prepare_weights(dev_bf16(c["W"]), c["lut"])
    M = 4096                                          # needs ~11 MB of scratch at K = 4096
    X = torch.zeros(M, 4096, dtype=torch.bfloat16, device="cuda")
    Y = torch.zeros(M, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.OscError) as e:
        B.osc_linear_static(w, X, Y)
    assert e.value.status == -5 and "osc_linear_static" in str(e.value)
    B.osc_linear_static(w, X[:0], Y[:0])              # M == 0 stays a no-op


def test_static_scratch_from_host_threads(B):
    """Several host threads call the entry point at once (ctypes drops the interpreter lock during the call), all on
    one stream as the shared scratch requires, all on the same problem so that the order in which their launches
    interleave on the stream does not matter: every result equals the one a single call gives."""
    import threading
    c = synth.osc_linear_case(21, 200, 512, 256, 2)
    w = B.osc_prepare_weights(dev_bf16(c["W"]), c["lut"])
    X = dev_bf16(c["X"])
    Y0 = torch.full((200, 256), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_linear_static(w, X, Y0)
    B.osc_sync_check()
    st = torch.cuda.Stream()
    nthreads, rounds = 4, 10
    Ys = [[torch.full((200, 256), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(rounds)]
          for _ in range(nthreads)]
    torch.cuda.synchronize()
    errors = []
    start = threading.Barrier(nthreads)

    def worker(i):
        try:
            start.wait()
            for Y in Ys[i]:
                B.osc_linear_static(w, X, Y, stream=st)
        except Exception as e:
            errors.append((i, repr(e)))

    ts = [threading.Thread(target=worker, args=(i,)) for i in range(nthreads)]
    for t in ts:
        t.start()
    for t in ts:
        t.join()
    st.synchronize()
    B.osc_sync_check()
    assert not errors, errors
    for i in range(nthreads):
        for Y in Ys[i]:
            assert torch.equal(Y.view(torch.int16), Y0.view(torch.int16))
