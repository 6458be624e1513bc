"""Metamorphic checks on the GPU path that need no oracle: a row's outputs depend on that row and the weights only,
an output feature's on that weight row only - so permuting activation rows or weight rows permutes the outputs bit
for bit (every output element is accumulated in the same K order whatever tile it lands in), for the pair, single-CTA
and few-row kernels alike; and a second call on other data leaves no trace in the first result."""
import numpy as np
import pytest
import torch

from paper_2604_12782_b200 import synth

pytestmark = pytest.mark.gpu

from gpu_util import dev_bf16, poison  # noqa: E402


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_12782_b200 import binding
    return binding


def run(B, w, X, M, N):
    sz = B.osc_act_sizes(w, M)
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.osc_linear(w, X, Y, poison(sz.workspace_bytes))
    return Y


@pytest.mark.parametrize("M,K,N", [(24, 512, 320), (100, 512, 320), (700, 1024, 512)])   # few-row, 128-row, pair kernels
def test_row_and_feature_permutations_permute_the_outputs(B, M, K, N):
    c = synth.osc_linear_case(M, M, K, N, 2)
    rng = np.random.default_rng(M)
    X, W = dev_bf16(c["X"]), dev_bf16(c["W"])
    w = B.osc_prepare_weights(W, c["lut"])
    Y = run(B, w, X, M, N)
    pr = torch.from_numpy(rng.permutation(M)).cuda()
    assert torch.equal(run(B, w, X[pr].contiguous(), M, N), Y[pr])
    pn = torch.from_numpy(rng.permutation(N)).cuda()
    w2 = B.osc_prepare_weights(W[pn].contiguous(), c["lut"])
    assert torch.equal(run(B, w2, X, M, N), Y[:, pn])
    # rows appended behind the tensor change nothing in front of them
    X2 = torch.cat([X, X[:5] * 3], dim=0).contiguous()
    assert torch.equal(run(B, w, X2, M + 5, N)[:M], Y)
    # a call on other data in between leaves no trace
    run(B, w, (X * 0.5).contiguous(), M, N)
    assert torch.equal(run(B, w, X, M, N), Y)
    B.osc_sync_check()


def test_fp8_row_permutation(B):
    M, K, N = 300, 768, 320
    c = synth.fp8_linear_case(1, M, K, N)
    X, W = dev_bf16(c["X"]), dev_bf16(c["W"])
    w = B.osc_fp8_prepare_weights(W)
    sz = B.osc_fp8_act_sizes(w, M)

    def go(Xd):
        Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        B.osc_fp8_linear(w, Xd, Y, poison(sz.workspace_bytes))
        return Y
    Y = go(X)
    pr = torch.from_numpy(np.random.default_rng(2).permutation(M)).cuda()
    assert torch.equal(go(X[pr].contiguous()), Y[pr])
    B.osc_sync_check()
