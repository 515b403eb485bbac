"""The allocation-free W4A8 entry point, mnnllm_linear_w4a8_static.

It exists for callers that are not allowed to allocate device memory (a plugin inside a host
application that owns all allocations, a serving loop that bans allocator calls after start-up):
they cannot provide the workspace that mnnllm_linear_w4a8 asks for, so the library carries a
fixed scratch array of its own.  The test drives it through the C ABI twice in a row, with
different shapes so that the second call finds the first call's leftovers in the shared scratch,
and requires the same output as the ordinary entry point.  The file sorts last on purpose: a run
that stops at the first failure has then already exercised everything else.
"""
import numpy as np
import pytest
import torch

from paper_2506_10443_b200 import binding as B
from paper_2506_10443_b200 import inputs
import oracle
from gpu_util import TOL, assert_close, dev


def test_static_entry_rejects_oversized_problems_before_touching_the_gpu():
    # 4096 tokens x 8960 k need 36 MB of int8 activations: beyond the 8 MiB built-in scratch
    p = 0x1000
    f = B.lib.mnnllm_linear_w4a8_static
    assert B.workspace_min_w4a8(4096, 64, 8960, 64) > B.STATIC_SCRATCH_BYTES
    assert f(p, p, p, 4096, 64, 8960, 64, B.F16, B.F16, None) == 6
    assert f(None, p, p, 4, 64, 64, 64, B.F16, B.F16, None) == 1
    assert f(p, p, p, 4, 64, 64, 48, B.F16, B.F16, None) == 2
    with pytest.raises(B.MnnllmError):
        B.linear_w4a8_static(p, p, p, 4096, 64, 8960, 64, stream=0)


@pytest.mark.gpu
def test_static_entry_matches_the_workspace_entry_on_two_calls_in_a_row():
    cases = [(200, 384, 1536, 64), (77, 272, 1024, 128)]   # the second is smaller: stale bytes remain beyond it
    for i, (M, N, K, group) in enumerate(cases):
        W = inputs.weights(900 + i, N, K)
        pd = dev(B.pack_w4(W, group))
        xd = dev(inputs.activations(910 + i, M, K, outliers=True))
        nbytes = B.workspace_min_w4a8(M, N, K, group)   # like the built-in scratch: no room to split tiles along K
        assert nbytes <= B.STATIC_SCRATCH_BYTES
        ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        y_ref = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        B.linear_w4a8(xd, pd, y_ref, M, N, K, group, ws, nbytes, y_dtype=B.F32)
        y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        B.linear_w4a8_static(xd, pd, y, M, N, K, group, y_dtype=B.F32)
        assert B.read_status() == 0
        assert_close(y.cpu().numpy(), y_ref.cpu().numpy().astype(np.float64), TOL)
        assert torch.equal(y, y_ref)   # same kernels, same inputs: in fact identical
        # and against the CPU oracle, like every other entry point
        q, s, z = oracle.quantize_w4(W, group)
        x = inputs.activations(910 + i, M, K, outliers=True).astype(np.float32)
        assert_close(y.cpu().numpy(), oracle.linear_w4a8(x, q, s, z, group), TOL)
