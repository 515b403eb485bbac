"""The bounded-wait / status-word path, exercised without any kernel of the library failing: a debug
kernel waits on a barrier nobody arrives at, gives up after a few tries, records a code and ends."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_10443_b200 import binding as B
from paper_2506_10443_b200 import inputs
from gpu_util import assert_close, dev, quantized

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_once_and_leaves_the_context_usable():
    assert B.read_status_code() == (0, 0)
    B.debug_wait_timeout(3)
    st, detail = B.read_status_code()
    assert st == 5 and detail == B.DEBUG_TIMEOUT_DETAIL          # MNNLLM_ERR_TIMEOUT with the kernel's code
    assert B.read_status_code() == (0, 0)                        # reading clears the word
    # the context is intact: an ordinary GEMV afterwards is still right
    N, K = 256, 1536
    W, packed, (q, s, z) = quantized(41, N, K, 64)
    x = inputs.activations(42, 1, K)
    y = torch.empty((1, N), dtype=torch.float16, device="cuda")
    B.linear_w4a16(dev(x), dev(packed), y, 1, N, K, 64)
    assert B.read_status_code() == (0, 0)
    assert_close(y.float().cpu().numpy(), oracle.linear_wa16(x.astype(np.float32), q, s, z, 64))


def test_debug_wait_argument_errors():
    assert B.lib.mnnllm_debug_wait_timeout(0, None) == 1
    assert B.lib.mnnllm_debug_wait_timeout(100000, None) == 1
