"""GPU parity of the per-token int8 activation quantiser: bit-exact against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_10443_b200 import binding as B
from paper_2506_10443_b200 import inputs
from gpu_util import dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("M,K,group,dtype", [
    (1, 64, 64, "f16"), (3, 1536, 64, "f16"), (64, 8960, 64, "f16"), (17, 3584, 128, "f16"),
    (5, 18944, 64, "f16"), (9, 1536, 64, "bf16"),
])
def test_act_quant_bit_exact(M, K, group, dtype):
    x = inputs.activations(M * 31 + K, M, K, outliers=True, dtype=dtype)
    if dtype == "f16":
        x[0, :8] = 0 if M > 1 else x[0, :8]
        xd, x32, xdt = dev(x), x.astype(np.float32), B.F16
    else:
        xd, x32, xdt = dev(inputs.bf16_bits(x)).view(torch.bfloat16), x, B.BF16
    if M > 2:
        x32[2] = 0   # an all-zero token
        xd[2] = 0
    a_q = torch.empty((M, K), dtype=torch.int8, device="cuda")
    a_scale = torch.empty((M,), dtype=torch.float32, device="cuda")
    A = torch.empty((M, K // group), dtype=torch.int32, device="cuda")
    B.quantize_activations(xd, M, K, group, a_q, a_scale, A, x_dtype=xdt)
    torch.cuda.synchronize()
    q0, s0, A0 = oracle.act_quant(x32, group)
    assert (a_q.cpu().numpy() == q0).all()
    assert (a_scale.cpu().numpy().view(np.uint32) == s0.view(np.uint32)).all()
    assert (A.cpu().numpy() == A0).all()
