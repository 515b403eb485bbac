"""GPU parity of the weight-only decode path (W4A16, W8A16) against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_10443_b200 import binding as B
from paper_2506_10443_b200 import inputs
from gpu_util import assert_bf16_within_1ulp, assert_close, dev, quantized

pytestmark = pytest.mark.gpu


def run_w4a16(x16, packed, M, N, K, group, y_dtype=B.F16):
    tdt = {B.F16: torch.float16, B.BF16: torch.bfloat16, B.F32: torch.float32}[y_dtype]
    y = torch.full((M, N), float("nan"), dtype=tdt, device="cuda")
    B.linear_w4a16_ex(dev(x16), dev(packed), y, M, N, K, group, B.F16, y_dtype)
    assert B.read_status() == 0
    return y.float().cpu().numpy()


def test_config1_single_gemv_seed0():
    # x fp16 [1,1536] ~ N(0,1); W [1536,1536] ~ N(0,0.02), int4 group 64; y fp16
    N = K = 1536
    W, packed, (q, s, z) = quantized(0, N, K, 64)
    x = inputs.activations(1, 1, K)
    y = torch.empty((1, N), dtype=torch.float16, device="cuda")
    B.linear_w4a16(dev(x), dev(packed), y, 1, N, K, 64)
    assert B.read_status() == 0
    assert_close(y.float().cpu().numpy(), oracle.linear_wa16(x.astype(np.float32), q, s, z, 64))


@pytest.mark.parametrize("N,K,M,group", [
    (16, 64, 1, 64),          # one slab
    (40, 192, 1, 64),         # ragged rows, partial chunk only
    (100, 8960, 1, 64),       # 17.5 chunks: a partial last chunk, many k-chunks per warp
    (256, 1536, 1, 64),       # k/v projection shape
    (1536, 8960, 1, 64),      # down projection: few rows, long K (cluster split-K)
    (2000, 1536, 2, 64),
    (777, 1024, 3, 64),
    (8960, 1536, 4, 64),      # gate/up projection, 4 tokens
    (520, 576, 8, 64),
    (300, 1536, 11, 64),      # more than 8 tokens: two passes
    (130, 3584, 1, 128),      # group 128
    (1000, 3584, 4, 128),
    (64, 640, 7, 128),
])
def test_w4a16_matches_oracle(N, K, M, group):
    W, packed, (q, s, z) = quantized(N * 7 + K + M, N, K, group)
    x = inputs.activations(N + K + M, M, K)
    y = run_w4a16(x, packed, M, N, K, group)
    assert_close(y, oracle.linear_wa16(x.astype(np.float32), q, s, z, group))


def test_w4a16_exact_on_lossless_weights():
    # weights on the quantisation grid, small integer activations: every product and sum is exact
    # in fp32, so the result must equal the integer arithmetic exactly
    rng = np.random.default_rng(4)
    N, K, group = 48, 1024, 64
    qi = rng.integers(0, 16, (N, K))
    qi[:, ::64] = 0
    qi[:, 1::64] = 15
    zero = rng.integers(0, 16, (N, K // group))
    W = ((qi - np.repeat(zero, group, axis=1)) * 0.125).astype(np.float32)
    x = rng.integers(-8, 9, (2, K)).astype(np.float16)
    packed = B.pack_w4(W, group)
    y = run_w4a16(x, packed, 2, N, K, group, B.F32)
    want = x.astype(np.float64) @ W.astype(np.float64).T
    assert (y == want).all()


def test_w4a16_output_dtypes():
    N, K, M, group = 512, 1536, 2, 64
    W, packed, (q, s, z) = quantized(77, N, K, group)
    x = inputs.activations(78, M, K)
    ref = oracle.linear_wa16(x.astype(np.float32), q, s, z, group)
    assert_close(run_w4a16(x, packed, M, N, K, group, B.F32), ref)
    assert_close(run_w4a16(x, packed, M, N, K, group, B.F32), ref, 2e-4)   # fp32 logits are much tighter
    y_bf16 = run_w4a16(x, packed, M, N, K, group, B.BF16)
    assert_bf16_within_1ulp(y_bf16, ref)


@pytest.mark.parametrize("N,K,M,group", [(256, 1536, 1, 64), (1536, 8960, 1, 64), (777, 1024, 3, 64), (1000, 3584, 4, 128),
                                         (300, 1536, 11, 64)])
def test_w4a16_bf16_activations_match_oracle(N, K, M, group):
    W, packed, (q, s, z) = quantized(N + 3 * K + M, N, K, group)
    xb = inputs.activations(N + K + 5 * M, M, K, dtype="bf16")      # fp32 array of bf16-exact values
    xd = dev(inputs.bf16_bits(xb)).view(torch.bfloat16)
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    B.linear_w4a16_ex(xd, dev(packed), y, M, N, K, group, B.BF16, B.F32)
    assert B.read_status() == 0
    assert_close(y.cpu().numpy(), oracle.linear_wa16(xb, q, s, z, group), 2e-4)


def test_w4a16_batch_qkv_one_launch():
    K, M = 1536, 1
    shapes = [1536, 256, 256]
    x = inputs.activations(90, M, K)
    xd = dev(x)
    probs, refs, ys = [], [], []
    keep = []
    for i, N in enumerate(shapes):
        W, packed, (q, s, z) = quantized(91 + i, N, K, 64)
        pd = dev(packed)
        y = torch.zeros((M, N), dtype=torch.float16, device="cuda")
        keep += [pd, y]
        probs.append(dict(x=xd, packed=pd, y=y, N=N, K=K, group=64, y_dtype=B.F16))
        refs.append(oracle.linear_wa16(x.astype(np.float32), q, s, z, 64))
        ys.append(y)
    B.linear_w4a16_batch(probs, M)
    assert B.read_status() == 0
    for y, ref in zip(ys, refs):
        assert_close(y.float().cpu().numpy(), ref)


def test_w4a16_deterministic_and_stream_ordered():
    N, K, M = 1536, 8960, 1
    W, packed, _ = quantized(5, N, K, 64)
    xd, pd = dev(inputs.activations(6, M, K)), dev(packed)
    outs = []
    s = torch.cuda.Stream()
    for _ in range(3):
        y = torch.empty((M, N), dtype=torch.float16, device="cuda")
        with torch.cuda.stream(s):
            B.linear_w4a16(xd, pd, y, M, N, K, 64, stream=s)
        s.synchronize()
        outs.append(y.cpu())
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])


def test_w4a16_argument_errors_on_gpu():
    y = torch.empty(64, dtype=torch.float16, device="cuda")
    st = B.lib.mnnllm_linear_w4a16(y.data_ptr() + 2, y.data_ptr(), y.data_ptr(), 1, 16, 64, 64, None)
    assert st == 3
    assert B.lib.mnnllm_linear_w4a16(y.data_ptr(), y.data_ptr(), y.data_ptr(), 1, 16, 64, 32, None) == 2
    assert B.lib.mnnllm_linear_w4a16_ex(y.data_ptr(), y.data_ptr(), y.data_ptr(), 1, 16, 64, 64, B.F32, B.F16, None) == 2
    assert B.lib.mnnllm_linear_w4a16_ex(y.data_ptr(), y.data_ptr(), y.data_ptr(), 1, 16, 64, 64, 7, B.F16, None) == 1


@pytest.mark.parametrize("N,K,M", [(16, 32, 1), (37, 96, 3), (1000, 3584, 1), (4096, 3584, 4), (200, 544, 8), (64, 1024, 9)])
def test_w8a16_matches_oracle(N, K, M):
    W = inputs.weights(300 + N, N, K)
    packed = B.pack_w8(W)
    q, s, z = oracle.quantize_w8(W)
    x = inputs.activations(301 + N, M, K)
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    B.linear_w8a16(dev(x), dev(packed), y, M, N, K, B.F32)
    assert B.read_status() == 0
    assert_close(y.cpu().numpy(), oracle.linear_wa16(x.astype(np.float32), q, s, z, K))
