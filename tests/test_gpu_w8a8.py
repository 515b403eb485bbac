"""GPU parity of the per-channel W8A8 prefill GEMM (mnnllm_linear_w8a8) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_10443_b200 import binding as B
from paper_2506_10443_b200 import inputs
from gpu_util import assert_bf16_within_1ulp, assert_close, dev

pytestmark = pytest.mark.gpu

TDT = {B.F16: torch.float16, B.BF16: torch.bfloat16, B.F32: torch.float32}
# fp32 outputs: one fp32 rounding of the int32 sum (2^-24 of up to ~3 x the signal after the zero-point
# term is taken off) and three fp32 products; far inside the path's 2e-3
TOL_F32 = 2e-5


def run(x, packed, M, N, K, y_dtype=B.F32, x_dtype=B.F16, stream=None):
    y = torch.full((M, N), float("nan"), dtype=TDT[y_dtype], device="cuda")
    ws_bytes = B.workspace_size_w8a8(M, K)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    B.linear_w8a8(x, packed, y, M, N, K, ws, ws_bytes, x_dtype, y_dtype, stream)
    torch.cuda.synchronize()
    assert B.read_status() == 0
    return y


@pytest.mark.parametrize("M,N,K", [
    (300, 384, 512),      # two 256-token tiles would leave SMs idle: 128-token tiles, ragged M
    (128, 128, 128),      # one tile, one stage
    (1, 16, 32),          # smallest: one token, one row block, a quarter of a stage
    (77, 200, 1536),      # ragged N (last row block partly filled) and M
    (515, 2000, 1088),    # K not a multiple of the 128-k stage; N not a multiple of 128
    (1024, 8960 * 2, 1536),   # gate+up of Qwen2-1.5B at 1024 tokens: 256-token tiles, several tiles per CTA
    (512, 1536, 8960),    # down: long K
])
def test_w8a8_matches_oracle(M, N, K):
    W = inputs.weights(11 + M, N, K)
    x = inputs.activations(12 + M, M, K, outliers=True)
    q, s, z = oracle.quantize_w8(W)
    y = run(dev(x), dev(B.pack_w8(W)), M, N, K)
    if M * N * K <= 1 << 31:
        assert_close(y.cpu().numpy(), oracle.linear_w8a8(x.astype(np.float32), q, s, z), TOL_F32)
    else:
        # full size: sampled tokens (first and last of the 256-token tiles and of their column halves).
        # The activation quantiser works per token, so the oracle on the sampled rows alone is the same.
        rows = sorted(r for r in {0, 1, 127, 128, 255, 256, 383, 511, 640, 769, M - 2, M - 1} if r < M)
        want = oracle.linear_w8a8(x[rows].astype(np.float32), q, s, z)
        assert_close(y.cpu().numpy()[rows], want, TOL_F32)
        assert torch.isfinite(y).all()


def test_w8a8_integer_exact_case():
    # weights on the 8-bit grid with scale 1/8 and integer activations with amax = 127: a_scale = 1,
    # every product and the int32 sum are exact and the fp32 rescale is exact too
    rng = np.random.default_rng(3)
    M, N, K = 260, 272, 640
    qi = rng.integers(0, 256, (N, K))
    qi[:, 0], qi[:, 1] = 0, 255
    zero = rng.integers(0, 256, (N, 1))
    W = ((qi - zero) * 0.125).astype(np.float32)
    x = rng.integers(-20, 21, (M, K)).astype(np.float16)
    x[:, 3] = 127
    y = run(dev(x), dev(B.pack_w8(W)), M, N, K)
    want = x.astype(np.float64) @ W.astype(np.float64).T
    assert (y.cpu().numpy() == want).all()


def test_w8a8_output_dtypes_and_bf16_input():
    M, N, K = 200, 320, 1024
    W = inputs.weights(21, N, K)
    q, s, z = oracle.quantize_w8(W)
    packed = dev(B.pack_w8(W))
    x = inputs.activations(22, M, K)
    want = oracle.linear_w8a8(x.astype(np.float32), q, s, z)
    y16 = run(dev(x), packed, M, N, K, B.F16)
    assert_close(y16.float().cpu().numpy(), want, 2.0 ** -11 + TOL_F32)
    ybf = run(dev(x), packed, M, N, K, B.BF16)
    assert_bf16_within_1ulp(ybf.float().cpu().numpy(), want)
    xb = torch.from_numpy(x.astype(np.float32)).cuda().to(torch.bfloat16)
    want_b = oracle.linear_w8a8(xb.float().cpu().numpy(), q, s, z)
    yb = run(xb, packed, M, N, K, B.F32, B.BF16)
    assert_close(yb.cpu().numpy(), want_b, TOL_F32)


def test_w8a8_zero_rows_and_zero_tokens():
    M, N, K = 130, 144, 256
    W = inputs.weights(31, N, K)
    W[5] = 0.0                      # a constant row: scale 1, code 0
    x = inputs.activations(32, M, K)
    x[7] = 0.0                      # an all-zero token: a_scale = 0
    q, s, z = oracle.quantize_w8(W)
    y = run(dev(x), dev(B.pack_w8(W)), M, N, K).cpu().numpy()
    assert (y[7] == 0).all() and (y[:, 5] == 0).all()
    assert_close(y, oracle.linear_w8a8(x.astype(np.float32), q, s, z), TOL_F32)


def test_w8a8_graph_replay_is_bit_identical_and_reuses_the_workspace():
    M, N, K = 384, 1536, 1536
    W = inputs.weights(41, N, K)
    packed = dev(B.pack_w8(W))
    x = dev(inputs.activations(42, M, K))
    y = torch.zeros((M, N), dtype=torch.float16, device="cuda")
    ws_bytes = B.workspace_size_w8a8(M, K)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    B.linear_w8a8(x, packed, y, M, N, K, ws, ws_bytes)
    torch.cuda.synchronize()
    first = y.clone()
    g = torch.cuda.CUDAGraph()
    cap = torch.cuda.Stream()
    cap.wait_stream(torch.cuda.current_stream())
    with torch.cuda.graph(g, stream=cap):
        B.linear_w8a8(x, packed, y, M, N, K, ws, ws_bytes, stream=cap)
    for _ in range(4):
        y.zero_()
        g.replay()
    torch.cuda.synchronize()
    assert B.read_status() == 0
    assert torch.equal(first, y)


def test_w8a8_argument_errors():
    x = torch.zeros((4, 64), dtype=torch.float16, device="cuda")
    y = torch.zeros((4, 16), dtype=torch.float16, device="cuda")
    packed = dev(B.pack_w8(np.ones((16, 64), np.float32)))
    ws = torch.zeros(B.workspace_size_w8a8(4, 64), dtype=torch.uint8, device="cuda")
    assert B.workspace_size_w8a8(4, 48) == 0
    with pytest.raises(B.MnnllmError) as e:
        B.linear_w8a8(x, packed, y, 4, 16, 48, ws, ws.numel())      # K not a multiple of 32
    assert e.value.status == 2
    with pytest.raises(B.MnnllmError) as e:
        B.linear_w8a8(x, packed, y, 4, 16, 64, ws, ws.numel() - 1)  # workspace too small
    assert e.value.status == 6
    with pytest.raises(B.MnnllmError) as e:
        B.linear_w8a8(x, packed, y, 0, 16, 64, ws, ws.numel())
    assert e.value.status == 1
    B.linear_w8a8(x, packed, y, 4, 16, 64, ws, ws.numel())
    torch.cuda.synchronize()
    assert B.read_status() == 0
