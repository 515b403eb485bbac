"""GPU parity of the W4A16 linear with LoRA bypass (mnnllm_linear_w4a16_lora) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_10443_b200 import binding as B
from paper_2506_10443_b200 import inputs
from gpu_util import assert_bf16_within_1ulp, assert_close, dev, quantized

pytestmark = pytest.mark.gpu

TDT = {B.F16: torch.float16, B.BF16: torch.bfloat16, B.F32: torch.float32}


def lora_pair(seed, N, K, r, scale=0.05):
    rng = np.random.default_rng(seed)
    A = (rng.standard_normal((N, r)) * scale).astype(np.float16)
    Bm = (rng.standard_normal((r, K)) * scale).astype(np.float16)
    return A, Bm


def run(x, packed, A, Bm, M, N, K, group, r, y_dtype=B.F32, x_dtype=B.F16, stream=None):
    y = torch.full((M, N), float("nan"), dtype=TDT[y_dtype], device="cuda")
    ws_bytes = B.workspace_size_lora(M, r)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    B.lora_workspace_init(ws, ws_bytes)
    B.linear_w4a16_lora(x, packed, A, Bm, y, M, N, K, group, r, ws, ws_bytes, x_dtype, y_dtype, stream)
    torch.cuda.synchronize()
    assert B.read_status() == 0
    return y


def want_of(x, qsz, A, Bm, group):
    q, s, z = qsz
    xf = np.asarray(x, np.float32)
    return oracle.lora_bypass(oracle.linear_wa16(xf, q, s, z, group), xf, A.astype(np.float32), Bm.astype(np.float32))


@pytest.mark.parametrize("M,N,K,group,r", [
    (1, 1536, 1536, 64, 8),      # o projection, one token
    (1, 1536, 8960, 64, 8),      # down: clusters split K, the bypass is added after the cluster reduction
    (4, 2000, 1536, 64, 16),     # ragged N, several tokens
    (8, 300, 3584, 128, 4),      # group 128, eight tokens
    (11, 256, 512, 64, 3),       # two passes over the weights (8 + 3 tokens), odd rank
    (2, 40, 64, 64, 64),         # smallest K, largest rank
])
def test_lora_matches_oracle(M, N, K, group, r):
    _, packed, qsz = quantized(61 + M, N, K, group)
    x = inputs.activations(62 + M, M, K)
    A, Bm = lora_pair(63 + M, N, K, r)
    y = run(dev(x), dev(packed), dev(A), dev(Bm), M, N, K, group, r)
    assert_close(y.cpu().numpy(), want_of(x, qsz, A, Bm, group))


def test_lora_term_dominant_is_tight():
    # weights a thousand times smaller than usual: the output is the bypass to three digits, and the
    # bypass is two fp32 sums of exact fp16 products, so the whole is held to 2e-5 of the row's
    # magnitude, a hundred times tighter than the path's 2e-3
    M, N, K, group, r = 3, 512, 1024, 64, 8
    W = inputs.weights(70, N, K) * np.float32(1e-3)
    packed, qsz = B.pack_w4(W, group), oracle.quantize_w4(W, group)
    x = inputs.activations(71, M, K)
    A, Bm = lora_pair(72, N, K, r, scale=0.5)
    y = run(dev(x), dev(packed), dev(A), dev(Bm), M, N, K, group, r)
    assert_close(y.cpu().numpy(), want_of(x, qsz, A, Bm, group), 2e-5)


def test_zero_lora_equals_plain_linear_bitwise():
    M, N, K, group, r = 2, 1536, 1536, 64, 8
    _, packed, _ = quantized(73, N, K, group)
    x, pd = dev(inputs.activations(74, M, K)), dev(packed)
    A, Bm = np.zeros((N, r), np.float16), np.zeros((r, K), np.float16)
    y = run(x, pd, dev(A), dev(Bm), M, N, K, group, r)
    y0 = torch.empty((M, N), dtype=torch.float32, device="cuda")
    B.linear_w4a16_ex(x, pd, y0, M, N, K, group, B.F16, B.F32)
    torch.cuda.synchronize()
    assert torch.equal(y, y0)


def test_lora_dtypes():
    M, N, K, group, r = 2, 640, 2048, 64, 8
    _, packed, qsz = quantized(75, N, K, group)
    x = inputs.activations(76, M, K)
    A, Bm = lora_pair(77, N, K, r)
    pd, Ad, Bd = dev(packed), dev(A), dev(Bm)
    want = want_of(x, qsz, A, Bm, group)
    y16 = run(dev(x), pd, Ad, Bd, M, N, K, group, r, B.F16)
    assert_close(y16.float().cpu().numpy(), want, 2.0 ** -11 + 2e-3)
    ybf = run(dev(x), pd, Ad, Bd, M, N, K, group, r, B.BF16)
    assert_bf16_within_1ulp(ybf.float().cpu().numpy(), want, fp32_tol=2e-3)
    xb = torch.from_numpy(x.astype(np.float32)).cuda().to(torch.bfloat16)
    yb = run(xb, pd, Ad, Bd, M, N, K, group, r, B.F32, B.BF16)
    assert_close(yb.cpu().numpy(), want_of(xb.float().cpu().numpy(), qsz, A, Bm, group))


def test_lora_graph_replay_and_argument_errors():
    M, N, K, group, r = 1, 1536, 1536, 64, 8
    _, packed, _ = quantized(78, N, K, group)
    x, pd = dev(inputs.activations(79, M, K)), dev(packed)
    A, Bm = lora_pair(80, N, K, r)
    Ad, Bd = dev(A), dev(Bm)
    y = torch.zeros((M, N), dtype=torch.float16, device="cuda")
    ws_bytes = B.workspace_size_lora(M, r)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    B.lora_workspace_init(ws, ws_bytes)
    B.linear_w4a16_lora(x, pd, Ad, Bd, y, M, N, K, group, r, ws, ws_bytes)
    torch.cuda.synchronize()
    first = y.clone()
    g = torch.cuda.CUDAGraph()
    cap = torch.cuda.Stream()
    cap.wait_stream(torch.cuda.current_stream())
    with torch.cuda.graph(g, stream=cap):
        B.linear_w4a16_lora(x, pd, Ad, Bd, y, M, N, K, group, r, ws, ws_bytes, stream=cap)
    for _ in range(3):
        y.zero_()
        g.replay()
    torch.cuda.synchronize()
    assert B.read_status() == 0 and torch.equal(first, y)
    words = ws[:8].view(torch.int32).cpu().tolist()
    assert words == [4, 0]      # epoch = launches so far (one eager, three replays); the CTA counter is back at zero
    assert B.workspace_size_lora(1, 65) == 0 and B.workspace_size_lora(0, 8) == 0
    with pytest.raises(B.MnnllmError) as e:
        B.linear_w4a16_lora(x, pd, Ad, Bd, y, M, N, K, group, 65, ws, ws_bytes)     # rank too large
    assert e.value.status == 1
    with pytest.raises(B.MnnllmError) as e:
        B.linear_w4a16_lora(x, pd, Ad, Bd, y, M, N, K, group, r, ws, ws_bytes - 1)  # workspace too small
    assert e.value.status == 6
    with pytest.raises(B.MnnllmError) as e:
        B.linear_w4a16_lora(x, pd, None, Bd, y, M, N, K, group, r, ws, ws_bytes)
    assert e.value.status == 1
