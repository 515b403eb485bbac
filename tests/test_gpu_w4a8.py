"""GPU parity of the prefill W4A8 path against the CPU oracle, through the C ABI: the int32 group
partials bit for bit, the outputs within 2e-3."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_10443_b200 import binding as B
from paper_2506_10443_b200 import inputs
from gpu_util import assert_bf16_within_1ulp, assert_close, dev, quantized

pytestmark = pytest.mark.gpu


def run_w4a8(x, packed, M, N, K, group, y_dtype=B.F16, x_dtype=B.F16):
    tdt = {B.F16: torch.float16, B.BF16: torch.bfloat16, B.F32: torch.float32}[y_dtype]
    nbytes = B.workspace_size_w4a8(M, N, K, group)
    assert nbytes > 0
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    y = torch.full((M, N), float("nan"), dtype=tdt, device="cuda")
    B.linear_w4a8(x, dev(packed), y, M, N, K, group, ws, nbytes, x_dtype=x_dtype, y_dtype=y_dtype)
    assert B.read_status() == 0
    return y.float().cpu().numpy()


@pytest.mark.parametrize("M,N,K,group", [
    (1, 16, 64, 64),         # one group, one row block
    (5, 40, 192, 64),        # K = 1.5 stages: a stage with a single group
    (130, 200, 320, 64),     # ragged in M, N and K against the 128 x 128 x 128 tiles
    (64, 256, 1536, 64),     # k/v projection, shortest prompt
    (33, 130, 1024, 128),    # group 128
    (96, 48, 8960, 64),      # the down projection's K: a partial last 512-k chunk
    (3, 300, 3584, 128),
])
def test_group_partials_bit_exact(M, N, K, group):
    W, packed, (q, s, z) = quantized(M + 3 * N + K, N, K, group)
    x = inputs.activations(M + N + K, M, K, outliers=True)
    G = K // group
    P = torch.full((M, N, G), -7777, dtype=torch.int32, device="cuda")
    a_q = torch.empty((M, K), dtype=torch.int8, device="cuda")
    a_scale = torch.empty((M,), dtype=torch.float32, device="cuda")
    A = torch.empty((M, G), dtype=torch.int32, device="cuda")
    B.debug_w4a8_partials(dev(x), dev(packed), P, a_q, a_scale, A, M, N, K, group)
    assert B.read_status() == 0
    aq0, as0, A0 = oracle.act_quant(x.astype(np.float32), group)
    assert (a_q.cpu().numpy() == aq0).all()
    assert (A.cpu().numpy() == A0).all()
    assert (a_scale.cpu().numpy().view(np.uint32) == as0.view(np.uint32)).all()
    assert (P.cpu().numpy() == oracle.group_partials(aq0, q, group)).all()


@pytest.mark.parametrize("M,N,K,group", [
    (1, 16, 64, 64),
    (5, 40, 192, 64),
    (130, 200, 320, 64),
    (64, 1536, 1536, 64),     # q/o projection, prompt of 64
    (256, 256, 1536, 64),     # k/v projection, prompt of 256
    (256, 512, 8960, 64),     # down projection rows, long K
    (300, 1000, 448, 64),     # G = 7: the last zero-point block holds three groups
    (77, 130, 1024, 128),
    (512, 384, 3584, 128),
])
def test_w4a8_matches_oracle(M, N, K, group):
    W, packed, (q, s, z) = quantized(2 * M + N + K, N, K, group)
    x = inputs.activations(M + 2 * N + K, M, K, outliers=True)
    y = run_w4a8(dev(x), packed, M, N, K, group, B.F32)
    assert_close(y, oracle.linear_w4a8(x.astype(np.float32), q, s, z, group))


@pytest.fixture
def short_prompt_kernel_up_to_64():
    """By default prompts of up to 32 tokens take the GEMV-shaped kernel; these tests drive it to its
    limit of 64 tokens (eight token tiles) and put the default back afterwards."""
    before = B.debug_set_w4a8_small_max(64)
    yield
    B.debug_set_w4a8_small_max(-1)
    assert before == 32


@pytest.mark.parametrize("M,N,K,group", [
    (7, 48, 512, 64),          # short prompts take the GEMV-shaped kernel (M <= 64): one chunk
    (8, 1000, 1536, 64),       # ragged last 16-row block
    (9, 2048, 1536, 64),       # q+k+v rows, two token tiles (the second almost empty)
    (33, 272, 8960, 64),       # partial last chunk, K cut into parts
    (64, 8960, 1536, 64),      # gate/up projection at the longest short prompt
    (64, 1536, 8960, 64),      # down projection: few rows, long K
    (17, 130, 1024, 128),      # group 128
    (64, 300, 3712, 128),      # group 128, K = 7.25 chunks
    (50, 200, 576, 64),        # last chunk of a single group
])
def test_w4a8_short_prompt_kernel_matches_oracle(M, N, K, group, short_prompt_kernel_up_to_64):
    W, packed, (q, s, z) = quantized(5 * M + N + K, N, K, group)
    x = inputs.activations(M + 7 * N + K, M, K, outliers=True)
    ref = oracle.linear_w4a8(x.astype(np.float32), q, s, z, group)
    assert_close(run_w4a8(dev(x), packed, M, N, K, group, B.F32), ref, 2e-4)
    assert_close(run_w4a8(dev(x), packed, M, N, K, group, B.F16), ref)
    # and every int32 group partial through the same kernel, bit for bit
    G = K // group
    P = torch.full((M, N, G), -7777, dtype=torch.int32, device="cuda")
    a_q = torch.empty((M, K), dtype=torch.int8, device="cuda")
    a_scale = torch.empty((M,), dtype=torch.float32, device="cuda")
    A = torch.empty((M, G), dtype=torch.int32, device="cuda")
    B.debug_w4a8_partials(dev(x), dev(packed), P, a_q, a_scale, A, M, N, K, group)
    assert B.read_status() == 0
    aq0, _, _ = oracle.act_quant(x.astype(np.float32), group)
    assert (a_q.cpu().numpy() == aq0).all()
    assert (P.cpu().numpy() == oracle.group_partials(aq0, q, group)).all()


def test_w4a8_short_prompt_batch_and_bf16_input(short_prompt_kernel_up_to_64):
    M, K, group = 40, 1536, 64
    shapes = [1536, 256, 250]
    xb = inputs.activations(71, M, K, outliers=True, dtype="bf16")
    xd = dev(inputs.bf16_bits(xb)).view(torch.bfloat16)
    probs, refs, ys, keep = [], [], [], []
    for i, N in enumerate(shapes):
        W, packed, (q, s, z) = quantized(72 + i, N, K, group)
        pd = dev(packed)
        y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        keep.append(pd)
        probs.append(dict(packed=pd, y=y, N=N, y_dtype=B.F32))
        refs.append(oracle.linear_w4a8(xb, q, s, z, group))
        ys.append(y)
    nbytes = B.workspace_size_w4a8(M, max(shapes), K, group)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    B.linear_w4a8_batch(probs, xd, M, K, group, ws, nbytes, x_dtype=B.BF16)
    assert B.read_status() == 0
    for y, ref in zip(ys, refs):
        assert_close(y.cpu().numpy(), ref, 2e-4)


@pytest.fixture
def limb_kernel_forced():
    """The integer-limb GEMM normally takes launches with at least 0.6 tiles per SM; these tests force it
    onto small shapes too and put the default back afterwards."""
    B.debug_set_w4a8_limb(2)
    yield
    B.debug_set_w4a8_limb(-1)


@pytest.mark.parametrize("M,N,K,group", [
    (65, 16, 64, 64),          # one group
    (130, 200, 320, 64),       # ragged in M, N and K against the 128 x 128 x 128 tiles
    (128, 128, 1024, 64),      # one full tile, two chunks
    (256, 512, 8960, 64),      # long K, partial last chunk
    (300, 1000, 448, 64),      # G = 7: the last zero-point block holds three groups
    (77, 130, 1024, 128),      # group 128
    (512, 384, 3584, 128),
    (1024, 1536, 1536, 64),    # q projection at the longest prompt
])
def test_w4a8_limb_kernel_matches_oracle(M, N, K, group, limb_kernel_forced):
    W, packed, (q, s, z) = quantized(2 * M + N + K + 1, N, K, group)
    x = inputs.activations(M + 2 * N + K + 1, M, K, outliers=True)
    ref = oracle.linear_w4a8(x.astype(np.float32), q, s, z, group)
    y = run_w4a8(dev(x), packed, M, N, K, group, B.F32)
    assert_close(y, ref, 2e-4)
    B.debug_set_w4a8_limb(0)      # and the per-group kernel on the same call, for comparison
    y_old = run_w4a8(dev(x), packed, M, N, K, group, B.F32)
    assert_close(y_old, ref, 2e-4)
    assert_close(y, y_old.astype(np.float64), 1e-5)


def test_w4a8_limb_kernel_falls_back_when_a_row_spans_too_many_binades(limb_kernel_forced):
    # one group of one row is constant (scale 1 against ~0.005 elsewhere: eight binades): the packer
    # clears the flag, the limb kernel returns at once and the per-group kernel does the work
    M, N, K, group = 140, 144, 1536, 64
    W = inputs.weights(31, N, K)
    W[5, 128:192] = 0.25
    packed, (q, s, z) = B.pack_w4(W, group), oracle.quantize_w4(W, group)
    off = -(-(128 + (N // 16) * ((K // 64) * 512 + 16 * (K // group) * 4)) // 128) * 128
    assert packed[off:off + 4].view(np.uint32)[0] == 0
    x = inputs.activations(32, M, K, outliers=True)
    y = run_w4a8(dev(x), packed, M, N, K, group, B.F32)
    assert_close(y, oracle.linear_w4a8(x.astype(np.float32), q, s, z, group), 2e-4)


def test_w4a8_limb_kernel_batch_and_weight_range(limb_kernel_forced):
    M, K, group = 200, 1536, 64
    x = (inputs.activations(41, M, K).astype(np.float32) + 1.0).astype(np.float16)
    for std in (1e-5, 3.0):
        probs, refs, ys, keep = [], [], [], []
        for i, N in enumerate((272, 130)):
            W = inputs.weights(42 + i, N, K, std=std)
            pd = dev(B.pack_w4(W, group))
            q, s, z = oracle.quantize_w4(W, group)
            y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
            keep.append(pd)
            probs.append(dict(packed=pd, y=y, N=N, y_dtype=B.F32))
            refs.append(oracle.linear_w4a8(x.astype(np.float32), q, s, z, group))
            ys.append(y)
        nbytes = B.workspace_size_w4a8(M, 272, K, group)
        ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        B.linear_w4a8_batch(probs, dev(x), M, K, group, ws, nbytes)
        assert B.read_status() == 0
        for y, ref in zip(ys, refs):
            assert_close(y.cpu().numpy(), ref)


def test_w4a8_output_and_input_dtypes():
    M, N, K, group = 70, 272, 1536, 64
    W, packed, (q, s, z) = quantized(11, N, K, group)
    x = inputs.activations(12, M, K, outliers=True)
    ref = oracle.linear_w4a8(x.astype(np.float32), q, s, z, group)
    y32 = run_w4a8(dev(x), packed, M, N, K, group, B.F32)
    assert_close(y32, ref, 2e-4)
    assert_close(run_w4a8(dev(x), packed, M, N, K, group, B.F16), ref)
    assert_bf16_within_1ulp(run_w4a8(dev(x), packed, M, N, K, group, B.BF16), ref)
    xb = inputs.activations(13, M, K, outliers=True, dtype="bf16")
    yb = run_w4a8(dev(inputs.bf16_bits(xb)).view(torch.bfloat16), packed, M, N, K, group, B.F32, x_dtype=B.BF16)
    assert_close(yb, oracle.linear_w4a8(xb, q, s, z, group))


@pytest.mark.parametrize("std", [1e-5, 2e-3, 3.0])
def test_w4a8_zero_point_term_over_the_weight_range(std):
    # tiny, small and large weights against activations with a non-zero mean (large group sums A, so
    # that the zero-point term dominates and cancels against the integer partials)
    M, N, K, group = 96, 144, 1536, 64
    W = inputs.weights(21, N, K, std=std)
    packed, (q, s, z) = B.pack_w4(W, group), oracle.quantize_w4(W, group)
    x = (inputs.activations(22, M, K).astype(np.float32) + 1.0).astype(np.float16)
    y = run_w4a8(dev(x), packed, M, N, K, group, B.F32)
    assert_close(y, oracle.linear_w4a8(x.astype(np.float32), q, s, z, group))


def test_w4a8_unusual_zero_points():
    # groups that do not straddle zero (negative and large zero points), a constant group and an
    # all-zero token: the zero-point term must stay exact
    rng = np.random.default_rng(5)
    M, N, K, group = 40, 64, 512, 64
    W = rng.normal(0, 0.02, (N, K)).astype(np.float32)
    W[:16] += 0.3
    W[16:32] -= 0.25
    W[32, :64] = 0.125
    x = inputs.activations(21, M, K, outliers=True)
    x[7] = 0
    packed = B.pack_w4(W, group)
    q, s, z = oracle.quantize_w4(W, group)
    y = run_w4a8(dev(x), packed, M, N, K, group, B.F32)
    assert_close(y, oracle.linear_w4a8(x.astype(np.float32), q, s, z, group))
    assert (y[7] == 0).all()


def test_w4a8_batch_qkv_one_launch():
    # three matrices on the same activations: one quantiser pass, one GEMM grid; ragged N on purpose
    M, K, group = 200, 1536, 64
    shapes = [1536, 256, 200]
    x = inputs.activations(41, M, K, outliers=True)
    xd = dev(x)
    probs, refs, ys, keep = [], [], [], []
    for i, N in enumerate(shapes):
        W, packed, (q, s, z) = quantized(42 + i, N, K, group)
        pd = dev(packed)
        y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        keep.append(pd)
        probs.append(dict(packed=pd, y=y, N=N, y_dtype=B.F32))
        refs.append(oracle.linear_w4a8(x.astype(np.float32), q, s, z, group))
        ys.append(y)
    nbytes = B.workspace_size_w4a8(M, max(shapes), K, group)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    B.linear_w4a8_batch(probs, xd, M, K, group, ws, nbytes)
    assert B.read_status() == 0
    for y, ref in zip(ys, refs):
        assert_close(y.cpu().numpy(), ref)
    assert B.lib.mnnllm_linear_w4a8_batch(B.make_batch_w4a8(probs), 5, xd.data_ptr(), M, K, group, B.F16, ws.data_ptr(),
                                          nbytes, None) == 1


@pytest.mark.parametrize("M,N,K,group", [
    (64, 1536, 8960, 64),     # down projection at a short prompt: 12 tiles, 17.5 chunks of K
    (200, 272, 3584, 128),    # ragged M and N, group 128
    (128, 128, 1024, 64),     # one tile, two chunks
])
def test_w4a8_tiles_split_along_k(M, N, K, group):
    # With the full workspace a problem with fewer tiles than SMs is cut along K and the parts are
    # summed in scratch memory; with the minimal workspace it is not.  Both must match the oracle,
    # agree closely with each other, and the split form must not depend on timing.
    W, packed, (q, s, z) = quantized(3 * M + N + K, N, K, group)
    x = inputs.activations(M + 5 * N + K, M, K, outliers=True)
    ref = oracle.linear_w4a8(x.astype(np.float32), q, s, z, group)
    xd, pd = dev(x), dev(packed)

    def run(nbytes):
        ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        B.linear_w4a8(xd, pd, y, M, N, K, group, ws, nbytes, y_dtype=B.F32)
        assert B.read_status() == 0
        return y.cpu().numpy()

    full, small = B.workspace_size_w4a8(M, N, K, group), B.workspace_min_w4a8(M, N, K, group)
    assert full > small
    y_split, y_whole = run(full), run(small)
    assert_close(y_split, ref)
    assert_close(y_whole, ref)
    assert_close(y_split, y_whole.astype(np.float64), 1e-5)
    for _ in range(3):
        assert (run(full).view(np.uint32) == y_split.view(np.uint32)).all()


def test_w4a8_split_calls_back_to_back_share_a_workspace():
    # The way a model runs it: calls on one stream, one workspace, replayed from a CUDA graph.  The
    # counters and scratch slots of the K split are reused by every call (the quantiser of a call
    # clears the counters, ordered behind the previous GEMM by the stream); outputs must not change
    # from replay to replay and must match calls made one at a time.
    M, group = 64, 64
    shapes = [(1536, 8960), (2048, 1536), (1536, 1536)]   # (N, K): all with fewer tiles than SMs
    nbytes = max(B.workspace_size_w4a8(M, N, K, group) for N, K in shapes)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    probs = []
    for i, (N, K) in enumerate(shapes):
        W, packed, _ = quantized(700 + i, N, K, group)
        x = dev(inputs.activations(710 + i, M, K, outliers=True))
        probs.append((x, dev(packed), N, K))
    ys = [torch.zeros((M, N), dtype=torch.float32, device="cuda") for _, _, N, _ in probs]

    def one_round(stream):
        for (x, pk, N, K), y in zip(probs, ys):
            B.linear_w4a8(x, pk, y, M, N, K, group, ws, nbytes, y_dtype=B.F32, stream=stream)

    one_round(None)
    torch.cuda.synchronize()
    assert B.read_status() == 0
    want = [y.clone() for y in ys]
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        one_round(s)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            for _ in range(4):
                one_round(s)
        for _ in range(5):
            for y in ys:
                y.zero_()
            g.replay()
            torch.cuda.synchronize()
            for y, w in zip(ys, want):
                assert torch.equal(y, w)
    assert B.read_status() == 0


def test_w4a8_deterministic():
    M, N, K, group = 200, 640, 1536, 64
    W, packed, _ = quantized(31, N, K, group)
    xd = dev(inputs.activations(32, M, K, outliers=True))
    a = run_w4a8(xd, packed, M, N, K, group)
    b = run_w4a8(xd, packed, M, N, K, group)
    assert (a == b).all()


def test_w4a8_argument_errors_on_gpu():
    t = torch.empty(1 << 16, dtype=torch.uint8, device="cuda")
    p = t.data_ptr()
    need = B.workspace_min_w4a8(4, 16, 64, 64)
    assert need > 0 and B.workspace_size_w4a8(4, 16, 96, 64) == 0
    f = B.lib.mnnllm_linear_w4a8
    assert f(p, p, p, 4, 16, 64, 64, B.F16, B.F16, p, need - 1, None) == 6       # workspace too small
    assert f(p, p, p, 4, 16, 64, 64, B.F16, B.F16, None, need, None) == 6
    assert f(p, p, p, 4, 16, 64, 64, B.F16, B.F16, p + 16, need, None) == 3      # workspace alignment
    assert f(p, p, p, 4, 16, 64, 32, B.F16, B.F16, p, need, None) == 2
    assert f(p, p, p, 4, 16, 64, 64, B.F32, B.F16, p, need, None) == 2
    assert f(None, p, p, 4, 16, 64, 64, B.F16, B.F16, p, need, None) == 1
