"""Parity at the full sizes of the workload list, through the same entry points and launch
configurations that bench.py times.  The oracle is too slow for whole outputs at these sizes, so a
seeded sample of output channels is recomputed one by one (a row of W is independent of the
others: quantising a subset of rows gives the same codes as quantising all of them)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_10443_b200 import binding as B
from paper_2506_10443_b200 import inputs
from paper_2506_10443_b200.workloads import LinearStack
from gpu_util import assert_close, dev

pytestmark = pytest.mark.gpu


def sample_rows(N, count, seed):
    rows = np.random.default_rng(seed).choice(N, size=min(count, N), replace=False)
    rows[:3] = [0, N - 1, (N // 16) * 16 - 1 if N >= 16 else 0]   # both ends and the last full 16-row block
    return np.unique(rows)


def ref_rows_wa16(W, rows, x, group):
    q, s, z = oracle.quantize_w4(W[rows], group)
    return oracle.linear_wa16(x.astype(np.float32), q, s, z, group)


def close_cols(y_gpu_rows, ref):
    # tolerance floor from the sampled outputs of the same token (the row rms of the sample)
    assert_close(y_gpu_rows, ref)


@pytest.mark.parametrize("model,config", [(inputs.QWEN2_1P5B, 2), (inputs.QWEN2_7B, 4)])
def test_decode_stack_layer_as_benchmarked(model, config):
    # one decoder layer issued exactly as bench.py issues it (q+k+v and gate+up batched launches)
    stack = LinearStack(model, config, 1, 64, layers=1)
    stack.run_w4a16()
    assert B.read_status() == 0
    for lin in stack.linears:
        W = inputs.weights(inputs.seed_for(config, 0, lin.matrix_id, 0), lin.N, lin.K)
        rows = sample_rows(lin.N, 96, lin.matrix_id)
        x = stack.x_view(0, lin.name).cpu().numpy()
        y = stack.y_view(0, lin.name).float().cpu().numpy()[:, rows]
        close_cols(y, ref_rows_wa16(W, rows, x, 64))


@pytest.mark.parametrize("M", [1, 4])
def test_lm_head_w4_group128_fp32_logits(M):
    N, K, group = inputs.LM_HEAD["N"], inputs.LM_HEAD["K"], inputs.LM_HEAD["group"]
    W = inputs.weights(5000, N, K)
    pd = dev(B.pack_w4(W, group))
    x = inputs.activations(5001 + M, M, K)
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    B.linear_w4a16_ex(dev(x), pd, y, M, N, K, group, B.F16, B.F32)
    assert B.read_status() == 0
    yh = y.cpu().numpy()
    assert np.isfinite(yh).all()
    rows = sample_rows(N, 128, 7)
    close_cols(yh[:, rows], ref_rows_wa16(W, rows, x, group))


def test_lm_head_w8_per_channel_fp32_logits():
    N, K, M = inputs.LM_HEAD["N"], inputs.LM_HEAD["K"], 4
    W = inputs.weights(5100, N, K)
    pd = dev(B.pack_w8(W))
    x = inputs.activations(5101, M, K)
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    B.linear_w8a16(dev(x), pd, y, M, N, K, B.F32)
    assert B.read_status() == 0
    yh = y.cpu().numpy()
    assert np.isfinite(yh).all()
    rows = sample_rows(N, 128, 8)
    q, s, z = oracle.quantize_w8(W[rows])
    close_cols(yh[:, rows], oracle.linear_wa16(x.astype(np.float32), q, s, z, K))


@pytest.mark.parametrize("model,config,M,names", [
    (inputs.QWEN2_1P5B, 3, 1024, ("q", "k", "gate", "down")),
    (inputs.QWEN2_1P5B, 3, 256, ("q", "o", "down")),   # o and down: tiles cut along K
    (inputs.QWEN2_1P5B, 3, 64, ("v", "down")),
    (inputs.QWEN2_7B, 4, 512, ("o", "up", "down")),
])
def test_prefill_layer_as_benchmarked(model, config, M, names):
    stack = LinearStack(model, config, M, 64, layers=1, outliers=True)
    stack.run_w4a8()
    assert B.read_status() == 0
    tokens = np.unique(np.concatenate([[0, M - 1], np.random.default_rng(M).choice(M, 14, replace=False)]))
    for lin in stack.linears:
        if lin.name not in names:
            continue
        W = inputs.weights(inputs.seed_for(config, 0, lin.matrix_id, 0), lin.N, lin.K)
        rows = sample_rows(lin.N, 48, lin.matrix_id + M)
        q, s, z = oracle.quantize_w4(W[rows], 64)
        x = stack.x_view(0, lin.name).cpu().numpy()[tokens]
        ref = oracle.linear_w4a8(x.astype(np.float32), q, s, z, 64)
        y = stack.y_view(0, lin.name).float().cpu().numpy()[np.ix_(tokens, rows)]
        close_cols(y, ref)


def test_prefill_group_partials_full_K_sampled():
    # the longest K of the workloads (down projection of Qwen2-7B): every group partial of a slab
    # of outputs, bit for bit
    M, N, K, group = 150, 256, 18944, 64
    W = inputs.weights(6000, N, K)
    x = inputs.activations(6001, M, K, outliers=True)
    G = K // group
    P = torch.empty((M, N, G), dtype=torch.int32, device="cuda")
    a_q = torch.empty((M, K), dtype=torch.int8, device="cuda")
    a_scale = torch.empty((M,), dtype=torch.float32, device="cuda")
    A = torch.empty((M, G), dtype=torch.int32, device="cuda")
    B.debug_w4a8_partials(dev(x), dev(B.pack_w4(W, group)), P, a_q, a_scale, A, M, N, K, group)
    assert B.read_status() == 0
    q, _, _ = oracle.quantize_w4(W, group)
    aq0, _, _ = oracle.act_quant(x.astype(np.float32), group)
    assert (P.cpu().numpy() == oracle.group_partials(aq0, q, group)).all()
