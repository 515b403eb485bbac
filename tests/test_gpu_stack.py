"""GPU parity of the one-launch decoder stack (mnnllm_linear_w4a16_stack) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_10443_b200 import binding as B
from paper_2506_10443_b200 import inputs
from gpu_util import assert_close, dev, quantized

pytestmark = pytest.mark.gpu

TDT = {B.F16: torch.float16, B.BF16: torch.bfloat16, B.F32: torch.float32}


class Stack:
    """A list of linears run through the stack entry: (N, K, deps, x_from) per problem; with
    x_from = j the input IS problem j's fp16 output (N_j == K): a true data dependency."""

    def __init__(self, shapes, M, group, seed, y_dtype=B.F16):
        self.M, self.group = M, group
        self.q, self.x_np, self.y, self.x_dev, keep = [], [], [], [], []
        probs = []
        for i, (N, K, deps, x_from) in enumerate(shapes):
            W, packed, qsz = quantized(seed + 17 * i, N, K, group)
            self.q.append(qsz)
            pd = dev(packed)
            keep.append(pd)
            dt = B.F16 if any(s[3] == i for s in shapes) else y_dtype
            y = torch.full((M, N), float("nan"), dtype=TDT[dt], device="cuda")
            self.y.append(y)
            if x_from is None:
                x = inputs.activations(seed + 1000 + i, M, K)
                self.x_np.append(x)
                xd = dev(x)
            else:
                assert shapes[x_from][0] == K
                self.x_np.append(None)
                xd = self.y[x_from]
            self.x_dev.append(xd)
            probs.append(dict(x=xd, packed=pd, y=y, N=N, K=K, y_dtype=dt, deps=deps))
        self.shapes, self._keep = shapes, keep
        self.plan = B.stack_plan_w4a16(probs, M, group)
        self.plan_dev = dev(self.plan)
        self.ws_bytes = B.stack_workspace_size(self.plan)
        self.ws = torch.empty(self.ws_bytes, dtype=torch.uint8, device="cuda")
        B.stack_workspace_init(self.ws, self.ws_bytes)

    def run(self, stream=None):
        B.linear_w4a16_stack(self.plan, self.plan_dev, self.ws, self.ws_bytes, stream)

    def check(self, tol=2e-3):
        outs = [y.float().cpu().numpy() for y in self.y]
        for i, (N, K, deps, x_from) in enumerate(self.shapes):
            q, s, z = self.q[i]
            # a chained problem is checked against the oracle applied to the GPU's own (already
            # checked) fp16 output of its predecessor: errors do not compound through the chain
            x = self.x_np[i].astype(np.float32) if x_from is None else outs[x_from].astype(np.float32)
            assert_close(outs[i], oracle.linear_wa16(x, q, s, z, self.group), tol)


def test_stack_independent_problems():
    st = Stack([(256, 1536, (), None), (40, 192, (), None), (1536, 8960, (), None), (100, 8960, (), None),
                (16, 64, (), None), (2000, 1536, (), None)], 1, 64, seed=11)
    st.run()
    assert B.read_status() == 0
    st.check()


@pytest.mark.parametrize("M", [1, 2, 3, 4, 8])
def test_stack_chain_with_data_dependencies(M):
    # q, k, v on one input; o reads v's output (K = 512); gate, up read o's; down reads gate's
    shapes = [(512, 1024, (), None), (128, 1024, (), None), (512, 1024, (), None),
              (1024, 512, (0, 1, 2), 2), (2560, 1024, (3,), 3), (2560, 1024, (3,), 3), (1024, 2560, (4, 5), 4)]
    st = Stack(shapes, M, 64, seed=100 + M)
    for _ in range(3):   # the counters carry over from launch to launch
        st.run()
    assert B.read_status() == 0
    st.check()


def test_stack_group128_and_output_dtypes():
    shapes = [(130, 3584, (), None), (1000, 3584, (0,), None), (64, 640, (1,), None)]
    for dt in (B.F32, B.BF16):
        st = Stack(shapes, 4, 128, seed=7, y_dtype=dt)
        st.run()
        assert B.read_status() == 0
        st.check(2e-3 if dt == B.F32 else 2.0 ** -8 + 2e-4)


def test_stack_matches_single_launches_bitwise_in_fp32_order_free_case():
    # exact case: weights on the grid, small integer activations: every sum is exact in fp32
    rng = np.random.default_rng(5)
    N, K, group, M = 1536, 8960, 64, 2
    qi = rng.integers(0, 16, (N, K))
    qi[:, ::64] = 0
    qi[:, 1::64] = 15
    zero = rng.integers(0, 16, (N, K // group))
    W = ((qi - np.repeat(zero, group, axis=1)) * 0.125).astype(np.float32)
    x = rng.integers(-8, 9, (M, K)).astype(np.float16)
    pd, xd = dev(B.pack_w4(W, group)), dev(x)
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    plan = B.stack_plan_w4a16([dict(x=xd, packed=pd, y=y, N=N, K=K, y_dtype=B.F32)], M, group)
    ws_bytes = B.stack_workspace_size(plan)
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device="cuda")
    B.linear_w4a16_stack(plan, dev(plan), ws, ws_bytes)
    assert B.read_status() == 0
    want = x.astype(np.float64) @ W.astype(np.float64).T
    assert (y.cpu().numpy() == want).all()


def test_stack_graph_replay_is_bit_identical():
    shapes = [(1536, 1536, (), None), (1536, 8960, (0,), None), (8960, 1536, (1,), 1)]
    st = Stack(shapes, 1, 64, seed=31)
    st.run()
    assert B.read_status() == 0
    first = [y.clone() for y in st.y]
    g = torch.cuda.CUDAGraph()
    cap = torch.cuda.Stream()
    cap.wait_stream(torch.cuda.current_stream())
    with torch.cuda.graph(g, stream=cap):
        st.run(cap)
    for _ in range(5):
        g.replay()
    assert B.read_status() == 0
    for a, b in zip(first, st.y):
        assert torch.equal(a, b)
    st.check()


def test_stack_argument_errors():
    x = torch.zeros((1, 1536), dtype=torch.float16, device="cuda")
    y = torch.zeros((1, 256), dtype=torch.float16, device="cuda")
    _, packed, _ = quantized(3, 256, 1536, 64)
    pd = dev(packed)
    good = dict(x=x, packed=pd, y=y, N=256, K=1536)
    with pytest.raises(B.MnnllmError) as e:
        B.stack_plan_w4a16([dict(good, deps=(0,))], 1, 64)       # depends on itself
    assert e.value.status == 1
    with pytest.raises(B.MnnllmError) as e:
        B.stack_plan_w4a16([good], 9, 64)                        # more than 8 tokens
    assert e.value.status == 2
    plan = B.stack_plan_w4a16([good], 1, 64)
    ws = torch.zeros(B.stack_workspace_size(plan), dtype=torch.uint8, device="cuda")
    with pytest.raises(B.MnnllmError) as e:
        B.linear_w4a16_stack(plan, dev(plan), ws, ws.numel() - 1)
    assert e.value.status == 6
