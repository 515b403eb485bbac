"""Helpers shared by the GPU parity tests."""
import numpy as np
import torch

import oracle
from paper_2506_10443_b200 import binding as B
from paper_2506_10443_b200 import inputs

TOL = 2e-3  # max relative error of fp16 / fp32 outputs (fp32 accumulation), see assert_close


def dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def assert_close(y_gpu: np.ndarray, y_ref: np.ndarray, tol: float = TOL):
    """|y - ref| <= tol * max(|ref|, rms of ref's row): relative error with a floor at the row's
    typical magnitude, since a pure elementwise ratio is meaningless at zero crossings."""
    y_gpu = np.asarray(y_gpu, np.float64)
    rms = np.sqrt((y_ref ** 2).mean(axis=1, keepdims=True))
    bound = tol * np.maximum(np.abs(y_ref), rms)
    err = np.abs(y_gpu - y_ref)
    worst = np.unravel_index(np.argmax(err - bound), err.shape)
    assert (err <= bound).all(), "worst at %s: got %r want %r (bound %r)" % (
        worst, y_gpu[worst], y_ref[worst], bound[worst])


def bf16_round(v: np.ndarray) -> np.ndarray:
    return inputs.round_to_bf16(np.asarray(v, np.float32)).astype(np.float64)


def assert_bf16_within_1ulp(y_gpu_f32: np.ndarray, y_ref: np.ndarray):
    """bf16 outputs: compare with the oracle value rounded to bf16, allow one bf16 ulp."""
    want = bf16_round(y_ref)
    ulp = np.maximum(np.abs(want), 2.0 ** -126) * 2.0 ** -7
    assert (np.abs(np.asarray(y_gpu_f32, np.float64) - want) <= ulp).all()


def quantized(seed, N, K, group):
    W = inputs.weights(seed, N, K)
    return W, B.pack_w4(W, group), oracle.quantize_w4(W, group)
