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


def assert_bf16_within_1ulp(y_gpu_f32: np.ndarray, y_ref: np.ndarray, fp32_tol: float = 2e-4):
    """bf16 outputs against the ORACLE value rounded to bf16: one bf16 ulp, plus the tolerance the
    fp32-output path is held to (the value that gets rounded is the kernel's fp32 sum, which may sit
    on the other side of a rounding boundary, and near a zero crossing an ulp is far below the
    row's rounding noise)."""
    y_ref = np.asarray(y_ref, np.float64)
    want = bf16_round(y_ref)
    ulp = np.maximum(np.abs(want), 2.0 ** -126) * 2.0 ** -7
    rms = np.sqrt((y_ref ** 2).mean(axis=1, keepdims=True))
    bound = ulp + fp32_tol * np.maximum(np.abs(y_ref), rms)
    err = np.abs(np.asarray(y_gpu_f32, np.float64) - want)
    worst = np.unravel_index(np.argmax(err - bound), err.shape)
    assert (err <= bound).all(), "worst at %s: got %r want %r" % (worst, y_gpu_f32[worst], want[worst])


def quantized(seed, N, K, group):
    W = inputs.weights(seed, N, K)
    return W, B.pack_w4(W, group), oracle.quantize_w4(W, group)
