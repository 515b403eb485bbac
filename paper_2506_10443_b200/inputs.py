"""Seeded synthetic inputs shaped like the paper's small-LLM workloads (Section 6: Qwen2-1.5B,
Qwen2-7B, prompts of 64/256/1024 tokens, 16 decode tokens).

This module only draws random numbers and lists shapes.  It contains none of the arithmetic of the
quantised linear layer: both the CPU oracle and the CUDA library receive the arrays made here.

Every array is a pure function of an integer seed (numpy's counter-based Philox generator), so the
tests, the benchmark and the oracle all see identical data without any file on disk.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List

import numpy as np


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=int(seed) & 0xFFFFFFFFFFFFFFFF))


def weights(seed: int, N: int, K: int, std: float = 0.02) -> np.ndarray:
    """fp32 [N, K] weights ~ N(0, std^2), the distribution the workload configs state."""
    w = _rng(seed).standard_normal((N, K), dtype=np.float32)
    w *= np.float32(std)
    return w


def activations(seed: int, M: int, K: int, outliers: bool = False, dtype: str = "f16") -> np.ndarray:
    """[M, K] activations ~ N(0, 1) rounded to the I/O dtype.

    With ``outliers`` a Bernoulli(0.01) mask drawn from the same generator multiplies entries by 20
    (the prefill configs' "1 % outliers x20").  Returns a numpy float16 array for ``f16``; for
    ``bf16`` returns float32 values that are exactly representable in bfloat16.
    """
    g = _rng(seed)
    x = g.standard_normal((M, K), dtype=np.float32)
    if outliers:
        mask = g.random((M, K), dtype=np.float32) < np.float32(0.01)
        x = np.where(mask, x * np.float32(20.0), x).astype(np.float32)
    if dtype == "f16":
        return x.astype(np.float16)
    if dtype == "bf16":
        return round_to_bf16(x)
    raise ValueError(dtype)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bfloat16 (ties to even); result stays in a float32 array."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(x.shape)


def bf16_bits(x_bf16_as_f32: np.ndarray) -> np.ndarray:
    """uint16 storage bits of values that are already bfloat16-exact."""
    return (np.ascontiguousarray(x_bf16_as_f32, dtype=np.float32).view(np.uint32) >> 16).astype(np.uint16)


@dataclass(frozen=True)
class Linear:
    """One linear layer of a decoder block: y[M, N] = x[M, K] . W[N, K]^T."""

    name: str
    N: int
    K: int
    matrix_id: int


def decoder_layer(hidden: int, kv_dim: int, inter: int) -> List[Linear]:
    """The seven linears of one decoder layer in execution order (q, k, v, o, gate, up, down)."""
    return [
        Linear("q", hidden, hidden, 0),
        Linear("k", kv_dim, hidden, 1),
        Linear("v", kv_dim, hidden, 2),
        Linear("o", hidden, hidden, 3),
        Linear("gate", inter, hidden, 4),
        Linear("up", inter, hidden, 5),
        Linear("down", hidden, inter, 6),
    ]


# Shapes of the workload configs.  Qwen2-1.5B: hidden 1536, 2 kv heads x 128, intermediate 8960;
# Qwen2-7B: hidden 3584 (Table 1), 4 kv heads x 128, intermediate 18944 (Table 1); 28 layers each.
QWEN2_1P5B = dict(hidden=1536, kv_dim=256, inter=8960, layers=28)
QWEN2_7B = dict(hidden=3584, kv_dim=512, inter=18944, layers=28)
LM_HEAD = dict(N=151936, K=3584, group=128)
PROMPT_LENGTHS = (64, 256, 1024)


def w4_bytes(N: int, K: int, group: int) -> int:
    """Bytes of int4 codes plus fp16 (scale, zero) pairs of an [N, K] matrix (a byte count only)."""
    return N * K // 2 + N * (K // group) * 4


def linear_bytes(N: int, K: int, group: int, M: int, y_bytes: int = 2) -> int:
    """Bytes a W4A16 linear has to move: packed weights once, fp16 activations in, outputs out."""
    return w4_bytes(N, K, group) + 2 * M * K + y_bytes * M * N


def stack(model: dict) -> List[Linear]:
    return decoder_layer(model["hidden"], model["kv_dim"], model["inter"])


def seed_for(config: int, layer: int, matrix_id: int, what: int = 0) -> int:
    """Seed = config*1000 + layer*10 + matrix id; ``what`` separates weights (0) from activations (1)."""
    return (config * 1000 + layer * 10 + matrix_id) * 2 + what
