"""ctypes front end of the CPU oracle (``mnnllm_oracle.cpp``).  TEST INFRASTRUCTURE: imported only by
tests, the smoke check and the benchmark's CPU-baseline legs; never by the product package.

The shared object is compiled next to the source with g++ on first use (``build()``), with
floating-point contraction off so that every fp32 operation of the quantisers rounds once, as
written.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mnnllm_oracle.cpp")
_LIB = os.path.join(_HERE, "libmnnllm_oracle.so")

__all__ = [
    "build", "num_threads", "f16_to_f32", "f32_to_f16", "quantize_w4", "quantize_w8", "dequant",
    "linear_wa16", "act_quant", "group_partials", "linear_w4a8", "linear_w8a8", "lora_bypass", "e4m3_to_f32", "f32_to_e4m3", "quantize_keys",
    "quantize_values", "attention_decode",
]


def build(force: bool = False) -> str:
    """Compile the oracle (plain g++, OpenMP over output rows) if missing or older than its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call([
            "g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
            "-fno-fast-math", _SRC, "-o", tmp,
        ])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _l():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        c = ctypes
        P = c.c_void_p
        lib.orc_f16_to_f32.restype = c.c_float
        lib.orc_f16_to_f32.argtypes = [c.c_uint16]
        lib.orc_f32_to_f16.restype = c.c_uint16
        lib.orc_f32_to_f16.argtypes = [c.c_float]
        lib.orc_quantize_w4.argtypes = [P, c.c_int, c.c_int, c.c_int, P, P, P]
        lib.orc_quantize_w8.argtypes = [P, c.c_int, c.c_int, P, P, P]
        lib.orc_dequant.argtypes = [P, P, P, c.c_int, c.c_int, c.c_int, P]
        lib.orc_linear_wa16.argtypes = [P, P, P, P, c.c_int, c.c_int, c.c_int, c.c_int, P]
        lib.orc_act_quant.argtypes = [P, c.c_int, c.c_int, c.c_int, P, P, P]
        lib.orc_group_partials.argtypes = [P, P, c.c_int, c.c_int, c.c_int, c.c_int, P]
        lib.orc_linear_w4a8.argtypes = [P, P, P, P, c.c_int, c.c_int, c.c_int, c.c_int, P]
        lib.orc_linear_w8a8.argtypes = [P, P, P, P, c.c_int, c.c_int, c.c_int, P]
        lib.orc_linear_w8a8.restype = None
        lib.orc_lora_bypass.argtypes = [P, P, P, c.c_int, c.c_int, c.c_int, c.c_int, P]
        lib.orc_lora_bypass.restype = None
        lib.orc_e4m3_to_f32.restype = c.c_float
        lib.orc_e4m3_to_f32.argtypes = [c.c_uint8]
        lib.orc_f32_to_e4m3.restype = c.c_uint8
        lib.orc_f32_to_e4m3.argtypes = [c.c_float]
        lib.orc_quantize_values.argtypes = [P, c.c_longlong, P]
        lib.orc_quantize_values.restype = None
        lib.orc_attention_decode.argtypes = [P, P, P, P, P, c.c_int, c.c_int, c.c_int, c.c_int, P]
        lib.orc_attention_decode.restype = None
        lib.orc_num_threads.restype = c.c_int
        for f in ("orc_quantize_w4", "orc_quantize_w8", "orc_dequant", "orc_linear_wa16",
                  "orc_act_quant", "orc_group_partials", "orc_linear_w4a8"):
            getattr(lib, f).restype = None
        _lib = lib
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


def linear_w8a8(x, q, s_bits, z_bits) -> np.ndarray:
    """y[M,N] fp64 of the per-channel W8A8 path (activations quantised per token inside)."""
    x = _c(x, np.float32)
    q = _c(q, np.uint8)
    M, K = x.shape
    N = q.shape[0]
    s_bits = _c(s_bits, np.uint16)
    z_bits = _c(z_bits, np.uint16)
    y = np.empty((M, N), np.float64)
    _l().orc_linear_w8a8(_p(x), _p(q), _p(s_bits), _p(z_bits), M, N, K, _p(y))
    return y


def lora_bypass(y, x, lora_A, lora_B) -> np.ndarray:
    """y + LoRA_A (LoRA_B x): y fp64 [M,N] (e.g. a linear's output), x [M,K], LoRA_A [N,r], LoRA_B [r,K]."""
    x = _c(x, np.float32)
    A = _c(lora_A, np.float32)
    Bm = _c(lora_B, np.float32)
    M, K = x.shape
    N, r = A.shape
    assert Bm.shape == (r, K)
    out = np.array(y, dtype=np.float64, order="C", copy=True)
    assert out.shape == (M, N)
    _l().orc_lora_bypass(_p(x), _p(A), _p(Bm), M, N, K, r, _p(out))
    return out


def e4m3_to_f32(bits: int) -> float:
    return float(_l().orc_e4m3_to_f32(int(bits)))


def f32_to_e4m3(x: float) -> int:
    return int(_l().orc_f32_to_e4m3(float(x)))


def quantize_keys(k: np.ndarray) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Keys [Hk, S, D] -> int8 codes per key vector (Eq. 1 along head_dim, codes 0..255): codes uint8
    [Hk, S, D], scale and zero fp16 bits [Hk, S]."""
    k = _c(k, np.float32)
    Hk, S, D = k.shape
    q, s, z = quantize_w8(k.reshape(Hk * S, D))
    return q.reshape(Hk, S, D), s.reshape(Hk, S), z.reshape(Hk, S)


def quantize_values(v: np.ndarray) -> np.ndarray:
    """Values [Hk, S, D] -> E4M3 bytes, element by element (round to nearest even, saturating at 448)."""
    v = _c(v, np.float32)
    out = np.empty(v.shape, np.uint8)
    _l().orc_quantize_values(_p(v), v.size, _p(out))
    return out


def attention_decode(q, k_codes, k_scale, k_zero, v_bytes) -> np.ndarray:
    """out[H, D] fp64 of one decoded token over the quantised cache (see orc_attention_decode)."""
    q = _c(q, np.float32)
    k_codes = _c(k_codes, np.uint8)
    k_scale = _c(k_scale, np.uint16)
    k_zero = _c(k_zero, np.uint16)
    v_bytes = _c(v_bytes, np.uint8)
    H, D = q.shape
    Hk, S, D2 = k_codes.shape
    assert D2 == D and v_bytes.shape == (Hk, S, D) and H % Hk == 0
    out = np.empty((H, D), np.float64)
    _l().orc_attention_decode(_p(q), _p(k_codes), _p(k_scale), _p(k_zero), _p(v_bytes), H, Hk, S, D, _p(out))
    return out


def num_threads() -> int:
    return int(_l().orc_num_threads())


def f16_to_f32(bits: int) -> float:
    return float(_l().orc_f16_to_f32(int(bits)))


def f32_to_f16(x: float) -> int:
    return int(_l().orc_f32_to_f16(float(x)))


def quantize_w4(W: np.ndarray, group: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Eq. 1 per (row, group): returns q uint8 [N,K] in 0..15, scale bits, zero bits (uint16 [N,G])."""
    W = _c(W, np.float32)
    N, K = W.shape
    assert K % group == 0
    q = np.empty((N, K), np.uint8)
    s = np.empty((N, K // group), np.uint16)
    z = np.empty((N, K // group), np.uint16)
    _l().orc_quantize_w4(_p(W), N, K, group, _p(q), _p(s), _p(z))
    return q, s, z


def quantize_w8(W: np.ndarray) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Per-channel Eq. 1 with codes in 0..255: q uint8 [N,K], scale/zero bits uint16 [N,1]."""
    W = _c(W, np.float32)
    N, K = W.shape
    q = np.empty((N, K), np.uint8)
    s = np.empty((N, 1), np.uint16)
    z = np.empty((N, 1), np.uint16)
    _l().orc_quantize_w8(_p(W), N, K, _p(q), _p(s), _p(z))
    return q, s, z


def dequant(q, s_bits, z_bits, group: int) -> np.ndarray:
    q = _c(q, np.uint8)
    N, K = q.shape
    s_bits = _c(s_bits, np.uint16)
    z_bits = _c(z_bits, np.uint16)
    out = np.empty((N, K), np.float64)
    _l().orc_dequant(_p(q), _p(s_bits), _p(z_bits), N, K, group, _p(out))
    return out


def linear_wa16(x, q, s_bits, z_bits, group: int) -> np.ndarray:
    """y[M,N] fp64 = x . w_hat^T for the weight-only paths (x: values of the fp16/bf16 activations)."""
    x = _c(x, np.float32)
    q = _c(q, np.uint8)
    M, K = x.shape
    N = q.shape[0]
    assert q.shape[1] == K
    s_bits = _c(s_bits, np.uint16)
    z_bits = _c(z_bits, np.uint16)
    y = np.empty((M, N), np.float64)
    _l().orc_linear_wa16(_p(x), _p(q), _p(s_bits), _p(z_bits), M, N, K, group, _p(y))
    return y


def act_quant(x, group: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Per-token symmetric int8: a_q int8 [M,K], a_scale fp32 [M], A_g int32 [M,G]."""
    x = _c(x, np.float32)
    M, K = x.shape
    a_q = np.empty((M, K), np.int8)
    a_scale = np.empty((M,), np.float32)
    A_g = np.empty((M, K // group), np.int32)
    _l().orc_act_quant(_p(x), M, K, group, _p(a_q), _p(a_scale), _p(A_g))
    return a_q, a_scale, A_g


def group_partials(a_q, q, group: int) -> np.ndarray:
    """P[M,N,G] int32 = per-group integer dot products of a_q rows with q rows."""
    a_q = _c(a_q, np.int8)
    q = _c(q, np.uint8)
    M, K = a_q.shape
    N = q.shape[0]
    P = np.empty((M, N, K // group), np.int32)
    _l().orc_group_partials(_p(a_q), _p(q), M, N, K, group, _p(P))
    return P


def linear_w4a8(x, q, s_bits, z_bits, group: int) -> np.ndarray:
    """y[M,N] fp64 of the W4A8 path (activations quantised per token inside)."""
    x = _c(x, np.float32)
    q = _c(q, np.uint8)
    M, K = x.shape
    N = q.shape[0]
    s_bits = _c(s_bits, np.uint16)
    z_bits = _c(z_bits, np.uint16)
    y = np.empty((M, N), np.float64)
    _l().orc_linear_w4a8(_p(x), _p(q), _p(s_bits), _p(z_bits), M, N, K, group, _p(y))
    return y
