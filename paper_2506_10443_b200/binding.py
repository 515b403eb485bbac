"""ctypes binding of ``libmnnllm_b200.so``: the same names as ``include/mnnllm.h`` without the
``mnnllm_`` prefix, argument marshalling only.  Device buffers are passed as ``torch.Tensor`` (their
``data_ptr()`` is used) or as raw integer addresses; streams as ``torch.cuda.Stream``, a raw
``cudaStream_t`` integer, or ``None`` for torch's current stream.

There is no fallback: if the library has not been built, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmnnllm_b200.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        "libmnnllm_b200.so is missing: build it with `python -m paper_2506_10443_b200.build` "
        "(there is no CPU or PyTorch fallback)")

lib = ctypes.CDLL(LIB_PATH)

F16, BF16, F32 = 0, 1, 2
OK = 0
MAX_BATCH = 8
_c = ctypes
_P = _c.c_void_p


class MnnllmError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        lib.mnnllm_status_string.restype = _c.c_char_p
        super().__init__("%s: %s (status %d)" % (where, lib.mnnllm_status_string(status).decode(), status))


class _ProblemW4A8(_c.Structure):
    _fields_ = [("packed", _P), ("y", _P), ("N", _c.c_int), ("y_dtype", _c.c_int)]


class _Problem(_c.Structure):
    _fields_ = [("x", _P), ("packed", _P), ("y", _P), ("N", _c.c_int), ("K", _c.c_int), ("group", _c.c_int),
                ("y_dtype", _c.c_int)]


class _StackProblem(_c.Structure):
    _fields_ = [("x", _P), ("packed", _P), ("y", _P), ("N", _c.c_int), ("K", _c.c_int), ("y_dtype", _c.c_int),
                ("n_deps", _c.c_int), ("deps", _c.c_int * 4)]


def _sig(name, restype, argtypes):
    f = getattr(lib, name)
    f.restype = restype
    f.argtypes = argtypes
    return f


_sig("mnnllm_status_string", _c.c_char_p, [_c.c_int])
_sig("mnnllm_packed_size_w4", _c.c_size_t, [_c.c_int, _c.c_int, _c.c_int])
_sig("mnnllm_pack_w4", _c.c_int, [_P, _c.c_int, _c.c_int, _c.c_int, _P])
_sig("mnnllm_unpack_w4", _c.c_int, [_P, _P, _P, _P])
_sig("mnnllm_packed_info", _c.c_int, [_P, _P, _P, _P, _P])
_sig("mnnllm_packed_size_w8", _c.c_size_t, [_c.c_int, _c.c_int])
_sig("mnnllm_pack_w8", _c.c_int, [_P, _c.c_int, _c.c_int, _P])
_sig("mnnllm_unpack_w8", _c.c_int, [_P, _P, _P, _P])
_sig("mnnllm_linear_w4a16", _c.c_int, [_P, _P, _P, _c.c_int, _c.c_int, _c.c_int, _c.c_int, _P])
_sig("mnnllm_linear_w4a16_ex", _c.c_int,
     [_P, _P, _P, _c.c_int, _c.c_int, _c.c_int, _c.c_int, _c.c_int, _c.c_int, _P])
_sig("mnnllm_linear_w4a16_batch", _c.c_int, [_c.POINTER(_Problem), _c.c_int, _c.c_int, _P])
_sig("mnnllm_stack_plan_size", _c.c_size_t, [_c.c_int])
_sig("mnnllm_stack_plan_w4a16", _c.c_int, [_c.POINTER(_StackProblem), _c.c_int, _c.c_int, _c.c_int, _c.c_int, _P])
_sig("mnnllm_stack_workspace_size", _c.c_size_t, [_P])
_sig("mnnllm_stack_workspace_init", _c.c_int, [_P, _c.c_size_t, _P])
_sig("mnnllm_linear_w4a16_stack", _c.c_int, [_P, _P, _P, _c.c_size_t, _P])
_sig("mnnllm_linear_w8a16", _c.c_int, [_P, _P, _P, _c.c_int, _c.c_int, _c.c_int, _c.c_int, _P])
_sig("mnnllm_workspace_size_lora", _c.c_size_t, [_c.c_int, _c.c_int])
_sig("mnnllm_lora_workspace_init", _c.c_int, [_P, _c.c_size_t, _P])
_sig("mnnllm_linear_w4a16_lora", _c.c_int, [_P, _P, _P, _P, _P] + [_c.c_int] * 7 + [_P, _c.c_size_t, _P])
_sig("mnnllm_kv_append", _c.c_int, [_P, _P, _P, _c.c_int, _c.c_int, _c.c_int, _c.c_int, _P, _P, _P])
_sig("mnnllm_attention_workspace_size", _c.c_size_t, [_c.c_int, _c.c_int, _c.c_int])
_sig("mnnllm_attention_workspace_init", _c.c_int, [_P, _c.c_size_t, _P])
_sig("mnnllm_attention_decode", _c.c_int, [_P, _P, _P, _P, _P] + [_c.c_int] * 6 + [_P, _c.c_size_t, _P])
_sig("mnnllm_workspace_size_w8a8", _c.c_size_t, [_c.c_int, _c.c_int])
_sig("mnnllm_linear_w8a8", _c.c_int, [_P, _P, _P, _c.c_int, _c.c_int, _c.c_int, _c.c_int, _c.c_int, _P, _c.c_size_t, _P])
_sig("mnnllm_workspace_size_w4a8", _c.c_size_t, [_c.c_int, _c.c_int, _c.c_int, _c.c_int])
_sig("mnnllm_workspace_min_w4a8", _c.c_size_t, [_c.c_int, _c.c_int, _c.c_int, _c.c_int])
_sig("mnnllm_linear_w4a8", _c.c_int,
     [_P, _P, _P, _c.c_int, _c.c_int, _c.c_int, _c.c_int, _c.c_int, _c.c_int, _P, _c.c_size_t, _P])
_sig("mnnllm_linear_w4a8_batch", _c.c_int,
     [_c.POINTER(_ProblemW4A8), _c.c_int, _P, _c.c_int, _c.c_int, _c.c_int, _c.c_int, _P, _c.c_size_t, _P])
_sig("mnnllm_linear_w4a8_static", _c.c_int,
     [_P, _P, _P, _c.c_int, _c.c_int, _c.c_int, _c.c_int, _c.c_int, _c.c_int, _P])
_sig("mnnllm_quantize_activations", _c.c_int, [_P, _c.c_int, _c.c_int, _c.c_int, _c.c_int, _P, _P, _P, _P])
_sig("mnnllm_debug_w4a8_partials", _c.c_int,
     [_P, _c.c_int, _P, _P, _P, _P, _P, _c.c_int, _c.c_int, _c.c_int, _c.c_int, _P])
_sig("mnnllm_debug_set_w4a8_small_max", _c.c_int, [_c.c_int])
_sig("mnnllm_debug_set_w4a8_limb", _c.c_int, [_c.c_int])
_sig("mnnllm_debug_wait_timeout", _c.c_int, [_c.c_int, _P])
_sig("mnnllm_bench_mma_i8", _c.c_int, [_c.c_ulonglong, _P, _P])
_sig("mnnllm_read_status", _c.c_int, [_P, _c.POINTER(_c.c_uint32)])
_sig("mnnllm_device_supported", _c.c_int, [])

EXPORTS = [
    "mnnllm_status_string", "mnnllm_packed_size_w4", "mnnllm_pack_w4", "mnnllm_unpack_w4", "mnnllm_packed_info",
    "mnnllm_packed_size_w8", "mnnllm_pack_w8", "mnnllm_unpack_w8", "mnnllm_linear_w4a16", "mnnllm_linear_w4a16_ex",
    "mnnllm_linear_w4a16_batch", "mnnllm_stack_plan_size", "mnnllm_stack_plan_w4a16", "mnnllm_stack_workspace_size",
    "mnnllm_stack_workspace_init", "mnnllm_linear_w4a16_stack", "mnnllm_linear_w8a16", "mnnllm_kv_append", "mnnllm_attention_workspace_size", "mnnllm_attention_workspace_init",
    "mnnllm_attention_decode", "mnnllm_workspace_size_lora", "mnnllm_lora_workspace_init", "mnnllm_linear_w4a16_lora", "mnnllm_workspace_size_w8a8", "mnnllm_linear_w8a8", "mnnllm_workspace_size_w4a8", "mnnllm_workspace_min_w4a8", "mnnllm_linear_w4a8", "mnnllm_linear_w4a8_batch", "mnnllm_linear_w4a8_static",
    "mnnllm_quantize_activations", "mnnllm_debug_w4a8_partials", "mnnllm_debug_set_w4a8_small_max", "mnnllm_debug_set_w4a8_limb", "mnnllm_debug_wait_timeout", "mnnllm_bench_mma_i8", "mnnllm_read_status", "mnnllm_device_supported",
]


def _ptr(t) -> int:
    if t is None:
        return 0
    if isinstance(t, int):
        return t
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return int(t.data_ptr())  # torch.Tensor


def _stream(stream) -> int:
    if stream is None:
        import torch
        return int(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, int):
        return stream
    return int(stream.cuda_stream)


def _check(status: int, where: str) -> None:
    if status != OK:
        raise MnnllmError(status, where)


# ---- host side ---------------------------------------------------------------------------------
def packed_size_w4(N: int, K: int, group: int) -> int:
    return int(lib.mnnllm_packed_size_w4(N, K, group))


def pack_w4(W: np.ndarray, group: int) -> np.ndarray:
    """fp32 [N, K] host weights -> packed uint8 host buffer (128-byte aligned)."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    N, K = W.shape
    size = packed_size_w4(N, K, group)
    if size == 0:
        raise MnnllmError(2, "packed_size_w4(%d, %d, %d)" % (N, K, group))
    out = aligned_empty(size)
    _check(lib.mnnllm_pack_w4(_ptr(W), N, K, group, _ptr(out)), "pack_w4")
    return out


def unpack_w4(packed: np.ndarray) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    N, K, group, bits = packed_info(packed)
    q = np.empty((N, K), np.uint8)
    s = np.empty((N, K // group), np.uint16)
    z = np.empty((N, K // group), np.uint16)
    _check(lib.mnnllm_unpack_w4(_ptr(packed), _ptr(q), _ptr(s), _ptr(z)), "unpack_w4")
    return q, s, z


def packed_info(packed: np.ndarray) -> Tuple[int, int, int, int]:
    v = [_c.c_int(0) for _ in range(4)]
    _check(lib.mnnllm_packed_info(_ptr(packed), *[_c.addressof(x) for x in v]), "packed_info")
    return tuple(int(x.value) for x in v)


def packed_size_w8(N: int, K: int) -> int:
    return int(lib.mnnllm_packed_size_w8(N, K))


def pack_w8(W: np.ndarray) -> np.ndarray:
    W = np.ascontiguousarray(W, dtype=np.float32)
    N, K = W.shape
    size = packed_size_w8(N, K)
    if size == 0:
        raise MnnllmError(2, "packed_size_w8(%d, %d)" % (N, K))
    out = aligned_empty(size)
    _check(lib.mnnllm_pack_w8(_ptr(W), N, K, _ptr(out)), "pack_w8")
    return out


def unpack_w8(packed: np.ndarray) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    N, K, group, bits = packed_info(packed)
    q = np.empty((N, K), np.uint8)
    s = np.empty((N, 1), np.uint16)
    z = np.empty((N, 1), np.uint16)
    _check(lib.mnnllm_unpack_w8(_ptr(packed), _ptr(q), _ptr(s), _ptr(z)), "unpack_w8")
    return q, s, z


def aligned_empty(nbytes: int, align: int = 128) -> np.ndarray:
    """Uninitialised uint8 host array whose address is a multiple of ``align``."""
    raw = np.empty(nbytes + align, np.uint8)
    off = (-raw.ctypes.data) % align
    return raw[off:off + nbytes]


# ---- device side -------------------------------------------------------------------------------
def device_supported() -> bool:
    return bool(lib.mnnllm_device_supported())


def linear_w4a16(x, packed, y, M: int, N: int, K: int, group: int, stream=None) -> None:
    _check(lib.mnnllm_linear_w4a16(_ptr(x), _ptr(packed), _ptr(y), M, N, K, group, _stream(stream)), "linear_w4a16")


def linear_w4a16_ex(x, packed, y, M, N, K, group, x_dtype=F16, y_dtype=F16, stream=None) -> None:
    _check(lib.mnnllm_linear_w4a16_ex(_ptr(x), _ptr(packed), _ptr(y), M, N, K, group, x_dtype, y_dtype,
                                      _stream(stream)), "linear_w4a16_ex")


def make_batch(problems: Sequence[dict]):
    """Marshals a list of dicts (x, packed, y, N, K, group, y_dtype) into the C array once, so that a
    benchmark loop can re-issue the same launch without Python-side allocation."""
    arr = (_Problem * len(problems))()
    for a, p in zip(arr, problems):
        a.x, a.packed, a.y = _ptr(p["x"]), _ptr(p["packed"]), _ptr(p["y"])
        a.N, a.K, a.group, a.y_dtype = p["N"], p["K"], p["group"], p.get("y_dtype", F16)
    return arr


def linear_w4a16_batch(problems, M: int, stream=None) -> None:
    arr = problems if isinstance(problems, _c.Array) else make_batch(problems)
    _check(lib.mnnllm_linear_w4a16_batch(arr, len(arr), M, _stream(stream)), "linear_w4a16_batch")


def stack_plan_w4a16(problems: Sequence[dict], M: int, group: int, n_sms: int = 0) -> np.ndarray:
    """Host plan of ``linear_w4a16_stack`` for a list of dicts (x, packed, y, N, K, y_dtype, deps).
    ``n_sms = 0`` plans for the current device.  Returns the plan as a uint8 host array; the caller
    copies it to the device."""
    arr = (_StackProblem * len(problems))()
    for a, p in zip(arr, problems):
        a.x, a.packed, a.y = _ptr(p["x"]), _ptr(p["packed"]), _ptr(p["y"])
        a.N, a.K, a.y_dtype = p["N"], p["K"], p.get("y_dtype", F16)
        deps = list(p.get("deps", ()))
        a.n_deps = len(deps)
        for i, d in enumerate(deps[:4]):
            a.deps[i] = d
    size = int(lib.mnnllm_stack_plan_size(len(arr)))
    if size == 0:
        raise MnnllmError(1, "stack_plan_size(%d)" % len(arr))
    out = aligned_empty(size)
    _check(lib.mnnllm_stack_plan_w4a16(arr, len(arr), M, group, n_sms, _ptr(out)), "stack_plan_w4a16")
    return out


def stack_workspace_size(plan_host: np.ndarray) -> int:
    return int(lib.mnnllm_stack_workspace_size(_ptr(plan_host)))


def stack_workspace_init(workspace, workspace_bytes: int, stream=None) -> None:
    _check(lib.mnnllm_stack_workspace_init(_ptr(workspace), workspace_bytes, _stream(stream)), "stack_workspace_init")


def linear_w4a16_stack(plan_host: np.ndarray, plan_dev, workspace, workspace_bytes: int, stream=None) -> None:
    _check(lib.mnnllm_linear_w4a16_stack(_ptr(plan_host), _ptr(plan_dev), _ptr(workspace), workspace_bytes,
                                         _stream(stream)), "linear_w4a16_stack")


def linear_w8a16(x, packed, y, M, N, K, y_dtype=F16, stream=None) -> None:
    _check(lib.mnnllm_linear_w8a16(_ptr(x), _ptr(packed), _ptr(y), M, N, K, y_dtype, _stream(stream)), "linear_w8a16")


def workspace_size_w4a8(M: int, N: int, K: int, group: int) -> int:
    return int(lib.mnnllm_workspace_size_w4a8(M, N, K, group))


def workspace_min_w4a8(M: int, N: int, K: int, group: int) -> int:
    return int(lib.mnnllm_workspace_min_w4a8(M, N, K, group))


def linear_w4a8(x, packed, y, M, N, K, group, workspace, workspace_bytes, x_dtype=F16, y_dtype=F16,
                stream=None) -> None:
    _check(lib.mnnllm_linear_w4a8(_ptr(x), _ptr(packed), _ptr(y), M, N, K, group, x_dtype, y_dtype, _ptr(workspace),
                                  workspace_bytes, _stream(stream)), "linear_w4a8")


def workspace_size_lora(M: int, rank: int) -> int:
    return int(lib.mnnllm_workspace_size_lora(M, rank))


def lora_workspace_init(workspace, workspace_bytes, stream=None) -> None:
    """Clears the counters of a LoRA workspace: once, before its first use."""
    _check(lib.mnnllm_lora_workspace_init(_ptr(workspace), workspace_bytes, _stream(stream)), "lora_workspace_init")


def linear_w4a16_lora(x, packed, lora_A, lora_B, y, M, N, K, group, rank, workspace, workspace_bytes, x_dtype=F16,
                      y_dtype=F16, stream=None) -> None:
    """W4A16 linear plus the LoRA bypass ``lora_A (lora_B x)``; lora_A fp16 [N, rank], lora_B fp16 [rank, K]."""
    _check(lib.mnnllm_linear_w4a16_lora(_ptr(x), _ptr(packed), _ptr(lora_A), _ptr(lora_B), _ptr(y), M, N, K, group, rank,
                                        x_dtype, y_dtype, _ptr(workspace), workspace_bytes, _stream(stream)),
           "linear_w4a16_lora")


def kv_append(k_codes, k_meta, v, Hk, S_cap, pos, k_new, v_new, head_dim=128, stream=None) -> None:
    """Quantises one new key (int8, Eq. 1 per key vector) and value (E4M3) per kv head into the cache at ``pos``."""
    _check(lib.mnnllm_kv_append(_ptr(k_codes), _ptr(k_meta), _ptr(v), Hk, S_cap, head_dim, pos, _ptr(k_new), _ptr(v_new),
                                _stream(stream)), "kv_append")


def attention_workspace_size(H: int, Hk: int, S: int) -> int:
    return int(lib.mnnllm_attention_workspace_size(H, Hk, S))


def attention_workspace_init(workspace, workspace_bytes, stream=None) -> None:
    _check(lib.mnnllm_attention_workspace_init(_ptr(workspace), workspace_bytes, _stream(stream)), "attention_workspace_init")


def attention_decode(q, k_codes, k_meta, v, out, H, Hk, S, S_cap, workspace, workspace_bytes, out_dtype=F16, head_dim=128,
                     stream=None) -> None:
    """One decoded token's attention over the quantised cache: q fp16 [H, 128] -> out [H, 128]."""
    _check(lib.mnnllm_attention_decode(_ptr(q), _ptr(k_codes), _ptr(k_meta), _ptr(v), _ptr(out), H, Hk, head_dim, S, S_cap,
                                       out_dtype, _ptr(workspace), workspace_bytes, _stream(stream)), "attention_decode")


def workspace_size_w8a8(M: int, K: int) -> int:
    return int(lib.mnnllm_workspace_size_w8a8(M, K))


def linear_w8a8(x, packed, y, M, N, K, workspace, workspace_bytes, x_dtype=F16, y_dtype=F16, stream=None) -> None:
    """Per-channel W8A8 linear (weights packed by ``pack_w8``)."""
    _check(lib.mnnllm_linear_w8a8(_ptr(x), _ptr(packed), _ptr(y), M, N, K, x_dtype, y_dtype, _ptr(workspace),
                                  workspace_bytes, _stream(stream)), "linear_w8a8")


def make_batch_w4a8(problems: Sequence[dict]):
    """Marshals dicts (packed, y, N, y_dtype) into the C array of ``linear_w4a8_batch``."""
    arr = (_ProblemW4A8 * len(problems))()
    for a, p in zip(arr, problems):
        a.packed, a.y, a.N, a.y_dtype = _ptr(p["packed"]), _ptr(p["y"]), p["N"], p.get("y_dtype", F16)
    return arr


def linear_w4a8_batch(problems, x, M, K, group, workspace, workspace_bytes, x_dtype=F16, stream=None) -> None:
    """Weight matrices that share the activations ``x``: one quantiser pass, one GEMM launch."""
    arr = problems if isinstance(problems, _c.Array) else make_batch_w4a8(problems)
    _check(lib.mnnllm_linear_w4a8_batch(arr, len(arr), _ptr(x), M, K, group, x_dtype, _ptr(workspace), workspace_bytes,
                                        _stream(stream)), "linear_w4a8_batch")


STATIC_SCRATCH_BYTES = 8 << 20


def linear_w4a8_static(x, packed, y, M, N, K, group, x_dtype=F16, y_dtype=F16, stream=None) -> None:
    """W4A8 linear that needs no workspace from the caller: for code that may not allocate device
    memory.  The scratch is a fixed ``STATIC_SCRATCH_BYTES`` array inside the library; problems that
    need more raise ``MnnllmError`` (status 6).  Calls that may overlap on the GPU share that
    array and race; keep them on one stream."""
    _check(lib.mnnllm_linear_w4a8_static(_ptr(x), _ptr(packed), _ptr(y), M, N, K, group, x_dtype, y_dtype,
                                         _stream(stream)), "linear_w4a8_static")


def quantize_activations(x, M, K, group, a_q, a_scale, A, x_dtype=F16, stream=None) -> None:
    _check(lib.mnnllm_quantize_activations(_ptr(x), x_dtype, M, K, group, _ptr(a_q), _ptr(a_scale), _ptr(A),
                                           _stream(stream)), "quantize_activations")


def debug_w4a8_partials(x, packed, P, a_q, a_scale, A, M, N, K, group, x_dtype=F16, stream=None) -> None:
    _check(lib.mnnllm_debug_w4a8_partials(_ptr(x), x_dtype, _ptr(packed), _ptr(P), _ptr(a_q), _ptr(a_scale), _ptr(A),
                                          M, N, K, group, _stream(stream)), "debug_w4a8_partials")


def debug_set_w4a8_small_max(max_tokens: int) -> int:
    """Moves the token count up to which ``linear_w4a8`` uses its short-prompt kernel (0..64; -1 restores
    the default); returns the value in force before."""
    return int(lib.mnnllm_debug_set_w4a8_small_max(max_tokens))


def debug_set_w4a8_limb(enabled: int) -> int:
    """Switches the integer-limb prefill GEMM (an alternative, off by default) off (0), on (1) or on
    whatever the number of tiles (2); -1 restores the default.  Returns 1 if it was on before."""
    return int(lib.mnnllm_debug_set_w4a8_limb(enabled))


DEBUG_TIMEOUT_DETAIL = 0x2000


def debug_wait_timeout(max_polls: int = 3, stream=None) -> None:
    """Enqueues a kernel whose bounded wait runs out on purpose (it records a status code and ends)."""
    _check(lib.mnnllm_debug_wait_timeout(max_polls, _stream(stream)), "debug_wait_timeout")


def bench_mma_i8(mmas_per_sm: int, cycles_out=None, stream=None) -> None:
    """Enqueues the int8 tensor-rate ceiling kernel (see mnnllm_bench_mma_i8)."""
    _check(lib.mnnllm_bench_mma_i8(mmas_per_sm, _ptr(cycles_out), _stream(stream)), "bench_mma_i8")


def read_status_code(stream=None):
    """(status, detail) of ``mnnllm_read_status``: status 0 or 5 (time-out), detail the raw word."""
    detail = _c.c_uint32(0)
    st = lib.mnnllm_read_status(_stream(stream), _c.byref(detail))
    return int(st), int(detail.value)


def read_status(stream=None) -> int:
    """Synchronises the stream and returns the device status word (0 = no bounded wait gave up)."""
    detail = _c.c_uint32(0)
    st = lib.mnnllm_read_status(_stream(stream), _c.byref(detail))
    if st not in (0, 5):
        raise MnnllmError(st, "read_status")
    return int(detail.value)
