"""The C-ABI library loads without a GPU and exports every symbol that include/mnnllm.h declares;
host-only entry points validate their arguments."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2506_10443_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "mnnllm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mnnllm_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    names = declared_symbols()
    assert len(names) >= 18
    for n in names:
        assert hasattr(B.lib, n), n
    assert sorted(B.EXPORTS) == [n for n in names if n != "mnnllm_w4a16_problem"]


def test_status_strings():
    B.lib.mnnllm_status_string.restype = ctypes.c_char_p
    seen = {B.lib.mnnllm_status_string(i) for i in range(7)}
    assert len(seen) == 7 and b"ok" in seen


def test_packed_size_rejects_bad_arguments():
    def trailer(n_row_blocks):   # 16-byte head + 16 bytes per padded row, 128-byte granules
        return -(-(16 + n_row_blocks * 16 * 16) // 128) * 128

    def up128(v):
        return -(-v // 128) * 128

    assert B.packed_size_w4(16, 64, 64) == up128(128 + 512 + 16 * 4) + trailer(1)
    assert B.packed_size_w4(17, 64, 64) == up128(128 + 2 * (512 + 64)) + trailer(2)
    assert B.packed_size_w4(16, 128, 128) == up128(128 + 1024 + 64) + trailer(1)
    for bad in [(0, 64, 64), (16, 0, 64), (16, 64, 32), (16, 96, 64), (16, 192, 128), (-1, 64, 64)]:
        assert B.packed_size_w4(*bad) == 0
    assert B.packed_size_w8(16, 32) == 128 + 512 + 64
    assert B.packed_size_w8(16, 48) == 0


def test_pack_argument_errors():
    W = np.zeros((16, 64), np.float32)
    out = B.aligned_empty(B.packed_size_w4(16, 64, 64))
    assert B.lib.mnnllm_pack_w4(None, 16, 64, 64, out.ctypes.data) == 1
    assert B.lib.mnnllm_pack_w4(W.ctypes.data, 16, 64, 64, None) == 1
    assert B.lib.mnnllm_pack_w4(W.ctypes.data, 16, 64, 48, out.ctypes.data) == 2
    junk = np.zeros(256, np.uint8)
    assert B.lib.mnnllm_unpack_w4(junk.ctypes.data, W.ctypes.data, W.ctypes.data, W.ctypes.data) == 1
    with pytest.raises(B.MnnllmError):
        B.packed_info(junk)


def test_gpu_entry_points_fail_loudly_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    # no CPU fallback: with valid-looking arguments the call reports an unsupported device
    st = B.lib.mnnllm_linear_w4a16(0x1000, 0x1000, 0x1000, 1, 16, 64, 64, None)
    assert st == 2
    assert B.lib.mnnllm_linear_w4a16(None, 0x1000, 0x1000, 1, 16, 64, 64, None) == 1
    assert B.lib.mnnllm_linear_w4a16(0x1008, 0x1000, 0x1000, 1, 16, 64, 64, None) == 3
    assert B.lib.mnnllm_linear_w4a16(0x1000, 0x1000, 0x1000, 1, 16, 64, 100, None) == 2
    assert not B.device_supported()
    need = B.workspace_min_w4a8(4, 16, 64, 64)
    assert need >= 4 * 64 + 4 * 4 + 4 * 4 * 8 and need % 256 == 0
    assert B.workspace_size_w4a8(4, 16, 64, 64) > need          # room for splitting tiles along K
    assert B.workspace_size_w4a8(4, 16, 64, 48) == 0 and B.workspace_min_w4a8(4, 16, 64, 48) == 0
    f = B.lib.mnnllm_linear_w4a8
    assert f(0x1000, 0x1000, 0x1000, 4, 16, 64, 64, B.F16, B.F16, 0x1000, need, None) == 2   # no device
    assert f(0x1000, 0x1000, 0x1000, 4, 16, 64, 64, B.F16, B.F16, 0x1000, need - 1, None) == 6
