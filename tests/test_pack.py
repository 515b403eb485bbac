"""Host packer against the oracle: codes, scale bits and zero bits must agree bit for bit, for the
shapes of the workload configs and for ragged ones; the layout must be what the header documents."""
import numpy as np
import pytest

import oracle
from paper_2506_10443_b200 import binding as B
from paper_2506_10443_b200 import inputs


@pytest.mark.parametrize("N,K,group", [
    (16, 64, 64), (1, 64, 64), (17, 128, 128), (40, 192, 64), (256, 1536, 64), (100, 8960, 64),
    (64, 3584, 64), (48, 18944, 64), (130, 3584, 128), (33, 640, 128),
])
def test_pack_unpack_matches_oracle(N, K, group):
    W = inputs.weights(100 + N + K, N, K)
    packed = B.pack_w4(W, group)
    assert packed.ctypes.data % 128 == 0 and len(packed) == B.packed_size_w4(N, K, group)
    assert B.packed_info(packed) == (N, K, group, 4)
    q, s, z = B.unpack_w4(packed)
    q0, s0, z0 = oracle.quantize_w4(W, group)
    assert (q == q0).all() and (s == s0).all() and (z == z0).all()


def test_special_values_match_oracle():
    rng = np.random.default_rng(1)
    W = rng.standard_normal((32, 256)).astype(np.float32)
    W[0, :64] = 0.25                      # constant group
    W[1, :64] = 0.0
    W[2, :64] *= 1e-9                     # scale underflows fp16
    W[3, :64] *= 1e6                      # scale overflows fp16 -> saturates
    W[4, :64] = W[4, :64] * 1e-3 + 100    # zero point far outside 0..15
    W[5, :64] = -np.abs(W[5, :64])        # all negative
    W[6, 5] = 1e-6                        # tiny values among ordinary ones
    packed = B.pack_w4(W, 64)
    q, s, z = B.unpack_w4(packed)
    q0, s0, z0 = oracle.quantize_w4(W, 64)
    assert (q == q0).all() and (s == s0).all() and (z == z0).all()


def test_documented_layout_nibbles_and_padding():
    N, K, group = 20, 576, 64           # 2 row blocks (12 padding rows), 9 slabs: chunks of 8 and 1
    W = inputs.weights(7, N, K)
    packed = B.pack_w4(W, group)
    q, s, z = oracle.quantize_w4(W, group)
    body = packed[128:]
    row_block = 9 * 512 + 16 * 9 * 4
    trailer_at = -(-(128 + 2 * row_block) // 128) * 128
    assert len(packed) == trailer_at + -(-(16 + 32 * 16) // 128) * 128
    # trailer: every scale of a row is an integer S times 2^row_exp, row_sum = sum_k q S (from the oracle's codes)
    assert packed[trailer_at:trailer_at + 4].view(np.uint32)[0] == 1
    info = packed[trailer_at + 16: trailer_at + 16 + 32 * 16].view(np.int32).reshape(32, 4)
    sv = s.view(np.float16).astype(np.float64)
    for n in range(32):
        if n >= N:
            assert (info[n, :3] == 0).all()
            continue
        S = sv[n] / 2.0 ** int(info[n, 3])
        assert (S == np.round(S)).all() and S.min() >= 1 and S.max() < 2 ** 16
        Sk = np.repeat(S.astype(np.int64), group)             # per k
        qk = q[n].astype(np.int64)
        lo = qk * (Sk & 4095)
        limbs = [lo & 255, lo >> 8, qk * (Sk >> 12)]
        assert (limbs[0] + 256 * limbs[1] + 4096 * limbs[2] == qk * Sk).all() and max(l.max() for l in limbs) <= 255
        assert [int(l.sum()) for l in limbs] == [int(v) for v in info[n, :3]]
    full_chunk = 8 * 512 + 16 * 8 * 4
    nib = [0, 4, 1, 5, 2, 6, 3, 7]
    for rb in range(2):
        for j, ns in ((0, 8), (1, 1)):
            chunk = body[rb * row_block + j * full_chunk:]
            for sl in range(ns):
                words = chunk[sl * 512:(sl + 1) * 512].view(np.uint32).reshape(32, 4)
                for lane in (0, 5, 31):
                    r, c = lane >> 2, lane & 3
                    for wd in range(4):
                        n = rb * 16 + r + 8 * (wd >> 1)
                        k0 = (j * 8 + sl) * 64 + 16 * c + 8 * (wd & 1)
                        for i in range(8):
                            got = (int(words[lane, wd]) >> (4 * i)) & 15
                            want = int(q[n, k0 + nib[i]]) if n < N else 0
                            assert got == want
            table = chunk[ns * 512: ns * 512 + 16 * ns * 4].view(np.uint16).reshape(16, ns, 2)
            for r in range(16):
                n = rb * 16 + r
                for g in range(ns):
                    if n < N:
                        assert table[r, g, 0] == s[n, j * 8 + g] and table[r, g, 1] == z[n, j * 8 + g]
                    else:
                        assert table[r, g, 0] == 0 and table[r, g, 1] == 0


@pytest.mark.parametrize("N,K", [(16, 32), (37, 96), (128, 3584), (50, 544)])
def test_pack_w8_matches_oracle(N, K):
    W = inputs.weights(200 + N, N, K)
    packed = B.pack_w8(W)
    assert B.packed_info(packed) == (N, K, K, 8)
    q, s, z = B.unpack_w8(packed)
    q0, s0, z0 = oracle.quantize_w8(W)
    assert (q == q0).all() and (s == s0).all() and (z == z0).all()
