"""GPU parity of the quantised-KV decode attention (mnnllm_kv_append, mnnllm_attention_decode) against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_10443_b200 import binding as B
from gpu_util import assert_close, dev

pytestmark = pytest.mark.gpu

D = 128


def kv(seed, Hk, S, outliers=False):
    rng = np.random.default_rng(seed)
    k = rng.standard_normal((Hk, S, D)).astype(np.float16)
    v = rng.standard_normal((Hk, S, D)).astype(np.float16)
    if outliers:
        k[:, :, 5] *= 8
        v[:, ::7, 9] = 1000.0      # beyond 448: saturates
        v[:, 3::11, 2] = 1e-3      # E4M3 subnormals
    return k, v


def cache_from_oracle(k, v):
    kc, ks, kz = oracle.quantize_keys(k.astype(np.float32))
    meta = ks.astype(np.uint32) | (kz.astype(np.uint32) << 16)
    return kc, ks, kz, meta, oracle.quantize_values(v.astype(np.float32))


def run_decode(q, kc, meta, vb, H, Hk, S, S_cap, out_dtype=B.F32):
    out = torch.full((H, D), float("nan"), dtype=torch.float32 if out_dtype == B.F32 else torch.float16, device="cuda")
    ws_bytes = B.attention_workspace_size(H, Hk, S)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    B.attention_workspace_init(ws, ws_bytes)
    B.attention_decode(q, kc, meta, vb, out, H, Hk, S, S_cap, ws, ws_bytes, out_dtype)
    torch.cuda.synchronize()
    assert B.read_status() == 0
    return out, ws


def test_append_is_bit_exact_with_the_oracle_quantisers():
    Hk, S_cap = 4, 40
    k, v = kv(1, Hk, S_cap, outliers=True)
    k[1, 7] = 0.25                      # a constant key: scale 1, codes 0
    kc_d = torch.zeros((Hk, S_cap, D), dtype=torch.uint8, device="cuda")
    meta_d = torch.zeros((Hk, S_cap), dtype=torch.int32, device="cuda")
    v_d = torch.zeros((Hk, S_cap, D), dtype=torch.uint8, device="cuda")
    for pos in range(S_cap):
        B.kv_append(kc_d, meta_d, v_d, Hk, S_cap, pos, dev(k[:, pos]), dev(v[:, pos]))
    torch.cuda.synchronize()
    kc, ks, kz, meta, vb = cache_from_oracle(k, v)
    assert (kc_d.cpu().numpy() == kc).all()
    assert (meta_d.cpu().numpy().view(np.uint32) == meta).all()
    assert (v_d.cpu().numpy() == vb).all()


@pytest.mark.parametrize("H,Hk,S", [
    (12, 2, 1000),     # Qwen2-1.5B heads, ragged last chunk
    (28, 4, 4096),     # Qwen2-7B heads, whole chunks, several splits per kv head
    (8, 8, 1),         # one token, one query head per kv head
    (16, 2, 257),      # eight query heads per kv head, one token past a chunk
    (3, 1, 70000),     # long sequence, more chunks than CTAs: several chunks per CTA
])
def test_decode_matches_oracle(H, Hk, S):
    k, v = kv(10 + H, Hk, S, outliers=True)
    kc, ks, kz, meta, vb = cache_from_oracle(k, v)
    q = np.random.default_rng(20 + H).standard_normal((H, D)).astype(np.float16)
    S_cap = S + 5
    pad = lambda a: np.concatenate([a, np.full((Hk, 5) + a.shape[2:], 255, a.dtype)], axis=1)   # rows past S: garbage
    out, _ = run_decode(dev(q), dev(pad(kc)), dev(pad(meta).view(np.int32)), dev(pad(vb)), H, Hk, S, S_cap)
    want = oracle.attention_decode(q.astype(np.float32), kc, ks, kz, vb)
    assert_close(out.cpu().numpy(), want, 2e-5)      # fp32 throughout; the path's bar is 2e-3


def test_decode_fp16_output_graph_replay_and_shared_workspace():
    H, Hk, S = 12, 2, 3000
    k, v = kv(31, Hk, S)
    kc, ks, kz, meta, vb = cache_from_oracle(k, v)
    q = dev(np.random.default_rng(32).standard_normal((H, D)).astype(np.float16))
    kc_d, meta_d, vb_d = dev(kc), dev(meta.view(np.int32)), dev(vb)
    out, ws = run_decode(q, kc_d, meta_d, vb_d, H, Hk, S, S, B.F16)
    want = oracle.attention_decode(q.cpu().numpy().astype(np.float32), kc, ks, kz, vb)
    assert_close(out.float().cpu().numpy(), want, 2.0 ** -11 + 2e-5)
    first = out.clone()
    g = torch.cuda.CUDAGraph()
    cap = torch.cuda.Stream()
    cap.wait_stream(torch.cuda.current_stream())
    with torch.cuda.graph(g, stream=cap):
        B.attention_decode(q, kc_d, meta_d, vb_d, out, H, Hk, S, S, ws, ws.numel(), B.F16, stream=cap)
    for _ in range(3):
        out.zero_()
        g.replay()
    torch.cuda.synchronize()
    assert B.read_status() == 0 and torch.equal(first, out)
    assert int(ws[:256].view(torch.int32).abs().sum()) == 0     # the counters are back at zero


def test_append_then_decode_end_to_end():
    # the cache built token by token on the GPU gives what the oracle gives on its own quantised cache
    H, Hk, S = 4, 2, 300
    k, v = kv(41, Hk, S)
    kc_d = torch.zeros((Hk, S, D), dtype=torch.uint8, device="cuda")
    meta_d = torch.zeros((Hk, S), dtype=torch.int32, device="cuda")
    v_d = torch.zeros((Hk, S, D), dtype=torch.uint8, device="cuda")
    for pos in range(S):
        B.kv_append(kc_d, meta_d, v_d, Hk, S, pos, dev(k[:, pos]), dev(v[:, pos]))
    q = np.random.default_rng(42).standard_normal((H, D)).astype(np.float16)
    out, _ = run_decode(dev(q), kc_d, meta_d, v_d, H, Hk, S, S)
    kc, ks, kz, meta, vb = cache_from_oracle(k, v)
    assert_close(out.cpu().numpy(), oracle.attention_decode(q.astype(np.float32), kc, ks, kz, vb), 2e-5)


def test_attention_argument_errors():
    kc = torch.zeros((2, 8, D), dtype=torch.uint8, device="cuda")
    meta = torch.zeros((2, 8), dtype=torch.int32, device="cuda")
    q = torch.zeros((4, D), dtype=torch.float16, device="cuda")
    out = torch.zeros((4, D), dtype=torch.float16, device="cuda")
    ws = torch.zeros(B.attention_workspace_size(4, 2, 8), dtype=torch.uint8, device="cuda")
    assert B.attention_workspace_size(5, 2, 8) == 0 and B.attention_workspace_size(18, 2, 8) == 0
    with pytest.raises(B.MnnllmError) as e:
        B.attention_decode(q, kc, meta, kc, out, 4, 2, 9, 8, ws, ws.numel())          # S beyond the cache
    assert e.value.status == 1
    with pytest.raises(B.MnnllmError) as e:
        B.attention_decode(q, kc, meta, kc, out, 4, 2, 8, 8, ws, ws.numel(), head_dim=64)
    assert e.value.status == 2
    with pytest.raises(B.MnnllmError) as e:
        B.attention_decode(q, kc, meta, kc, out, 4, 2, 8, 8, ws, 16)                  # workspace too small
    assert e.value.status == 6
    with pytest.raises(B.MnnllmError) as e:
        B.kv_append(kc, meta, kc, 2, 8, 8, q, q)                                      # position outside the cache
    assert e.value.status == 1
