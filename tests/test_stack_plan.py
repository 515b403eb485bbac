"""Host logic of the one-launch decoder stack: the plan is built without a GPU (n_sms given)."""
import struct

import numpy as np
import pytest

from paper_2506_10443_b200 import binding as B
from paper_2506_10443_b200 import inputs

HDR = struct.Struct("<IIiiiiiiiIiI")          # magic, version, count, M, group, MP, n_ctas, slots, max_quanta, smem, window, xs
PROB = struct.Struct("<QQQQ" + "i" * 10 + "4i4i" + "ii")


def fake_problems(model, layers=2):
    """Decoder-layer shapes with made-up (aligned) device addresses: the plan only stores them."""
    probs, addr, prev_down = [], 1 << 20, None
    for _ in range(layers):
        idx = {}
        for lin in inputs.stack(model):
            deps = {"q": [prev_down], "k": [prev_down], "v": [prev_down], "o": [idx.get("q"), idx.get("k"), idx.get("v")],
                    "gate": [idx.get("o")], "up": [idx.get("o")], "down": [idx.get("gate"), idx.get("up")]}[lin.name]
            idx[lin.name] = len(probs)
            probs.append(dict(x=addr, packed=addr + (1 << 12), y=addr + (1 << 13), N=lin.N, K=lin.K,
                              deps=[d for d in deps if d is not None]))
            addr += 1 << 16
        prev_down = idx["down"]
    return probs


def parse(plan):
    raw = plan.tobytes()
    h = HDR.unpack_from(raw, 0)
    hdr = dict(zip("magic version count M group MP n_ctas slots max_quanta smem window xs".split(), h))
    probs = []
    for p in range(hdr["count"]):
        f = PROB.unpack_from(raw, 64 + 112 * p)
        d = dict(zip("packed x y rbb N K NB NC NS gran rot weff y_dtype n_deps".split(), f[:14]))
        d["deps"], d["deps_nb"], d["stage_x"] = f[14:18], f[18:22], f[22]
        probs.append(d)
    return hdr, probs


def cta_range(NB, NC, gran, cv, n):
    """The dealing rule the kernel applies to a plan entry (runs of `gran` quanta, evenly)."""
    U = NB * NC // gran
    if U < n:
        return (cv * gran, cv * gran + gran) if cv < U else (0, 0)
    return (U * cv // n) * gran, (U * (cv + 1) // n) * gran


@pytest.mark.parametrize("model,M", [(inputs.QWEN2_1P5B, 1), (inputs.QWEN2_7B, 1), (inputs.QWEN2_1P5B, 8), (inputs.QWEN2_7B, 4)])
@pytest.mark.parametrize("n_sms", [148, 132, 64])
def test_plan_covers_every_quantum_once_and_fits_shared_memory(model, M, n_sms):
    probs = fake_problems(model)
    hdr, out = parse(B.stack_plan_w4a16(probs, M, 64, n_sms=n_sms))
    assert hdr["count"] == len(probs) and hdr["n_ctas"] == n_sms and hdr["M"] == M
    assert hdr["slots"] >= 2 and hdr["smem"] <= 227 * 1024 and 1 <= hdr["window"] < hdr["slots"]
    for want, d in zip(probs, out):
        assert (d["N"], d["K"]) == (want["N"], want["K"])
        assert d["NB"] == -(-d["N"] // 16) and d["NC"] == -(-d["K"] // 512) and d["NS"] == d["K"] // 64
        assert d["gran"] in (1, d["NC"]) and 1 <= d["weff"] <= 14 and 0 <= d["rot"] < n_sms
        if d["NC"] <= 14:
            assert d["weff"] % d["NC"] == 0       # a warp keeps one k-chunk's activations
        assert list(d["deps"][:d["n_deps"]]) == want["deps"]
        assert [out[i]["NB"] for i in want["deps"]] == list(d["deps_nb"][:d["n_deps"]])
        seen = np.zeros(d["NB"] * d["NC"], np.int32)
        for cv in range(n_sms):
            q0, q1 = cta_range(d["NB"], d["NC"], d["gran"], cv, n_sms)
            assert q1 - q0 <= hdr["max_quanta"]
            seen[q0:q1] += 1
        assert (seen == 1).all()


def test_small_problems_of_one_stage_start_on_different_sms():
    hdr, out = parse(B.stack_plan_w4a16(fake_problems(inputs.QWEN2_1P5B, 1), 1, 64, n_sms=148))
    q, k, v = out[0], out[1], out[2]
    used = []
    for d in (q, k, v):
        U = d["NB"] * d["NC"] // d["gran"]
        assert U < 148
        used.append({(cv + d["rot"]) % 148 for cv in range(U)})
    assert not (used[0] & used[1]) and not (used[1] & used[2]) and not (used[0] & used[2])


def test_plan_argument_errors():
    good = fake_problems(inputs.QWEN2_1P5B, 1)
    with pytest.raises(B.MnnllmError) as e:
        B.stack_plan_w4a16(good, 1, 32, n_sms=148)
    assert e.value.status == 2
    bad = [dict(good[0], deps=[0])]
    with pytest.raises(B.MnnllmError) as e:
        B.stack_plan_w4a16(bad, 1, 64, n_sms=148)
    assert e.value.status == 1
    bad = [dict(good[0], x=good[0]["x"] + 2)]
    with pytest.raises(B.MnnllmError) as e:
        B.stack_plan_w4a16(bad, 1, 64, n_sms=148)
    assert e.value.status == 3
