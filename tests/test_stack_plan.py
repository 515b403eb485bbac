"""Host logic of the one-launch decoder stack: the plan is built without a GPU (n_sms given)."""
import struct

import numpy as np
import pytest

from paper_2506_10443_b200 import binding as B
from paper_2506_10443_b200 import inputs

HDR = struct.Struct("<IIiiiiiiiII")           # magic, version, count, M, group, MP, n_ctas, slots, max_quanta, smem, xs
PROB = struct.Struct("<4Q4QQQ" + "4i4i" + "i" * 10 + "4i4i" + "ii")


def fake_problems(model, layers=2):
    """Decoder-layer shapes with made-up (aligned) device addresses: the plan only stores them."""
    probs, addr, prev_down = [], 1 << 20, None
    for _ in range(layers):
        idx = {}
        for lin in inputs.stack(model):
            deps = {"q": [prev_down], "k": [prev_down], "v": [prev_down], "o": [idx.get("q"), idx.get("k"), idx.get("v")],
                    "gate": [idx.get("o")], "up": [idx.get("o")], "down": [idx.get("gate"), idx.get("up")]}[lin.name]
            idx[lin.name] = len(probs)
            if lin.name in ("q", "o", "gate", "down"):      # q, k, v read one input; so do gate and up
                x_addr = addr
            probs.append(dict(x=x_addr, packed=addr + (1 << 12), y=addr + (1 << 13), N=lin.N, K=lin.K,
                              deps=[d for d in deps if d is not None]))
            addr += 1 << 16
        prev_down = idx["down"]
    return probs


def parse(plan):
    raw = plan.tobytes()
    h = HDR.unpack_from(raw, 0)
    hdr = dict(zip("magic version count M group MP n_ctas slots max_quanta smem xs".split(), h))
    probs = []
    for p in range(hdr["count"]):
        f = PROB.unpack_from(raw, 64 + 192 * p)
        d = dict(packed=f[0:4], y=f[4:8], x=f[8], rbb=f[9], N=f[10:14], nb_end=f[14:18])
        d.update(zip("K NB NC NS gran rot weff y_dtypes n_deps stage_x".split(), f[18:28]))
        d["deps"], d["deps_nb"] = f[28:32], f[32:36]
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
    # q+k+v and gate+up share their input and their predecessors: 4 problems per layer in the plan
    assert hdr["count"] == 8 and hdr["n_ctas"] == n_sms and hdr["M"] == M
    assert hdr["slots"] >= 14 and hdr["smem"] <= 227 * 1024
    assert hdr["slots"] % 14 == 0   # every consumer warp owns the same number of slots
    groups = [[0, 1, 2], [3], [4, 5], [6], [7, 8, 9], [10], [11, 12], [13]]
    for members, d in zip(groups, out):
        want = [probs[i] for i in members]
        assert list(d["N"][:len(want)]) == [w["N"] for w in want] and d["K"] == want[0]["K"]
        assert list(d["packed"][:len(want)]) == [w["packed"] for w in want] and d["x"] == want[0]["x"]
        nb = np.cumsum([-(-w["N"] // 16) for w in want])
        assert list(d["nb_end"][:len(want)]) == list(nb) and d["NB"] == nb[-1]
        assert d["NC"] == -(-d["K"] // 512) and d["NS"] == d["K"] // 64
        assert d["gran"] in (1, d["NC"]) and 1 <= d["weff"] <= 14 and 0 <= d["rot"] < n_sms
        if d["NC"] <= 14:
            assert d["weff"] % d["NC"] == 0       # a warp keeps one k-chunk's activations
        want_deps = sorted({next(g for g, ms in enumerate(groups) if u in ms) for u in want[0]["deps"]})
        assert sorted(d["deps"][:d["n_deps"]]) == want_deps
        assert [out[i]["NB"] for i in d["deps"][:d["n_deps"]]] == list(d["deps_nb"][:d["n_deps"]])
        seen = np.zeros(d["NB"] * d["NC"], np.int32)
        for cv in range(n_sms):
            q0, q1 = cta_range(d["NB"], d["NC"], d["gran"], cv, n_sms)
            assert q1 - q0 <= hdr["max_quanta"]
            seen[q0:q1] += 1
        assert (seen == 1).all()


def test_small_problems_of_one_stage_start_on_different_sms():
    # k and v of a layer whose q has different predecessors are not fused: they must not pile up
    probs = fake_problems(inputs.QWEN2_1P5B, 1)[:3]
    probs[1] = dict(probs[1], x=probs[1]["x"] + 64)
    probs[2] = dict(probs[2], x=probs[2]["x"] + 128)
    hdr, out = parse(B.stack_plan_w4a16(probs, 1, 64, n_sms=148))
    assert hdr["count"] == 3
    used = []
    for d in out:
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
