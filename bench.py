#!/usr/bin/env python
"""Benchmark of the weight-quantised linear stack on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One step = one pass of the whole linear stack of the workload over one batch of synthetic input
(decode: one token through all 28 layers x 7 linears).  Rank 0 prints ONE JSON line.  With N > 1
(launched by torchrun) every rank runs an independent replica on its own GPU: the path has no
exchange step, so there is no collective on the data path.

`--impl reference` times the CPU oracle (a deliberately plain program) on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0        # burst; about 1400 sustained
INT8_OVER_BF16 = 2.0                 # nominal dense tensor-rate ratio (4.5 POPS int8 : 2.25 PFLOPS bf16)

PROFILE_OF = {   # committed ncu summary of the dominant kernel of a workload (profiles/)
    "decode_qwen2_1p5b_w4a16_g64": "gemv_w4a16_decode_qwen2_1p5b.txt",
    "decode_qwen2_7b_w4a16_g64": "gemv_w4a16_decode_qwen2_7b.txt",
    "prefill_qwen2_1p5b_w4a8_g64_m1024": "gemm_w4a8_prefill_qwen2_1p5b_m1024.txt",
    "prefill_qwen2_1p5b_w4a8_g64_m64": "gemm_w4a8_prefill_qwen2_1p5b_m64.txt",
    "prefill_qwen2_7b_w4a8_g64_m512": "gemm_w4a8_prefill_qwen2_7b_m512.txt",
    "prefill_qwen2_1p5b_w8a8_m1024": "gemm_w8a8_prefill_qwen2_1p5b_m1024.txt",
}


def kernel_sources_sha1(names):
    """sha1 over the named files of csrc/: a profile summary records it, so that counters taken
    from another version of the kernel are recognised."""
    import hashlib

    h = hashlib.sha1()
    for n in sorted(names):
        with open(os.path.join(ROOT, "paper_2506_10443_b200", "csrc", n), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def traffic_from_profile(workload):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of the workload's dominant kernel, read
    from the committed ncu summary; None when there is none or the kernel's sources have changed
    since (the summary carries 'traffic_bytes_per_launch = N', 'kernel_sources = a.cu b.cuh ...' and
    'kernel_sources_sha1 = ...' lines)."""
    import re

    name = PROFILE_OF.get(workload)
    path = os.path.join(ROOT, "profiles", name) if name else None
    if not path or not os.path.exists(path):
        return None
    text = open(path).read()
    m = re.search(r"^traffic_bytes_per_launch\s*=\s*(\d+)", text, re.M)
    src = re.search(r"^kernel_sources\s*=\s*(.+)$", text, re.M)
    sha = re.search(r"^kernel_sources_sha1\s*=\s*([0-9a-f]{40})", text, re.M)
    if not (m and src and sha):
        return None
    try:
        if kernel_sources_sha1(src.group(1).split()) != sha.group(1):
            return None
    except OSError:
        return None
    return int(m.group(1))


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": FALLBACK_BF16_TFLOPS,
            "bf16_tflops_sustained": 1400.0}, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the benchmark runs."""

    def __init__(self, torch_device_index: int, period_s: float = 0.02):
        self.period = period_s
        self.samples = []  # (t, sm_mhz, reasons bitmask)
        self.ok = False
        self.sm_max = None
        self._stop = threading.Event()
        try:
            import pynvml
            import torch

            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(torch_device_index).uuid)
            handle = None
            for i in range(pynvml.nvmlDeviceGetCount()):
                h = pynvml.nvmlDeviceGetHandleByIndex(i)
                u = pynvml.nvmlDeviceGetUUID(h)
                u = u.decode() if isinstance(u, bytes) else u
                if uuid in u:
                    handle = h
                    break
            if handle is None:
                handle = pynvml.nvmlDeviceGetHandleByIndex(torch_device_index)
            self.nv, self.h = pynvml, handle
            self.sm_max = int(pynvml.nvmlDeviceGetMaxClockInfo(handle, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception as e:  # NVML missing: the line says so instead of inventing clocks
            self.err = repr(e)
        self.thread = threading.Thread(target=self._run, daemon=True)

    def _reasons(self):
        nv = self.nv
        for name in ("nvmlDeviceGetCurrentClocksEventReasons", "nvmlDeviceGetCurrentClocksThrottleReasons"):
            f = getattr(nv, name, None)
            if f is not None:
                try:
                    return int(f(self.h))
                except Exception:
                    pass
        return 0

    def _run(self):
        while not self._stop.is_set():
            try:
                mhz = int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
                self.samples.append((time.perf_counter(), mhz, self._reasons()))
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self.ok:
            self.thread.start()

    def stop(self):
        self._stop.set()
        if self.ok:
            self.thread.join(timeout=2)

    def summary(self, t0: float, t1: float):
        if not self.ok:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "note": "NVML unavailable"}
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        note = "sampled inside the timed region"
        if not inside:  # region shorter than the sampling period: take every sample under load
            inside = self.samples[1:] or self.samples
            note = "timed region shorter than the sampling period; samples cover warm-up + timed + e2e loops"
        bits = 0
        for s in inside:
            bits |= s[2]
        names = {
            0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
            0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
            0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting",
        }
        reasons = [n for b, n in names.items() if bits & b and n != "gpu_idle"]
        mhz = sorted(s[1] for s in inside)
        return {"sm_mhz": mhz[len(mhz) // 2] if mhz else None, "sm_max_mhz": self.sm_max, "reasons": reasons,
                "samples": len(inside), "note": note}


# --------------------------------------------------------------------------------------------------
# workloads
# --------------------------------------------------------------------------------------------------
def _wl(model, config, M, kind):
    return {"model": model, "config": config, "M": M, "kind": kind}


WORKLOADS = {
    # decode: one token through the stack, W4A16, HBM-bound; prefill: a prompt of M tokens, W4A8
    "decode_qwen2_1p5b_w4a16_g64": _wl("QWEN2_1P5B", 2, 1, "decode"),
    "decode_qwen2_7b_w4a16_g64": _wl("QWEN2_7B", 4, 1, "decode"),
    "prefill_qwen2_1p5b_w4a8_g64_m64": _wl("QWEN2_1P5B", 3, 64, "prefill"),
    "prefill_qwen2_1p5b_w4a8_g64_m256": _wl("QWEN2_1P5B", 3, 256, "prefill"),
    "prefill_qwen2_1p5b_w4a8_g64_m1024": _wl("QWEN2_1P5B", 3, 1024, "prefill"),
    "prefill_qwen2_7b_w4a8_g64_m512": _wl("QWEN2_7B", 4, 512, "prefill"),
}
DEFAULT_WORKLOAD = "decode_qwen2_1p5b_w4a16_g64"
GROUP = 64


def metric_of(kind):
    """(metric, unit, dtype): decode is graded on bytes moved, prefill on integer operations."""
    if kind == "decode":
        return "decode W4 GEMV GB/s", "GB/s", "f32"
    return "prefill W4A8 TOPS", "TOPS", "int8"


def units_of_linear(kind, N, K, M):
    """Algorithmic work of one linear in the metric's unit x 1e9 (bytes) or x 1e12 (int8 ops)."""
    from paper_2506_10443_b200 import inputs   # byte counts only: the oracle arm must not load the CUDA library

    return inputs.linear_bytes(N, K, GROUP, M) if kind == "decode" else 2 * M * N * K


def scale_of(kind):
    return 1e9 if kind == "decode" else 1e12


def oracle_linear(kind, x, q, s, z):
    import oracle

    if kind == "decode":
        return oracle.linear_wa16(x, q, s, z, GROUP)
    return oracle.linear_w4a8(x, q, s, z, GROUP)


def oracle_prepare(wl, model, layer, frac):
    """Oracle inputs of one layer (rows [0, frac*N) of every linear): quantised offline, untimed."""
    import oracle
    from paper_2506_10443_b200 import inputs

    out = []
    for lin in inputs.stack(model):
        rows = lin.N if frac >= 1.0 else max(1, int(np.ceil(frac * lin.N)))
        W = inputs.weights(inputs.seed_for(wl["config"], layer, lin.matrix_id, 0), lin.N, lin.K)[:rows]
        q, s, z = oracle.quantize_w4(W, GROUP)
        x = inputs.activations(inputs.seed_for(wl["config"], layer, lin.matrix_id, 1), wl["M"], lin.K,
                               outliers=wl["kind"] == "prefill").astype(np.float32)
        out.append((x, q, s, z, units_of_linear(wl["kind"], rows, lin.K, wl["M"])))
    return out


def oracle_sample(wl, model, seconds):
    """A sample of the workload sized so that one oracle pass over it takes about `seconds`:
    whole layers if they fit, else the first rows of every linear of layer 0."""
    import oracle
    from paper_2506_10443_b200 import inputs

    layer_units = sum(units_of_linear(wl["kind"], t.N, t.K, wl["M"]) for t in inputs.stack(model))
    cal = oracle_prepare(wl, model, 0, 0.02 if wl["kind"] == "decode" else 0.002)
    t = time.perf_counter()
    for x, q, s, z, _ in cal:
        oracle_linear(wl["kind"], x, q, s, z)
    rate = sum(c[4] for c in cal) / max(time.perf_counter() - t, 1e-6)
    frac = rate * seconds / layer_units
    if frac >= 1.0:
        n_layers = min(model["layers"], int(frac))
        sample = [p for l in range(n_layers) for p in oracle_prepare(wl, model, l, 1.0)]
        what = "%d of %d layers (7 linears each), %d token(s)" % (n_layers, model["layers"], wl["M"])
    else:
        sample = oracle_prepare(wl, model, 0, frac)
        what = "first %.2f %% of the rows of each of the 7 linears of layer 0, %d token(s)" % (100 * frac, wl["M"])
    return sample, what, oracle.num_threads()


def run_reference(args):
    """The reference arm: the CPU oracle as it stands, on the host cores, same metric and config.
    Each step is a bounded sample of the workload sized from a calibration pass so that the whole
    run (warm-up + steps) stays within about two minutes of oracle time."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from paper_2506_10443_b200 import inputs

    wl = WORKLOADS[args.workload]
    model = getattr(inputs, wl["model"])
    metric, unit, _ = metric_of(wl["kind"])
    budget = min(2.0, 120.0 / max(args.steps + args.warmup, 1))
    sample, what, threads = oracle_sample(wl, model, budget)
    step_units = sum(p[4] for p in sample)

    def step():
        for x, q, s, z, _ in sample:
            oracle_linear(wl["kind"], x, q, s, z)

    for _ in range(args.warmup):
        step()
    t = time.perf_counter()
    for _ in range(args.steps):
        step()
    total_s = time.perf_counter() - t
    value = step_units * args.steps / total_s / scale_of(wl["kind"])
    what += ", per step"
    line = {
        "impl": "reference", "metric": metric, "value": value, "unit": unit, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_s / max(args.steps, 1),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "sample": what, "algorithmic_units_per_step": step_units},
        "cpu_baseline": {"value": value, "unit": unit, "cores": threads, "kind": "oracle", "sample": what},
        "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def _time_steps(step, steps, warmup):
    """Milliseconds per step of `step()` on the current stream (CUDA events, after warm-up)."""
    import torch

    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def _graph_of(run):
    """Captures `run(stream)` into a CUDA graph (after one eager call that resolves per-device state)."""
    import torch

    run()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    cap = torch.cuda.Stream()
    cap.wait_stream(torch.cuda.current_stream())
    with torch.cuda.graph(g, stream=cap):
        run(cap)
    torch.cuda.synchronize()
    return g


def _hbm_entry(kernel, nbytes, ms, hbm, **extra):
    gbs = nbytes / (ms * 1e-3) / 1e9
    e = {"metric": "decode W4 GEMV GB/s", "value": gbs, "unit": "GB/s", "ms_per_step": ms,
         "roofline": {"bound": "hbm", "kernel": kernel, "achieved": gbs, "peak": hbm, "unit": "GB/s", "frac": gbs / hbm}}
    e.update(extra)
    return e


def _tensor_entry(ops, ms, M, int8_peak, ceiling, kernel="gemm_w4a8_kernel", **extra):
    tops = ops / (ms * 1e-3) / 1e12
    roof = {"bound": "tensor", "kernel": kernel, "achieved": tops, "peak": int8_peak, "unit": "TOP/s",
            "frac": tops / int8_peak, "frac_of_nominal_4500": tops / 4500.0,
            "frac_of_measured_int8_mma_ceiling": (tops / ceiling) if ceiling else None}
    e = {"metric": "prefill W4A8 TOPS", "value": tops, "unit": "TOPS", "ms_per_step": ms,
         "tokens_per_s": M / (ms * 1e-3), "roofline": roof}
    e.update(extra)
    return e


def int8_mma_ceiling(device_index):
    """tcgen05.mma kind::i8 issued back to back on resident shared-memory tiles for >= 100 ms: the
    ceiling of the instruction at the clock the GPU holds meanwhile (see mnnllm_bench_mma_i8)."""
    import torch

    from paper_2506_10443_b200 import binding as B

    sms = torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count
    sampler = ClockSampler(device_index, period_s=0.005)
    sampler.start()
    cycles = torch.zeros(sms, dtype=torch.int64, device="cuda")
    B.bench_mma_i8(40000, cycles)   # warm-up
    torch.cuda.synchronize()
    mmas = 3_200_000                # x 64 cycles at full rate: ~0.1-0.15 s
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    e0.record()
    B.bench_mma_i8(mmas, cycles)
    e1.record()
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    assert B.read_status() == 0
    ms = e0.elapsed_time(e1)
    ops = 2.0 * 128 * 128 * 32 * mmas * sms
    cyc = float(cycles.max().item())
    sampler.stop()
    clk = sampler.summary(t0, t1)
    return {"metric": "tcgen05.mma kind::i8 issue ceiling", "value": ops / (ms * 1e-3) / 1e12, "unit": "TOP/s",
            "ms": ms, "mmas_per_sm": mmas, "shape": "128x128x32, operands resident in shared memory",
            "mac_per_clk_per_sm": 128.0 * 128 * 32 * mmas / cyc, "sm_mhz_from_cycles": cyc / (ms * 1e-3) / 1e6,
            "clocks": clk}


def _sec_decode_one_launch(ctx):
    """The same decode step through the one-launch entry point (mnnllm_linear_w4a16_stack)."""
    stack = ctx["stack"]()
    g = _graph_of(stack.run_w4a16_stack)
    ms = _time_steps(g.replay, 300, 20)
    return {"decode_one_launch_qwen2_1p5b": _hbm_entry(
        "stack_w4a16_kernel", stack.algorithmic_bytes_w4a16, ms, ctx["hbm"], launches_per_step=1,
        note="whole stack as one persistent cooperative launch with device-side dependency counters")}


def _sec_single_gemv(ctx):
    """The single-GEMV workload: x [1, 1536], W [1536, 1536]; L2 flushed before every launch."""
    import torch

    from paper_2506_10443_b200 import binding as B
    from paper_2506_10443_b200 import inputs

    stack = ctx["stack"]()
    lin = stack.linears[0]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    xq, pq, yq = stack.x_view(0, "q"), stack.layers[0].packed["q"], stack.y_view(0, "q")
    times = []
    for i in range(60):
        flush.fill_(i & 0xFF)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        B.linear_w4a16(xq, pq, yq, 1, lin.N, lin.K, GROUP)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    ms = float(np.median(times[10:]))
    return {"single_gemv_1536x1536_m1": _hbm_entry(
        "gemv_w4a16_kernel", inputs.linear_bytes(lin.N, lin.K, GROUP, 1), ms, ctx["hbm"],
        note="latency-bound: 1.3 MB is 0.2 us of HBM time; one launch timed alone with events, L2 flushed "
             "(256 MB written) before each; median of 50")}


def _sec_prefill_1p5b(ctx):
    """W4A8 prefill of 64 / 256 / 1024-token prompts over the stack's packed weights."""
    import torch

    from paper_2506_10443_b200 import binding as B
    from paper_2506_10443_b200.workloads import LinearStack

    stack, out = ctx["stack"](), {}
    for M, reps in ((64, 50), (256, 30), (1024, 20)):
        pre = LinearStack(ctx["model"], 3, M, GROUP, outliers=True, weights_from=stack, distinct=4)
        g = _graph_of(pre.run_w4a8)
        assert B.read_status() == 0
        ms = _time_steps(g.replay, reps, 3)
        e = _tensor_entry(pre.ops, ms, M, ctx["int8_peak"], ctx["ceiling"],
                          note="activations of 4 distinct layers, reused by the others")
        if M == 64:   # 4 M = 256 int8 operations per weight byte: below the ridge, graded on bytes
            nbytes = pre.weight_bytes + sum(2 * M * (t.K + t.N) for t in pre.linears) * pre.n_layers
            gbs = nbytes / (ms * 1e-3) / 1e9
            e["roofline_hbm"] = {"bound": "hbm", "achieved": gbs, "peak": ctx["hbm"], "unit": "GB/s", "frac": gbs / ctx["hbm"]}
        e["traffic"] = traffic_from_profile("prefill_qwen2_1p5b_w4a8_g64_m%d" % M)
        out["prefill_w4a8_m%d" % M] = e
        del g, pre
    torch.cuda.empty_cache()
    return out


def _sec_qwen2_7b(ctx):
    """Qwen2-7B: decode (launch per group of linears, and one launch) and a 512-token prefill.  Four
    layers of distinct weights (524 MB, four times L2), reused in turn by the 28 layers: every pass
    streams its weights from DRAM."""
    import torch

    from paper_2506_10443_b200 import binding as B
    from paper_2506_10443_b200 import inputs
    from paper_2506_10443_b200.workloads import LinearStack

    out, hbm = {}, ctx["hbm"]
    s7 = LinearStack(inputs.QWEN2_7B, 4, 1, GROUP, distinct=4)
    g = _graph_of(s7.run_w4a16)
    ms = _time_steps(g.replay, 100, 10)
    out["decode_qwen2_7b"] = _hbm_entry(
        "gemv_w4a16_kernel", s7.algorithmic_bytes_w4a16, ms, hbm, launches_per_step=s7.launches_per_step_w4a16,
        tokens_per_s=1.0 / (ms * 1e-3), traffic=traffic_from_profile("decode_qwen2_7b_w4a16_g64"),
        note="28 layers over 4 layers of distinct weights and inputs")
    del g
    g = _graph_of(s7.run_w4a16_stack)
    ms = _time_steps(g.replay, 100, 10)
    out["decode_one_launch_qwen2_7b"] = _hbm_entry("stack_w4a16_kernel", s7.algorithmic_bytes_w4a16, ms, hbm,
                                                   launches_per_step=1)
    del g
    p7 = LinearStack(inputs.QWEN2_7B, 4, 512, GROUP, outliers=True, weights_from=s7, distinct=4)
    g = _graph_of(p7.run_w4a8)
    ms = _time_steps(g.replay, 10, 3)
    out["prefill_qwen2_7b_w4a8_m512"] = _tensor_entry(p7.ops, ms, 512, ctx["int8_peak"], ctx["ceiling"],
                                                      traffic=traffic_from_profile("prefill_qwen2_7b_w4a8_g64_m512"),
                                                      note="28 layers over 4 layers of distinct weights and inputs")
    assert B.read_status() == 0
    del g, p7, s7
    torch.cuda.empty_cache()
    return out


def _sec_lm_head(ctx):
    """LM head 151936 x 3584: int4 group 128 (1 and 4 tokens) and int8 per channel, fp32 logits."""
    import torch

    from paper_2506_10443_b200 import binding as B
    from paper_2506_10443_b200 import inputs

    out, hbm = {}, ctx["hbm"]
    N, K, grp = inputs.LM_HEAD["N"], inputs.LM_HEAD["K"], inputs.LM_HEAD["group"]
    W = inputs.weights(inputs.seed_for(5, 0, 0, 0), N, K)
    x = torch.from_numpy(inputs.activations(inputs.seed_for(5, 0, 0, 1), 4, K)).cuda()
    y = torch.empty((4, N), dtype=torch.float32, device="cuda")
    p4 = torch.from_numpy(B.pack_w4(W, grp)).cuda()
    for Mh in (1, 4):
        ms = _time_steps(lambda: B.linear_w4a16_ex(x, p4, y, Mh, N, K, grp, B.F16, B.F32), 50, 5)
        out["lm_head_w4a16_g128_m%d" % Mh] = _hbm_entry(
            "gemv_w4a16_kernel", inputs.w4_bytes(N, K, grp) + 2 * Mh * K + 4 * Mh * N, ms, hbm)
    del p4
    p8 = torch.from_numpy(B.pack_w8(W)).cuda()
    del W
    ms = _time_steps(lambda: B.linear_w8a16(x, p8, y, 1, N, K, B.F32), 50, 5)
    e = _hbm_entry("gemv_w8a16_kernel", N * K + 4 * N + 2 * K + 4 * N, ms, hbm)
    e["metric"] = "decode W8 GEMV GB/s"
    out["lm_head_w8a16_m1"] = e
    assert B.read_status() == 0
    return out


def _sec_prefill_w8a8(ctx):
    """Per-channel W8A8 prefill (no per-group rescale) on Qwen2-1.5B shapes at 1024 tokens: a layer's
    linears as four calls (q+k+v and gate+up stacked along N) over four layers of distinct int8 weights
    (188 MB, more than L2), 28 layers per step like the W4A8 rows; and the gate+up shape alone
    (17920 x 1536), where 560 tiles keep every SM busy."""
    import torch

    from paper_2506_10443_b200 import binding as B
    from paper_2506_10443_b200 import inputs

    M, out = 1024, {}
    lins = inputs.decoder_layer(ctx["model"]["hidden"], ctx["model"]["kv_dim"], ctx["model"]["inter"])
    # q, k, v and gate, up read the same activations: their weight matrices are stacked along N before
    # packing (one call each, four calls per layer)
    fused = [lins[0:3], lins[3:4], lins[4:6], lins[6:7]]
    ws_bytes = max(B.workspace_size_w8a8(M, t.K) for t in lins)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    layers = []
    for layer in range(4):
        calls = []
        for grp in fused:
            W = np.concatenate([inputs.weights(inputs.seed_for(6, layer, t.matrix_id, 0), t.N, t.K) for t in grp])
            x = inputs.activations(inputs.seed_for(6, layer, grp[0].matrix_id, 1), M, grp[0].K, outliers=True)
            calls.append((torch.from_numpy(x).cuda(), torch.from_numpy(B.pack_w8(W)).cuda(),
                          torch.empty((M, W.shape[0]), dtype=torch.float16, device="cuda"), W.shape[0], grp[0].K))
        layers.append(calls)

    def run(stream=None):
        for i in range(ctx["model"]["layers"]):
            for x, pk, y, N, K in layers[i % 4]:
                B.linear_w8a8(x, pk, y, M, N, K, ws, ws_bytes, B.F16, B.F16, stream)

    g = _graph_of(run)
    assert B.read_status() == 0
    ms = _time_steps(g.replay, 10, 3)
    ops = 2.0 * M * sum(t.N * t.K for t in lins) * ctx["model"]["layers"]
    e = _tensor_entry(ops, ms, M, ctx["int8_peak"], ctx["ceiling"], kernel="gemm_w8a8_kernel",
                      note="four calls per layer (q+k+v and gate+up stacked along N; quantiser + GEMM each), 4 layers of distinct weights and inputs",
                      traffic=traffic_from_profile("prefill_qwen2_1p5b_w8a8_m1024"))
    e["metric"] = "prefill W8A8 TOPS"
    out["prefill_w8a8_m1024"] = e
    del g
    # gate and up stacked alone: one [17920, 1536] matrix
    t = lins[4]
    N2 = 2 * t.N
    x, pk, y = layers[0][2][:3]
    ms = _time_steps(lambda: B.linear_w8a8(x, pk, y, M, N2, t.K, ws, ws_bytes), 50, 5)
    e = _tensor_entry(2.0 * M * N2 * t.K, ms, M, ctx["int8_peak"], ctx["ceiling"], kernel="gemm_w8a8_kernel",
                      note="one call (quantiser + GEMM), M=1024 N=17920 K=1536, weights 27.5 MB (L2-resident)")
    e["metric"] = "prefill W8A8 TOPS"
    out["prefill_w8a8_gate_up_m1024"] = e
    assert B.read_status() == 0
    del layers, pk, x, y, ws
    torch.cuda.empty_cache()
    return out


def _sec_decode_w8a16(ctx):
    """W8A16 decode (per-channel int8 weights, Section 4.2's GPU pairing) over the Qwen2-1.5B stack: one
    token, seven launches per layer, 28 layers of distinct weights (1.3 GB: every pass streams from DRAM)."""
    import torch

    from paper_2506_10443_b200 import binding as B
    from paper_2506_10443_b200 import inputs

    lins = inputs.decoder_layer(ctx["model"]["hidden"], ctx["model"]["kv_dim"], ctx["model"]["inter"])
    n_layers = ctx["model"]["layers"]
    calls, nbytes = [], 0
    for layer in range(n_layers):
        for t in lins:
            W = inputs.weights(inputs.seed_for(7, layer % 4, t.matrix_id, 0) + 100000 * (layer // 4), t.N, t.K)
            x = inputs.activations(inputs.seed_for(7, layer, t.matrix_id, 1), 1, t.K)
            calls.append((torch.from_numpy(x).cuda(), torch.from_numpy(B.pack_w8(W)).cuda(),
                          torch.empty((1, t.N), dtype=torch.float16, device="cuda"), t.N, t.K))
            nbytes += t.N * t.K + 4 * t.N + 2 * t.K + 2 * t.N   # int8 codes, fp16 scale and zero, x, y

    def run(stream=None):
        for x, pk, y, N, K in calls:
            B.linear_w8a16(x, pk, y, 1, N, K, B.F16, stream)

    g = _graph_of(run)
    assert B.read_status() == 0
    ms = _time_steps(g.replay, 100, 10)
    e = _hbm_entry("gemv_w8a16_kernel", nbytes, ms, ctx["hbm"], launches_per_step=len(calls),
                   tokens_per_s=1.0 / (ms * 1e-3))
    e["metric"] = "decode W8 GEMV GB/s"
    del g, calls
    torch.cuda.empty_cache()
    return {"decode_w8a16_qwen2_1p5b": e}


def _sec_decode_lora(ctx):
    """W4A16 decode with a rank-8 LoRA bypass on every linear (Section 5.5), Qwen2-1.5B stack, one token:
    one launch per linear (the GEMV's CTAs compute LoRA_B x between them and add LoRA_A (LoRA_B x) where
    they store).  Timed
    beside the same seven launches per layer without the bypass (the batched q+k+v / gate+up form of
    the headline has no LoRA entry)."""
    import torch

    from paper_2506_10443_b200 import binding as B
    from paper_2506_10443_b200 import inputs

    stack, r = ctx["stack"](), 8
    rng = np.random.default_rng(8)
    ws_bytes = B.workspace_size_lora(1, r)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")   # one workspace: the calls are on one stream
    B.lora_workspace_init(ws, ws_bytes)
    calls, extra = [], 0
    for li in range(stack.n_layers):
        for t in stack.linears:
            A = torch.from_numpy((rng.standard_normal((t.N, r)) * 0.05).astype(np.float16)).cuda()
            Bm = torch.from_numpy((rng.standard_normal((r, t.K)) * 0.05).astype(np.float16)).cuda()
            calls.append((stack.x_view(li, t.name), stack.layers[li].packed[t.name], A, Bm, stack.y_view(li, t.name), t.N, t.K, ws))
            extra += 2 * r * (t.N + t.K)

    def run_lora(stream=None):
        for x, pk, A, Bm, y, N, K, ws in calls:
            B.linear_w4a16_lora(x, pk, A, Bm, y, 1, N, K, GROUP, r, ws, ws_bytes, B.F16, B.F16, stream)

    def run_plain(stream=None):
        for x, pk, A, Bm, y, N, K, ws in calls:
            B.linear_w4a16_ex(x, pk, y, 1, N, K, GROUP, B.F16, B.F16, stream)

    g = _graph_of(run_lora)
    ms = _time_steps(g.replay, 100, 10)
    del g
    g = _graph_of(run_plain)
    ms0 = _time_steps(g.replay, 100, 10)
    del g
    assert B.read_status() == 0
    e = _hbm_entry("gemv_w4a16_kernel", stack.algorithmic_bytes_w4a16 + extra, ms, ctx["hbm"],
                   launches_per_step=len(calls), tokens_per_s=1.0 / (ms * 1e-3), rank=r,
                   ms_per_step_without_bypass=ms0, launches_without_bypass=len(calls),
                   lora_bytes_fraction=extra / stack.algorithmic_bytes_w4a16)
    e["metric"] = "decode W4 GEMV + LoRA GB/s"
    return {"decode_lora_r8_qwen2_1p5b": e}


def _sec_attention_decode(ctx):
    """Decode attention over a quantised KV cache (int8 keys, E4M3 values; Section 4.2) with Qwen2-1.5B
    heads (12 query, 2 kv, head_dim 128) and Qwen2-7B heads (28 / 4): 28 layers per step, each with its own
    cache (every pass streams from DRAM), 4096 and 32768 tokens of context.  Bytes = codes + values +
    4 bytes of scale/zero per key."""
    import torch

    from paper_2506_10443_b200 import binding as B

    out = {}
    for name, H, Hk, S in (("qwen2_1p5b_s4096", 12, 2, 4096), ("qwen2_1p5b_s32768", 12, 2, 32768),
                           ("qwen2_7b_s32768", 28, 4, 32768)):
        n_layers = 28
        gen = torch.Generator(device="cuda").manual_seed(9)
        kc = torch.randint(0, 256, (n_layers, Hk, S, 128), dtype=torch.uint8, device="cuda", generator=gen)
        # values: random E4M3 bytes below the NaN pattern; keys: scale 2^-6 (fp16 0x2400), zero 128 (0x5800)
        vb = torch.randint(0, 0x78, (n_layers, Hk, S, 128), dtype=torch.uint8, device="cuda", generator=gen)
        meta = torch.full((n_layers, Hk, S), 0x58002400, dtype=torch.int32, device="cuda")
        q = torch.randn((n_layers, H, 128), device="cuda", generator=gen).half()
        o = torch.empty((n_layers, H, 128), dtype=torch.float16, device="cuda")
        ws_bytes = B.attention_workspace_size(H, Hk, S)
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
        B.attention_workspace_init(ws, ws_bytes)

        def run(stream=None):
            for l in range(n_layers):
                B.attention_decode(q[l], kc[l], meta[l], vb[l], o[l], H, Hk, S, S, ws, ws_bytes, B.F16, stream=stream)

        g = _graph_of(run)
        assert B.read_status() == 0
        ms = _time_steps(g.replay, 50, 5)
        nbytes = n_layers * (Hk * S * (128 + 128 + 4) + 2 * 2 * H * 128)
        e = _hbm_entry("attn_decode_kernel", nbytes, ms, ctx["hbm"], launches_per_step=n_layers, context_tokens=S,
                       heads="%d query / %d kv" % (H, Hk))
        e["metric"] = "decode attention (int8 K, fp8 V) GB/s"
        out["attention_decode_" + name] = e
        del g, kc, vb, meta
        torch.cuda.empty_cache()
    return out


SECONDARY = {   # name -> function; also runnable alone: python bench.py --secondary-only NAME
    "decode_one_launch": _sec_decode_one_launch,
    "single_gemv": _sec_single_gemv,
    "prefill_1p5b": _sec_prefill_1p5b,
    "prefill_w8a8": _sec_prefill_w8a8,
    "decode_w8a16": _sec_decode_w8a16,
    "decode_lora": _sec_decode_lora,
    "attention_decode": _sec_attention_decode,
    "qwen2_7b": _sec_qwen2_7b,
    "lm_head": _sec_lm_head,
}


def secondary_measurements(stack_fn, model, peaks, device_index, only=None):
    """The other rows of the hot path on the same GPU, reported beside the headline, each with its
    own roofline: the measured int8 tensor-core ceiling, the one-launch form of the same decode step,
    the single-GEMV workload (cold L2), the W4A8 prefill of 64 / 256 / 1024-token prompts over the same
    packed weights, the Qwen2-7B decode and prefill stacks, the LM-head GEMVs."""
    out = {}
    ceil = None
    if only is None or only.startswith("prefill") or only == "qwen2_7b" or only == "int8_mma_ceiling":
        out["int8_mma_ceiling"] = ceil = int8_mma_ceiling(device_index)
    ctx = {"stack": stack_fn, "model": model, "hbm": float(peaks["hbm_gbs"]),
           "int8_peak": float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])) * INT8_OVER_BF16,
           "ceiling": ceil["value"] if ceil else None}
    for name, fn in SECONDARY.items():
        if only is None or only == name:
            out.update(fn(ctx))
    return out


def run_ours(args):
    import torch

    from paper_2506_10443_b200 import binding as B   # raises if the CUDA library is missing
    from paper_2506_10443_b200 import inputs
    from paper_2506_10443_b200.workloads import LinearStack

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a GPU: there is no CPU path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod

        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if not B.device_supported():
        raise SystemExit("the kernels are built for compute capability 10.x only")

    wl = WORKLOADS[args.workload]
    kind, M = wl["kind"], wl["M"]
    model = getattr(inputs, wl["model"])
    metric, unit, dtype = metric_of(kind)
    if args.secondary_only:   # one group of the secondary measurements alone (used for profiling)
        peaks, _ = measured_peaks()
        made = {}

        def lazy_stack():
            if "s" not in made:
                made["s"] = LinearStack(inputs.QWEN2_1P5B, 2, 1, GROUP, distinct=8)   # 210 MB of weights: above L2
            return made["s"]

        print(json.dumps({"secondary": secondary_measurements(lazy_stack, inputs.QWEN2_1P5B, peaks, local_rank,
                                                              only=args.secondary_only)}), flush=True)
        return
    # every rank: an independent replica of the workload.  The 7B stack draws four layers of distinct
    # weights (524 MB, four times L2) and reuses them in turn: the host time to draw 6.5 G random
    # numbers is not part of what is measured, and every pass still streams its weights from DRAM.
    distinct = 4 if wl["model"] == "QWEN2_7B" else None
    stack = LinearStack(model, wl["config"], M, GROUP, outliers=kind == "prefill", distinct=distinct)
    run = stack.run_w4a16 if kind == "decode" else stack.run_w4a8
    launches = stack.launches_per_step_w4a16 if kind == "decode" else stack.launches_per_step_w4a8
    step_units = stack.algorithmic_bytes_w4a16 if kind == "decode" else stack.ops
    stream = torch.cuda.current_stream()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # one untimed pass resolves per-device state (function attributes, symbol addresses), then capture
    run()
    assert B.read_status() == 0
    graph = None
    if not args.no_graph:
        graph = torch.cuda.CUDAGraph()
        cap = torch.cuda.Stream()
        cap.wait_stream(stream)
        with torch.cuda.graph(graph, stream=cap):
            run(cap)
        torch.cuda.synchronize()

    def step():
        if graph is not None:
            graph.replay()
        else:
            run()

    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(args.warmup):
        step()
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    barrier()
    t1 = time.perf_counter()
    ms = ev0.elapsed_time(ev1)
    assert B.read_status() == 0

    # end to end: the step's activations come from pinned host memory, its outputs go back to it
    e2e_steps = max(1, min(args.steps, 500))
    for _ in range(3):
        stack.xin.copy_(stack.xin_host, non_blocking=True)
        step()
        stack.yout_host.copy_(stack.yout, non_blocking=True)
        torch.cuda.synchronize()
    barrier()
    ee0, ee1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ee0.record()
    for _ in range(e2e_steps):
        stack.xin.copy_(stack.xin_host, non_blocking=True)
        step()
        stack.yout_host.copy_(stack.yout, non_blocking=True)
        stream.synchronize()   # the host reads the result of every step
    ee1.record()
    barrier()
    e2e_ms = ee0.elapsed_time(ee1)
    sampler.stop()

    from paper_2506_10443_b200.replicas import max_over_ranks

    ms, e2e_ms = max_over_ranks([ms, e2e_ms], "cuda")   # a step takes as long as its slowest replica

    if rank == 0:
        peaks, peaks_kind = measured_peaks()
        ms_per_step = ms / args.steps
        one = step_units / (ms_per_step * 1e-3) / scale_of(kind)          # one replica
        value = one * world
        e2e_value = step_units * world / (e2e_ms / e2e_steps * 1e-3) / scale_of(kind)
        if kind == "decode":
            roof = {"bound": "hbm", "kernel": "gemv_w4a16_kernel", "achieved": one, "peak": float(peaks["hbm_gbs"]),
                    "unit": "GB/s", "peak_source": "HBM copy rate, of " + peaks_kind}
            l2 = "weights of one step (%.0f MB) exceed L2 (126 MB); no flush" % (stack.weight_bytes / 1e6)
        else:
            peak = float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])) * INT8_OVER_BF16
            roof = {"bound": "tensor", "kernel": "gemm_w4a8_kernel", "achieved": one, "peak": peak, "unit": "TOP/s",
                    "peak_source": "sustained cuBLAS bf16 rate x 2 (nominal int8:bf16 ratio), of " + peaks_kind,
                    "frac_of_nominal_4500": one / 4500.0,
                    "note": "the timed region also holds the activation-quantiser launches (HBM-bound, small)"}
            l2 = "weights + activations of one step (%.0f MB) exceed L2 (126 MB); no flush" % (
                (stack.weight_bytes + 2 * stack.xin.numel() + 2 * stack.yout.numel()) / 1e6)
        roof.update({"frac": roof["achieved"] / roof["peak"], "launches_per_step": launches,
                     "avg_launch_us": 1e3 * ms_per_step / launches,
                     "algorithmic_units_per_launch": step_units / launches,
                     "traffic": traffic_from_profile(args.workload)})
        line = {
            "metric": metric, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": dtype, "data": "synthetic",
            "config": {
                "workload": args.workload, "tokens_per_step": M, "group": GROUP, "layers": stack.n_layers,
                "linears_per_layer": 7, "weight_bytes": stack.weight_bytes, "algorithmic_units_per_step": step_units,
                "l2": l2, "cuda_graph": graph is not None,
                "distinct_layers": stack.distinct,
                "parallelism": "replicas only" if world > 1 else "single GPU",
            },
            "tokens_per_s": M * world / (ms_per_step * 1e-3),
            "e2e": {"value": e2e_value, "unit": unit, "h2d_bytes_per_step": int(stack.xin_host.numel() * 2),
                    "d2h_bytes_per_step": int(stack.yout_host.numel() * 2), "steps": e2e_steps,
                    "ms_per_step": e2e_ms / e2e_steps},
            "gpu_launches": launches * args.steps,
            "clocks": sampler.summary(t0, t1),
            "roofline": roof,
        }
        if world == 1 and kind == "decode" and not args.no_secondary:
            line["secondary"] = secondary_measurements(lambda: stack, model, peaks, local_rank)
        if world == 1 and not args.no_cpu_baseline:
            sample, what, threads = oracle_sample(wl, model, args.cpu_seconds)
            t = time.perf_counter()
            passes = 0
            while passes == 0 or time.perf_counter() - t < args.cpu_seconds:   # about cpu_seconds of oracle work
                for x, q, s, z, _ in sample:
                    oracle_linear(kind, x, q, s, z)
                passes += 1
            spent = time.perf_counter() - t
            line["cpu_baseline"] = {
                "value": passes * sum(p[4] for p in sample) / spent / scale_of(kind), "unit": unit, "cores": threads,
                "kind": "oracle", "sample": "%s, %d pass(es), %.1f s of oracle time" % (what, passes, spent),
            }
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--no-graph", action="store_true", help="issue the launches directly instead of replaying a CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-secondary", action="store_true",
                    help="skip the extra measurements (prefill on the same weights, LM-head GEMVs) added to the line")
    ap.add_argument("--secondary-only", default=None, choices=sorted(SECONDARY) + ["int8_mma_ceiling"],
                    help="run one group of the secondary measurements alone and print it")
    ap.add_argument("--cpu-seconds", type=float, default=10.0, help="oracle time budget of the cpu_baseline leg")
    args = ap.parse_args()
    decode = WORKLOADS[args.workload]["kind"] == "decode"
    if args.steps is None:
        args.steps = (3000 if decode else 100) if args.impl == "ours" else 5
    if args.warmup is None:
        args.warmup = (50 if decode else 5) if args.impl == "ours" else 3
    args.steps = max(args.steps, 1)
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
