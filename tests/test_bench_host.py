"""Host-side checks of bench.py that need no GPU."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_never_loads_the_cuda_library():
    # the oracle arm must be able to run with libmnnllm_b200.so deleted: nothing it imports may import
    # the binding (which dlopens the library)
    code = (
        "import sys, types; sys.argv=['bench.py','--impl','reference','--steps','1','--warmup','3'];"
        "import bench; import numpy as np;"
        "wl=bench.WORKLOADS[bench.DEFAULT_WORKLOAD];"
        "from paper_2506_10443_b200 import inputs;"
        "sample=bench.oracle_prepare(wl, inputs.QWEN2_1P5B, 0, 0.002);"
        "[bench.oracle_linear(wl['kind'], x, q, s, z) for x, q, s, z, _ in sample];"
        "assert bench.units_of_linear('decode', 1536, 1536, 1) == 1536*1536//2 + 1536*24*4 + 2*1536 + 2*1536;"
        "assert 'paper_2506_10443_b200.binding' not in sys.modules, 'binding imported';"
        "assert 'paper_2506_10443_b200.workloads' not in sys.modules, 'workloads imported';"
        "print('ok')"
    )
    out = subprocess.run([sys.executable, "-c", code], cwd=ROOT, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and out.stdout.strip().endswith("ok"), out.stderr[-2000:]


def test_traffic_is_only_reported_for_an_unchanged_kernel(tmp_path, monkeypatch):
    sys.path.insert(0, ROOT)
    import bench

    prof = tmp_path / "profiles"
    prof.mkdir()
    name = bench.PROFILE_OF["decode_qwen2_1p5b_w4a16_g64"]
    sha = bench.kernel_sources_sha1(["gemv_w4a16.cu", "ptx.cuh"])
    (prof / name).write_text("x\ntraffic_bytes_per_launch = 12345\nkernel_sources = gemv_w4a16.cu ptx.cuh\n"
                             "kernel_sources_sha1 = %s\n" % sha)
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    monkeypatch.setattr(bench, "kernel_sources_sha1", lambda names: sha)
    assert bench.traffic_from_profile("decode_qwen2_1p5b_w4a16_g64") == 12345
    monkeypatch.setattr(bench, "kernel_sources_sha1", lambda names: "0" * 40)   # the kernel has changed since
    assert bench.traffic_from_profile("decode_qwen2_1p5b_w4a16_g64") is None
    assert bench.traffic_from_profile("no such workload") is None
