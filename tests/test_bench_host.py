"""Host logic of bench.py (no GPU): the clock sampler's parsing and time windows against a fake nvidia-smi, the
peak table, the kernel-sources hash that gates `roofline.traffic`, the workload shapes, and the oracle arm on a
tiny layer."""
import json
import os
import stat
import subprocess
import sys
import time

import numpy as np
import pytest

import bench
from paper_2202_00774_b200 import inputs

FAKE_SMI = """#!/usr/bin/env python3
import datetime, sys, time
n = 0
while True:
    now = datetime.datetime.now().strftime("%Y/%m/%d %H:%M:%S.%f")[:-3]
    clock = 1965 if n % 2 == 0 else 1800
    cap = "Active" if n % 2 else "Not Active"
    print("%s, %d, 1965, 700.0, 0x4, Not Active, Not Active, Not Active, %s" % (now, clock, cap), flush=True)
    n += 1
    time.sleep(0.02)
"""


@pytest.fixture
def fake_smi(tmp_path, monkeypatch):
    exe = tmp_path / "nvidia-smi"
    exe.write_text(FAKE_SMI.replace("/usr/bin/env python3", sys.executable))
    exe.chmod(exe.stat().st_mode | stat.S_IEXEC)
    monkeypatch.setenv("PATH", str(tmp_path) + os.pathsep + os.environ["PATH"])
    return exe


def test_clock_sampler_reports_only_samples_inside_the_windows(fake_smi):
    s = bench.ClockSampler(0)
    time.sleep(0.3)                      # samples before the first window: must not count
    s.begin()
    time.sleep(0.4)
    s.end()
    time.sleep(0.3)
    out = s.stop()
    assert 5 <= out["samples"] <= 30     # 0.4 s at 20 ms per line, not the whole second
    assert out["sm_max_mhz"] == 1965.0
    assert out["sm_mhz"] in (1800.0, 1882.5, 1965.0)
    assert out["reasons"] == ["sw_power_cap"]


def test_clock_sampler_without_windows_reports_everything(fake_smi):
    s = bench.ClockSampler(0)
    time.sleep(0.3)
    out = s.stop()
    assert out["samples"] >= 5


def test_clock_sampler_survives_a_missing_tool(monkeypatch, tmp_path):
    monkeypatch.setenv("PATH", str(tmp_path))
    out = bench.ClockSampler(0).stop()
    assert out == {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}


def test_peaks_measured_and_fallback(monkeypatch, tmp_path):
    pk = bench.peaks()
    assert pk["hbm"] > 1000 and pk["bf16"] >= pk["bf16_sustained"] > 100
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    assert bench.peaks()["source"] == "fallback"
    (tmp_path / "MEASURED_PEAKS.json").write_text(json.dumps({"hbm_gbs": 6000, "bf16_tflops": 1500}))
    pk = bench.peaks()
    assert pk == dict(hbm=6000.0, bf16=1500.0, bf16_sustained=1500.0, source="measured")


def test_kernel_sources_hash_ignores_comments_but_not_code(monkeypatch, tmp_path):
    src = tmp_path / "paper_2202_00774_b200" / "csrc"
    src.mkdir(parents=True)
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))

    def write(dgrad, ptx="int y;\n"):
        (src / "dgrad.cu").write_text(dgrad)
        (src / "ptx.cuh").write_text(ptx)
        return bench.kernel_sources_sha()

    base = write("int x = 1;  // one\n\nint z;\n")
    assert write("// a new heading\nint x = 1;  // uno\nint z;\n") == base
    assert write("int x = 2;  // one\n\nint z;\n") != base
    assert write("int x = 1;\nint z;\n", ptx="int y = 0;\n") != base


def test_traffic_is_reported_only_for_the_sources_it_was_measured_on(monkeypatch):
    assert bench.measured_traffic("gemm_large", "two_pass") is None
    assert bench.measured_traffic("resnet9", "fused") is None
    monkeypatch.setitem(bench.NCU_TRAFFIC, "sources_sha", "0" * 16)
    assert bench.measured_traffic("resnet9", "two_pass") is None


def test_workloads_have_the_shapes_the_metric_is_quoted_on():
    r9 = bench.workload_layers("resnet9")
    assert [(l.Cout, l.Cin, l.H) for l in r9] == [(128, 64, 32), (128, 128, 16), (128, 128, 16), (256, 128, 16),
                                                  (512, 256, 8), (512, 512, 4), (512, 512, 4)]
    assert all(l.B == 512 and l.R == 3 and l.stride == 1 for l in r9)
    assert sum(bench.layer_flops(l) for l in r9) == pytest.approx(386.5e9, rel=1e-3)
    (g,) = bench.workload_layers("gemm_large")
    assert bench.layer_flops(g) == 2.0 * 16384 * 4096 * 4096
    (f,) = bench.workload_layers("fc_small")
    assert bench.layer_flops(f) == 2.0 * 256 * 512 * 256


def test_oracle_arm_counts_the_flops_of_its_sample():
    layer = inputs.ConvLayer("tiny", 2, 6, 6, 16, 32, 3, 3, 1, 1)
    arm = bench.OracleArm([layer], "resnet9", 2, 4, bench.SCHEMES["magnitude"])
    flops = arm.step(10)
    assert arm.last_pixels == [10]
    assert flops == 2.0 * 10 * 16 * 9 * 32
    assert arm.step(10 ** 6) == 2.0 * 72 * 16 * 9 * 32      # capped at the layer's pixels


def test_reference_arm_prints_one_json_line_on_rank_zero_only():
    env = dict(os.environ, RANK="1")
    out = subprocess.run([sys.executable, os.path.join(bench.ROOT, "bench.py"), "--impl", "reference", "--workload", "fc_small",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env["RANK"] = "0"
    out = subprocess.run([sys.executable, os.path.join(bench.ROOT, "bench.py"), "--impl", "reference", "--workload", "fc_small",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["gpu_launches"] == 0 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
