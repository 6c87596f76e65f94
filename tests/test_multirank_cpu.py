"""The path shards by batch with nothing to exchange, so several GPUs run independent replicas.
What the ranks share is only the timing protocol (barrier, max over ranks, rank 0 reports).
These tests run that logic as two gloo processes on the CPU."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=int(os.environ["RANK"]), world_size=2)
mine = 10.0 + 5.0 * dist.get_rank()          # rank 1 is the slow one
got = bench.max_over_ranks(mine, dist, "cpu")
dist.barrier()
assert got == 15.0, got
# whole-job value: units of all ranks over the slowest rank's time
flops_per_rank = 3.0e12
value = 2 * flops_per_rank / (got * 1e-3) / 1e12
print("rank", dist.get_rank(), "value", value)
dist.destroy_process_group()
"""


def test_max_over_ranks_two_gloo_processes(tmp_path):
    pytest.importorskip("torch")
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT, port=29731))
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT="29731")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=180) for p in procs]
    for p, (out, err) in zip(procs, outs):
        assert p.returncode == 0, err[-2000:]
        assert "value 400.0" in out


def test_reference_arm_only_rank0_reports(tmp_path):
    """Under a multi-rank launch the oracle arm runs on rank 0 alone; other ranks exit 0 silently."""
    results = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), OMP_NUM_THREADS="2")
        r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                            "--steps", "1", "--warmup", "0", "--workload", "fc_small"],
                           env=env, capture_output=True, text=True, timeout=600)
        assert r.returncode == 0, r.stderr[-2000:]
        results.append(r.stdout.strip())
    assert results[1] == ""
    line = json.loads(results[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["gpu_launches"] == 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0
