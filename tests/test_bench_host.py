"""Host-side logic of the bench: FLOP/byte accounting against hand-computed totals, the
replica aggregation across ranks (gloo, world size 2), and the reference arm's JSON line."""
import json
import os
import subprocess
import sys

import pytest

import bench
from paper_1901_00858_b200 import workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_flop_totals_match_the_network_arithmetic():
    tot = lambda wl: sum(bench.layer_flops(wl.batch, l) for l in wl.expanded())
    assert abs(tot(workloads.workload(0)) - 2 * 16 * 3 * 9 * 32 * 32) < 1
    assert abs(tot(workloads.workload(1)) / 1e9 - 0.659) < 0.001
    assert abs(tot(workloads.workload(2, 1)) / 1e9 - 30.69) < 0.01
    assert abs(tot(workloads.workload(2, 16)) / 1e9 - 491.1) < 0.1
    assert abs(tot(workloads.workload(3, 1)) / 1e9 - 1.135) < 0.002
    assert abs(tot(workloads.workload(4, 64)) / 1e9 - 477.1) < 0.1
    assert len(workloads.workload(4).expanded()) == 49
    assert len(workloads.workload(4).expanded_unique()) == 20
    assert sum(l.count for l in workloads.workload(4).expanded_unique()) == 49
    assert len(workloads.workload(3).expanded()) == 27
    byt = sum(bench.layer_bytes(64, l) for l in workloads.workload(4).expanded())
    assert abs(byt / 1e6 - 2430.6) < 0.5


def test_aggregate_is_sum_over_max():
    a = bench.aggregate([1e12, 1e12], [16, 16], 0.5)
    assert a["tflops"] == pytest.approx(4.0) and a["images_per_s"] == pytest.approx(64.0)


_WORKER = r"""
import os, sys, torch, torch.distributed as dist
sys.path.insert(0, os.environ["HGC_ROOT"])
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
# each replica reports its own time; the job's step time is the slowest rank's
ms = torch.tensor([10.0 + 5.0 * rank], dtype=torch.float64)
dist.all_reduce(ms, op=dist.ReduceOp.MAX)
launches = torch.tensor([13], dtype=torch.int64)
dist.all_reduce(launches)
agg = bench.aggregate([2e12] * world, [16] * world, float(ms[0]) * 1e-3)
if rank == 0:
    print("RESULT", float(ms[0]), int(launches[0]), agg["tflops"], agg["images_per_s"])
dist.destroy_process_group()
"""


def test_replica_aggregation_over_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER)
    env = dict(os.environ, HGC_ROOT=ROOT)
    out = subprocess.run(
        [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
         "--master-addr", "127.0.0.1", "--master-port", "29573", str(script)],
        env=env, capture_output=True, text=True, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    line = [l for l in out.stdout.splitlines() if l.startswith("RESULT")][0].split()
    assert float(line[1]) == 15.0 and int(line[2]) == 26
    assert float(line[3]) == pytest.approx(2 * 2e12 / 15e-3 / 1e12)
    assert float(line[4]) == pytest.approx(32 / 15e-3)


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--workload", "alexnet_pair_n1", "--steps", "2", "--warmup", "1"],
                         capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    d = json.loads(out.stdout.strip().splitlines()[-1])
    assert d["impl"] == "reference" and d["unit"] == "TFLOP/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
