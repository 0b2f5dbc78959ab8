"""The N > 1 path of the benchmark on CPU: two `gloo` ranks.

With several GPUs every rank runs an independent job of the same shape (no
collective on the data path); what the ranks share is the timing protocol:
barrier, slowest rank's time, whole-job throughput.  That host logic, and the
rank-0-only behaviour of the oracle arm, are exercised here without a GPU.
"""
import json
import os
import subprocess
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["CCDC_ROOT"])
import torch, torch.distributed as dist
import bench
from paper_1805_01993_b200 import build, ccdc
from paper_1805_01993_b200.inputs import values_numpy

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
# the slowest rank decides: rank r pretends to have needed 10*(r+1) ms for 4 steps
ms = bench.max_over_ranks(10.0 * (rank + 1), world, "cpu") / 4
value = bench.whole_job_value(world, 1_000_000_000, ms)
# independent jobs: same plan on every rank (host-only call), different inputs
build.build_library()
plan = ccdc.Plan(4, 2, 12, 4, 16, "int32")
v = values_numpy(12, 4, 16, "int32", seed=bench.rank_seed(rank))
sig = torch.tensor([float(int(v.view("uint32").sum() % 1000003)), float(plan.coded_bits)], dtype=torch.float64)
gathered = [torch.zeros_like(sig) for _ in range(world)]
dist.all_gather(gathered, sig)
dist.barrier()
if rank == 0:
    print(json.dumps({"ms": ms, "value": value, "sums": [g[0].item() for g in gathered],
                      "bits": [g[1].item() for g in gathered]}))
dist.destroy_process_group()
"""


def run_two_ranks(script_args, env_extra=None):
    env = dict(os.environ, CCDC_ROOT=str(ROOT), MASTER_ADDR="127.0.0.1")
    env.update(env_extra or {})
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29517"] + script_args
    return subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=600, cwd=str(ROOT))


def test_timing_protocol_and_independent_jobs(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    res = run_two_ranks([str(script)])
    assert res.returncode == 0, res.stderr[-2000:]
    line = [l for l in res.stdout.splitlines() if l.startswith("{")][-1]
    out = json.loads(line)
    assert out["ms"] == pytest.approx(20.0 / 4)                 # max over ranks, per step
    assert out["value"] == pytest.approx(2 * 1e9 / 5e-3 / 1e9)  # both ranks' bytes over the slowest time
    assert out["bits"][0] == out["bits"][1]                     # same scheme on every rank
    assert out["sums"][0] != out["sums"][1]                     # different synthetic inputs


def test_reference_arm_runs_on_rank0_only():
    """`bench.py --impl reference` under torchrun: rank 0 prints the one line, the
    other rank exits 0 without work."""
    res = run_two_ranks(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                         "--workload", "cfg1"])
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    out = json.loads(lines[0])
    assert out["impl"] == "reference" and out["n_gpus"] == 2 and out["cpu_baseline"]["kind"] == "oracle"
    assert out["e2e"]["h2d_bytes_per_step"] == 0 and out["value"] > 0
