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


SHARD_WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["CCDC_ROOT"])
import numpy as np, torch, torch.distributed as dist
from oracle.ccdc_oracle import Oracle
from paper_1805_01993_b200 import build, ccdc
from paper_1805_01993_b200.inputs import values_numpy

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
build.build_library()
K, r, N, Q, B = 6, 2, 15, 6, 20
plan = ccdc.Plan(K, r, N, Q, B, "int32", shard=(rank, world))
o = Oracle(K, r, N, Q, B, "int32")
o.run(values_numpy(N, Q, B, "int32", seed=4))
ref = o.coded()                                     # [round][sender rank][s]
sp, s = plan.coded_row_elems, plan.segment_elems
# what this rank's nodes send, in the order of the rank's send buffer (stand-in for the encode kernel)
send = torch.zeros(plan.coded_send_bytes // 4, dtype=torch.int32).view(-1, sp)
per = send.shape[0]
for g in range(plan.num_groups):
    for a, k in enumerate(plan.group(g)):
        if plan.node_is_local(k):
            send[plan.coded_row_position(g, a) - rank * per, :s] = torch.from_numpy(ref[g, a].view(np.int32))
coded = torch.zeros(plan.coded_bytes // 4, dtype=torch.int32)
dist.all_gather_into_tensor(coded, send.reshape(-1))        # the exchange between GPUs
coded = coded.view(-1, sp)
ok = all(np.array_equal(coded[plan.coded_row_position(g, a), :s].numpy().view(np.uint32), ref[g, a])
         for g in range(plan.num_groups) for a in range(r + 1))
flag = torch.tensor([1 if ok else 0])
dist.all_reduce(flag, op=dist.ReduceOp.MIN)
if rank == 0:
    print(json.dumps({"ok": int(flag.item()), "rows": int(coded.shape[0]), "send_rows": per}))
dist.destroy_process_group()
"""


VALUE_SHARD_WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["CCDC_ROOT"])
import numpy as np, torch, torch.distributed as dist
from oracle.ccdc_oracle import Oracle
from paper_1805_01993_b200 import build, ccdc
from paper_1805_01993_b200.inputs import values_numpy

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
build.build_library()
K, r, N, Q, B = 4, 2, 12, 8, 12                     # Q/K = 2: packets of 24 words, segments of 12, 6 per rank
per = Q // K
v = values_numpy(N, Q, B, "int32", seed=8)
full = Oracle(K, r, N, Q, B, "int32")
want = full.run(v)                                   # [Q][B]
b_local = ccdc.value_shard(K, r, Q, B, rank, world)
pos = np.array([ccdc.value_shard_position(K, r, Q, B, rank, world, x) for x in range(per * b_local)])
# this rank's slice of every packet (the library's position map applied in numpy), shuffled alone
packets = v.reshape(N, K, per * B)
local = np.ascontiguousarray(packets[:, :, pos]).reshape(N, Q, b_local)
o = Oracle(K, r, N, Q, b_local, "int32")
mine = torch.from_numpy(o.run(local).reshape(K, per * b_local).copy())
# the only traffic between the ranks: the output slices, gathered at the end
parts = [torch.zeros_like(mine) for _ in range(world)]
dist.all_gather(parts, mine)
got = np.zeros((K, per * B), dtype=np.int32)
for g, t in enumerate(parts):
    where = [ccdc.value_shard_position(K, r, Q, B, g, world, x) for x in range(per * b_local)]
    got[:, where] = t.numpy()
bits = torch.tensor([o.coded_bits], dtype=torch.int64)
dist.all_reduce(bits)
if rank == 0:
    print(json.dumps({"ok": int(np.array_equal(got.reshape(Q, B), want)), "bits": int(bits.item()),
                      "full_bits": int(full.coded_bits)}))
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


def test_node_sharded_exchange_over_a_real_all_gather(tmp_path):
    """Two ranks, three logical nodes each: the rows each rank's nodes send (taken from
    the oracle, standing in for the encode kernel) are all-gathered with gloo and
    every coded row is found where the plan says the decode will look for it."""
    script = tmp_path / "shard_worker.py"
    script.write_text(SHARD_WORKER)
    res = run_two_ranks([str(script)])
    assert res.returncode == 0, res.stderr[-2000:]
    out = json.loads([l for l in res.stdout.splitlines() if l.startswith("{")][-1])
    assert out["ok"] == 1 and out["rows"] == 2 * out["send_rows"] == 20 * 3


def test_value_shards_need_no_exchange(tmp_path):
    """Two ranks, each owning half of every segment: each runs the whole scheme (here the oracle,
    standing in for the kernels) on its slice alone; gathering the output slices gives the
    unsharded job's outputs, and the ranks' multicast bits add up to the unsharded count."""
    script = tmp_path / "value_shard_worker.py"
    script.write_text(VALUE_SHARD_WORKER)
    res = run_two_ranks([str(script)])
    assert res.returncode == 0, res.stderr[-2000:]
    out = json.loads([l for l in res.stdout.splitlines() if l.startswith("{")][-1])
    assert out["ok"] == 1 and out["bits"] == out["full_bits"]


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
