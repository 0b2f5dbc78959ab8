"""The several-GPU forms of the shuffle, checked on one GPU against the oracle.

* value-dimension shards: the ranks' jobs run one after the other; the output
  slices scattered back give the unsharded outputs, the coded rows are slices of
  the unsharded coded rows;
* gamma groups of jobs in one plan;
* node shards with peer stores: two PROCESSES share the one GPU, each maps the
  other's coded buffer (CUDA IPC) and its encode kernel stores every row into both
  buffers.  No kernel of one rank waits for the other: the ranks meet on the host
  between the encode and the decode.
"""
import json
import os
import subprocess
import sys
from pathlib import Path

import numpy as np
import pytest

from oracle.ccdc_oracle import Oracle
from paper_1805_01993_b200.inputs import values_numpy

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def ccdc():
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    from paper_1805_01993_b200 import build, ccdc as mod

    build.build_library()
    mod.lib()
    return mod


def bits(t):
    return t.detach().cpu().contiguous().numpy().view(np.uint32)


@pytest.mark.parametrize("dtype", ["int32", "float32"])
@pytest.mark.parametrize("K,r,N,Q,B,world", [(4, 2, 12, 4, 64, 2), (6, 3, 20, 12, 3 * 1030, 5), (10, 3, 480, 10, 96, 4),
                                             (5, 2, 10, 5, 2 * 4100, 2), (6, 1, 12, 6, 21, 3)])
def test_value_shards_run_alone_and_add_up(ccdc, K, r, N, Q, B, world, dtype):
    o = Oracle(K, r, N, Q, B, dtype)
    v = values_numpy(N, Q, B, dtype, seed=world)
    o.load_values(v)
    o.shuffle()
    ref_coded = o.coded().reshape(-1, o.s)
    full_v = torch.from_numpy(v).cuda()
    tdt = full_v.dtype
    out = torch.full((Q, B), 7, dtype=tdt, device="cuda")
    total_bits = 0
    w = o.s // world
    for rank in range(world):
        b_local = ccdc.value_shard(K, r, Q, B, rank, world)
        local_v = torch.empty((N, Q, b_local), dtype=tdt, device="cuda")
        ccdc.value_shard_copy(K, r, Q, B, rank, world, True, full_v, local_v, N)
        plan = ccdc.Plan(K, r, N, Q, b_local, dtype)
        assert plan.segment_elems == w
        part = plan.alloc_partitions()
        plan.fill_partitions(part, local_v)
        coded = plan.alloc(plan.coded_bytes)
        out_local = plan.alloc(plan.out_bytes)
        plan.shuffle(part, coded, out_local, plan.alloc(plan.workspace_bytes))
        ccdc.value_shard_copy(K, r, Q, B, rank, world, False, out_local, out, 1)
        torch.cuda.synchronize()
        got = bits(coded).reshape(-1, plan.coded_row_elems)[:, :w]
        assert np.array_equal(got, ref_coded[:, rank * w:(rank + 1) * w])
        total_bits += plan.coded_bits
    assert total_bits == o.coded_bits
    ref = o.reduce()
    got = out.cpu().numpy()
    if dtype == "int32":
        assert np.array_equal(got, ref)
    else:
        _, a64 = o.direct()
        assert np.all(np.abs(got.astype(np.float64) - ref.astype(np.float64)) <= 1e-5 * a64 + 1e-30)
    with pytest.raises(ccdc.CcdcError):
        ccdc.value_shard(K, r, Q, B, 0, 7 * o.s + 1)


@pytest.mark.parametrize("dtype", ["int32", "float32"])
@pytest.mark.parametrize("K,r,N,Q,B,gamma", [(4, 2, 6, 4, 40, 2), (5, 2, 9, 5, 37, 3), (6, 3, 8, 12, 2050, 2)])
def test_gamma_groups_of_jobs_in_one_plan(ccdc, K, r, N, Q, B, gamma, dtype):
    """J = gamma * C(K, r+1) jobs through the same two launches: each group against the oracle's
    J-job run on that group's files."""
    plan = ccdc.Plan(K, r, N, Q, B, dtype, jobs=True, gamma=gamma)
    group_jobs = plan.J // gamma
    v = values_numpy(plan.J * N, Q, B, dtype, seed=gamma)
    part = plan.alloc_partitions()
    plan.fill_partitions(part, torch.from_numpy(v).cuda())
    coded = plan.alloc(plan.coded_bytes)
    out = plan.alloc(plan.out_bytes)
    plan.shuffle(part, coded, out, plan.alloc(plan.workspace_bytes))
    torch.cuda.synchronize()
    s, sp = plan.segment_elems, plan.coded_row_elems
    got_coded = bits(coded).reshape(gamma, -1, sp)[:, :, :s]
    got_out = out.cpu().numpy().reshape(gamma, group_jobs * Q, B)
    bits_total = 0
    for g in range(gamma):
        o = Oracle(K, r, N, Q, B, dtype, mode="paper")
        o.load_values(v[g * group_jobs * N:(g + 1) * group_jobs * N])
        o.shuffle()
        assert np.array_equal(got_coded[g], o.coded().reshape(-1, s))
        ref = o.reduce().reshape(group_jobs * Q, B)
        if dtype == "int32":
            assert np.array_equal(got_out[g], ref)
        else:
            _, a64 = o.direct()
            err = np.abs(got_out[g].astype(np.float64) - ref.astype(np.float64))
            assert np.all(err <= 1e-5 * a64.reshape(ref.shape) + 1e-30)
        bits_total += o.coded_bits
    assert plan.coded_bits == bits_total


PEER_WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["CCDC_ROOT"])
import numpy as np, torch, torch.distributed as dist
from oracle.ccdc_oracle import Oracle
from paper_1805_01993_b200 import ccdc
from paper_1805_01993_b200.inputs import values_numpy

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
torch.cuda.set_device(0)                            # both ranks share the one GPU
K, r, N, Q, B, dtype = 6, 2, 15, 6, 5000, os.environ["CCDC_DTYPE"]
plan = ccdc.Plan(K, r, N, Q, B, dtype, shard=(rank, world))
v = values_numpy(N, Q, B, dtype, seed=12)
o = Oracle(K, r, N, Q, B, dtype)
o.load_values(v); o.shuffle()
part = plan.alloc_partitions()
plan.fill_partitions(part, torch.from_numpy(v).cuda())
mine = ccdc.PeerBuffer.create(plan.coded_bytes)
handles = [None] * world
dist.all_gather_object(handles, mine.handle)        # 64 bytes per rank over the host channel
peers = [mine if d == rank else ccdc.PeerBuffer.open(handles[d], plan.coded_bytes) for d in range(world)]
plan.encode_fused_peers(part, peers)                # every row this rank's nodes send, into both buffers
torch.cuda.synchronize()
dist.barrier()                                      # the other rank's rows have landed in my buffer
coded = plan.alloc(plan.coded_bytes)
mine.copy_to(coded)
out = torch.zeros(Q * B, dtype=plan.torch_dtype, device="cuda")
plan.decode_reduce(part, mine, out, plan.alloc(plan.workspace_bytes))
torch.cuda.synchronize()
s, sp = plan.segment_elems, plan.coded_row_elems
got = coded.cpu().numpy().view(np.uint32).reshape(-1, sp)[:, :s]
ref = o.coded().reshape(-1, s)
order = [plan.coded_row_position(g, a) for g in range(plan.num_groups) for a in range(r + 1)]
coded_ok = bool(np.array_equal(got[order], ref))
# outputs of my nodes
want = o.reduce().reshape(K, -1)
have = out.cpu().numpy().reshape(K, -1)
nodes = [k for k in range(K) if plan.node_is_local(k)]
if dtype == "int32":
    out_ok = all(np.array_equal(have[k], want[k]) for k in nodes)
else:
    _, a64 = o.direct()
    a64 = a64.reshape(K, -1)
    out_ok = all(np.all(np.abs(have[k].astype(np.float64) - want[k].astype(np.float64)) <= 1e-5 * a64[k] + 1e-30) for k in nodes)
dist.barrier()                                      # nobody unmaps a buffer the other still reads
for d, p in enumerate(peers):
    if d != rank:
        p.release()
dist.barrier()
mine.release()
res = [None] * world
dist.all_gather_object(res, {"rank": rank, "coded_ok": coded_ok, "out_ok": bool(out_ok), "nodes": nodes})
if rank == 0:
    print(json.dumps(res))
dist.destroy_process_group()
"""


@pytest.mark.parametrize("dtype", ["int32", "float32"])
def test_peer_stores_between_two_processes_on_one_gpu(ccdc, tmp_path, dtype):
    script = tmp_path / "peer_worker.py"
    script.write_text(PEER_WORKER)
    env = dict(os.environ, CCDC_ROOT=str(ROOT), MASTER_ADDR="127.0.0.1", CCDC_DTYPE=dtype)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29533", str(script)]
    res = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=600, cwd=str(ROOT))
    assert res.returncode == 0, res.stdout[-1500:] + res.stderr[-3000:]
    out = json.loads([l for l in res.stdout.splitlines() if l.startswith("[{")][-1])
    assert len(out) == 2 and all(x["coded_ok"] and x["out_ok"] for x in out)
    assert sorted(out[0]["nodes"] + out[1]["nodes"]) == list(range(6))
