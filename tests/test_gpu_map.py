"""Parity of the tensor-core Map (partial gradients of linear regression) and of
the whole job Map -> shuffle -> reduce with the CPU oracle.

The oracle evaluates g = X^T (X w - y) in binary64 on the same bf16-representable
X and w and rounds once to fp32.  The CUDA Map accumulates bf16 products in fp32,
so its values agree to fp32 accumulation error, not bit for bit; what must hold
exactly is that the r replicas of a file's values are bit-identical (XOR decoding
depends on it).  Tolerances:
  Map value j:      |gpu - oracle| <= 1e-5 * sum_i |X_ij| |u_i|
  Reduce output:    |gpu - oracle| <= 1e-5 * sum_n |v_{q,n}|   (the evaluation's rule)
"""
import numpy as np
import pytest

from oracle.ccdc_oracle import Oracle, map_linear_regression
from paper_1805_01993_b200.inputs import CONFIGS, bf16_bits, regression_files

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def ccdc():
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    from paper_1805_01993_b200 import build, ccdc as mod

    build.build_library()
    mod.lib()
    return mod


def to_bf16_cuda(a):
    return torch.from_numpy(bf16_bits(a).view(np.int16)).cuda().view(torch.bfloat16)


def run_job(ccdc, K, r, N, Q, B, rows, seed):
    d = Q * B
    X, y, w = regression_files(N, rows, d, seed=seed)
    plan = ccdc.Plan(K, r, N, Q, B, "float32")
    # ---- oracle: Map in binary64, then the scheme
    v = np.stack([map_linear_regression(X[n], w, y[n], Q) for n in range(N)])
    o = Oracle(K, r, N, Q, B, "float32")
    ref_out = o.run(v)
    # ---- CUDA: every node maps its own copy of its files
    files_x, files_y = [], []
    for k in range(K):
        idx = plan.node_files(k)
        files_x.append(to_bf16_cuda(X[idx]).contiguous())
        files_y.append(torch.from_numpy(y[idx]).cuda().contiguous())
    wd = to_bf16_cuda(w)
    part = plan.alloc_partitions()
    for p in part:
        p.fill_(float("nan"))
    ws = torch.empty(plan.map_workspace_bytes(rows) // 4, dtype=torch.float32, device="cuda")
    before = ccdc.num_kernel_launches()
    plan.map(files_x, files_y, wd, rows, part, ws)
    torch.cuda.synchronize()
    plan.map_status(rows, ws)
    assert ccdc.num_kernel_launches() - before >= 1
    # Map values against the oracle, and replicas against each other
    Xd = X.astype(np.float64)
    u = np.einsum("nij,j->ni", Xd, w.astype(np.float64)) - y.astype(np.float64)
    scale = np.einsum("nij,ni->nj", np.abs(Xd), np.abs(u))            # sum_i |X_ij||u_i|
    first = {}
    worst = 0.0
    for k in range(K):
        got = part[k].cpu().numpy().reshape(-1, d)
        for i, n in enumerate(plan.node_files(k)):
            err = np.abs(got[i].astype(np.float64) - v[n].reshape(-1))
            assert np.all(err <= 1e-5 * scale[n]), (k, n, float((err / scale[n]).max()))
            worst = max(worst, float((err / scale[n]).max()))
            if n in first:
                assert np.array_equal(first[n].view(np.uint32), got[i].view(np.uint32)), \
                    f"replicas of file {n} differ"
            else:
                first[n] = got[i].copy()
    assert len(first) == N
    # ---- shuffle + reduce on the mapped partitions
    coded = plan.alloc(plan.coded_bytes)
    out = plan.alloc(plan.out_bytes)
    wsp = plan.alloc(plan.workspace_bytes)
    plan.shuffle(part, coded, out, wsp)
    torch.cuda.synchronize()
    got_out = out.cpu().numpy().reshape(Q, B)
    _, a64 = o.direct()
    err = np.abs(got_out.astype(np.float64) - ref_out.astype(np.float64))
    assert np.all(err <= 1e-5 * a64), float((err / a64).max())
    # the full gradient: sum over all files, against binary64
    full = np.einsum("nij,ni->j", Xd, u).reshape(Q, B)
    assert np.all(np.abs(got_out - full) <= 1e-5 * a64)
    # exact consistency on the device side: the shuffle of the GPU's own Map values
    # must reproduce their fixed-order sum (decode loses nothing)
    mine = np.stack([first[n].reshape(Q, B) for n in range(N)])
    o2 = Oracle(K, r, N, Q, B, "float32")
    ref2 = o2.run(mine)
    s, sp = plan.segment_elems, plan.coded_row_elems
    assert np.array_equal(coded.cpu().numpy().view(np.uint32).reshape(-1, sp)[:, :s], o2.coded().reshape(-1, s))
    _, a2 = o2.direct()
    assert np.all(np.abs(got_out.astype(np.float64) - ref2) <= 1e-5 * a2)
    return worst


def test_map_small(ccdc):
    worst = run_job(ccdc, 4, 2, 12, 4, 128, rows=32, seed=7)
    assert worst < 1e-5
    assert ccdc.map_last_kernel() == "k_map"        # d = 512: served by the register kernel


def test_map_wide_files(ccdc):
    # d = 2048 columns, 48 rows, r = K-1: the smallest shape of the cluster kernel (one block per cluster)
    run_job(ccdc, 4, 3, 8, 4, 512, rows=48, seed=8)
    assert ccdc.map_last_kernel() == "k_map_cluster"


def test_map_cluster_of_two_with_split_files(ccdc):
    # d = 4096 (clusters of two blocks), 128 rows = 4 units per file, 24 Map executions: with more
    # clusters than files every file is cut over several clusters and summed by the combine pass
    run_job(ccdc, 4, 2, 12, 4, 1024, rows=128, seed=10)
    assert ccdc.map_last_kernel() == "k_map_cluster"


def test_cfg5_full_job(ccdc):
    w = CONFIGS["cfg5"]
    worst = run_job(ccdc, w.K, w.r, w.N, w.Q, w.B, rows=w.map_rows, seed=9)
    assert worst < 1e-5
    assert ccdc.map_last_kernel() == "k_map_cluster"


@pytest.mark.parametrize("K,r,N,Q,B,rows", [
    (4, 2, 12, 4, 512, 32),      # d = 2048, one block per cluster, one row block per cluster (shortest pipeline)
    (4, 2, 12, 4, 512, 64),      # d = 2048, two row blocks per unit, every file cut over four clusters
    (4, 2, 12, 4, 2048, 48),     # d = 8192, clusters of four, rows not a multiple of 32: one unit per file
    (4, 2, 12, 4, 4096, 32),     # d = 16384, clusters of eight
    (4, 3, 4, 4, 512, 4096),     # the longest files the call accepts
    (6, 2, 15, 6, 1024, 160),    # d = 6144 is not a cluster shape: register kernel
])
def test_map_cluster_shapes(ccdc, K, r, N, Q, B, rows):
    worst = run_job(ccdc, K, r, N, Q, B, rows=rows, seed=11 + rows)
    assert worst < 1e-5
    d = Q * B
    assert ccdc.map_last_kernel() == ("k_map_cluster" if d in (2048, 4096, 8192, 16384) else "k_map")


def test_job_from_host_buffers(ccdc):
    """ccdc_job_host (copies in, Map, shuffle, copy out) gives bit for bit what the separate calls give on
    device-resident inputs, and its outputs match the oracle."""
    K, r, N, Q, B, rows = 4, 2, 12, 4, 512, 64
    d = Q * B
    X, y, w = regression_files(N, rows, d, seed=21)
    plan = ccdc.Plan(K, r, N, Q, B, "float32")
    hx = [torch.from_numpy(bf16_bits(X[plan.node_files(k)]).view(np.int16)).pin_memory() for k in range(K)]
    hy = [torch.from_numpy(np.ascontiguousarray(y[plan.node_files(k)])).pin_memory() for k in range(K)]
    hw = torch.from_numpy(bf16_bits(w).view(np.int16)).pin_memory()
    dx = [torch.empty_like(t, device="cuda") for t in hx]
    dy = [torch.empty_like(t, device="cuda") for t in hy]
    dw = torch.empty_like(hw, device="cuda")
    part = plan.alloc_partitions()
    coded, out, wsp = plan.alloc(plan.coded_bytes), plan.alloc(plan.out_bytes), plan.alloc(plan.workspace_bytes)
    mws = torch.empty(plan.map_workspace_bytes(rows) // 4, dtype=torch.float32, device="cuda")
    host_out = torch.empty(out.numel(), dtype=out.dtype).pin_memory()
    plan.job_host(hx, hy, hw, rows, host_out, dx, dy, dw, part, coded, out, mws, wsp)
    torch.cuda.synchronize()
    plan.map_status(rows, mws)
    # the separate calls on the device copies
    part2 = plan.alloc_partitions()
    out2, coded2 = plan.alloc(plan.out_bytes), plan.alloc(plan.coded_bytes)
    plan.map([t.view(torch.bfloat16) for t in dx], dy, dw.view(torch.bfloat16), rows, part2, mws)
    plan.shuffle(part2, coded2, out2, wsp)
    torch.cuda.synchronize()
    assert torch.equal(host_out, out2.cpu())
    # and the oracle on the binary64 Map values
    v = np.stack([map_linear_regression(X[n], w, y[n], Q) for n in range(N)])
    o = Oracle(K, r, N, Q, B, "float32")
    ref = o.run(v)
    _, a64 = o.direct()
    got = host_out.numpy().view(np.float32).reshape(Q, B).astype(np.float64)
    assert np.all(np.abs(got - ref) <= 1e-5 * a64)


REGISTER_VARIANT = r"""
import sys
sys.path.insert(0, sys.argv[1])
from pathlib import Path
from paper_1805_01993_b200 import build, ccdc
ccdc._LIB_PATH = build.build_variant(Path(sys.argv[2]) / "libccdc_reg.so", ("CCDC_MAP_USE_CLUSTER=0",))
sys.path.insert(0, str(Path(sys.argv[1]) / "tests"))
import test_gpu_map as t
t.run_job(ccdc, 4, 2, 12, 4, 128, rows=32, seed=7)
t.run_job(ccdc, 4, 3, 8, 4, 512, rows=48, seed=8)
t.run_job(ccdc, 8, 3, 112, 8, 1024, rows=128, seed=9)
assert ccdc.map_last_kernel() == "k_map"
print("register variant ok")
"""


@pytest.mark.parametrize("seed", [31, 32])
def test_drawn_map_jobs(ccdc, seed):
    """Ten drawn jobs per seed inside the shapes the Map accepts (rows a multiple of 16, d a multiple of
    512): K up to 8, every r, up to 3 files per batch, Q/K up to 2; Map values, replicas, coded rows and
    outputs as in run_job.  Both Map kernels are reached."""
    import random
    from math import comb

    rng = random.Random(seed)
    done, kernels = 0, set()
    while done < 10:
        K = rng.randint(3, 8)
        r = rng.randint(1, K - 1)
        N = rng.choice([1, 1, 2, 3]) * comb(K, r)
        Q = K * rng.choice([1, 1, 2])
        d = 512 * rng.choice([1, 2, 3, 4, 4, 5, 8, 8, 12, 16, 16, 32, 32])
        rows = 16 * rng.choice([1, 2, 2, 3, 4, 5, 8, 10, 16, 32])
        if comb(K, r) > 60 or N < K or d % Q or N * rows * d > 40_000_000:
            continue
        try:
            worst = run_job(ccdc, K, r, N, Q, d // Q, rows=rows, seed=seed * 100 + done)
        except AssertionError as e:
            raise AssertionError(f"{(K, r, N, Q, d // Q, rows)}: {e}") from e
        assert worst < 1e-5
        kernels.add(ccdc.map_last_kernel())
        done += 1
    assert kernels == {"k_map", "k_map_cluster"}


def test_register_kernel_on_cluster_shapes(ccdc, tmp_path):
    """The register kernel is the fallback for devices that cannot run the cluster kernel: built
    with the cluster kernel switched off, it is held to the same parity on the shapes the cluster
    kernel normally takes."""
    import subprocess
    import sys
    from pathlib import Path

    root = Path(__file__).resolve().parent.parent
    script = tmp_path / "register_variant.py"
    script.write_text(REGISTER_VARIANT)
    res = subprocess.run([sys.executable, str(script), str(root), str(tmp_path)], capture_output=True, text=True,
                         timeout=900)
    assert res.returncode == 0 and "register variant ok" in res.stdout, res.stdout[-2000:] + res.stderr[-2000:]


def test_map_refuses_bad_shapes(ccdc):
    plan = ccdc.Plan(4, 2, 12, 4, 128, "float32")
    z = torch.zeros(16, device="cuda")
    with pytest.raises(ccdc.CcdcError) as e:
        plan.map([z] * 4, [z] * 4, z, 24, [z] * 4, z)          # rows not a multiple of 16
    assert e.value.status == ccdc.ESIZE
    iplan = ccdc.Plan(4, 2, 12, 4, 128, "int32")
    with pytest.raises(ccdc.CcdcError) as e:
        iplan.map([z] * 4, [z] * 4, z, 32, [z] * 4, z)
    assert e.value.status == ccdc.ESTATE
    odd = ccdc.Plan(4, 2, 12, 4, 100, "float32")               # d = 400 is not a multiple of 512
    with pytest.raises(ccdc.CcdcError) as e:
        odd.map([z] * 4, [z] * 4, z, 32, [z] * 4, z)
    assert e.value.status == ccdc.ESIZE
