"""Host-side checks of the C-ABI library: it loads, exports what the header
declares, refuses what the paper's setting excludes, and its placement and
multicast schedule agree with the oracle's (written independently)."""
import ctypes
import re
from itertools import combinations
from math import comb
from pathlib import Path

import pytest

from oracle.ccdc_oracle import Oracle
from paper_1805_01993_b200 import build as ccdc_build
from paper_1805_01993_b200 import ccdc

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module", autouse=True)
def built():
    ccdc_build.build_library()


def declared_functions():
    text = (ROOT / "include" / "ccdc.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ccdc_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert len(names) >= 25
    handle = ctypes.CDLL(str(ccdc_build.LIB))
    for name in names:
        assert hasattr(handle, name), f"{name} declared in ccdc.h but not exported"
    assert sorted(ccdc.SIGNATURES) == names, "Python binding and header disagree"


def test_invalid_parameters():
    bad = [(1, 1, 4, 1, 4), (4, 0, 12, 4, 8), (4, 4, 12, 4, 8), (4, 2, 3, 4, 8), (4, 2, 13, 4, 8),
           (4, 2, 12, 6, 8), (4, 2, 12, 4, 0), (33, 2, 528, 33, 4)]
    for args in bad:
        with pytest.raises(ccdc.CcdcError) as e:
            ccdc.Plan(*args, "int32")
        assert e.value.status == ccdc.EINVAL
    with pytest.raises(ccdc.CcdcError):
        ccdc.Plan(4, 2, 7, 4, 8, "int32", jobs=True)
    with pytest.raises(ccdc.CcdcError) as e:
        ccdc.Plan(32, 15, comb(32, 15), 32, 8, "int32")       # schedule too large
    assert e.value.status == ccdc.ESIZE
    with pytest.raises(ccdc.CcdcError) as e:
        ccdc.Plan(20, 10, comb(20, 10), 20, 8, "int32")       # 5.9 GB of decode tables
    assert e.value.status == ccdc.ESIZE
    assert b"invalid" in ccdc.lib().ccdc_strerror(ccdc.EINVAL)
    assert ccdc.lib().ccdc_plan_num_groups(None) == 0


SHAPES = [(32, 1, 32, 32, 4), (32, 31, 32, 32, 4), (12, 6, 924, 12, 2), (3, 2, 6, 3, 8), (4, 2, 12, 4, 6), (4, 1, 8, 8, 3), (5, 3, 10, 10, 5), (5, 4, 5, 5, 2),
          (6, 3, 40, 6, 4), (7, 2, 21, 7, 9), (10, 3, 480, 10, 16)]


@pytest.mark.parametrize("K,r,N,Q,B", SHAPES)
def test_single_job_plan_matches_oracle_plan(K, r, N, Q, B):
    p = ccdc.Plan(K, r, N, Q, B, "float32")
    o = Oracle(K, r, N, Q, B, "float32")
    assert (p.J, p.num_batches, p.num_groups, p.files_per_batch) == (1, o.nbatch, o.nround, o.b)
    assert (p.packet_elems, p.segment_elems) == (o.len, o.s)
    assert p.coded_row_elems % 4 == 0 and 0 <= p.coded_row_elems - o.s < 4
    for b in range(o.nbatch):
        nodes, f0, job = p.batch(b)
        assert nodes == o.batch_nodes(b) and job == 0 and list(range(f0, f0 + o.b)) == o.batch_files(b)
        for n in o.batch_files(b):
            assert p.batch_of_file(n) == nodes
    for g in range(o.nround):
        assert p.group(g) == o.round_group(g) and p.group_batches(g) == o.round_batches(g)
    assert p.coded_bits == comb(K, r + 1) * (r + 1) * 32 * o.s
    for k in range(K):
        assert p.partition_bytes(k) == o.node_num_files(k) * Q * B * 4
        assert p.node_batches(k) == [b for b in range(o.nbatch) if k in o.batch_nodes(b)]
        assert p.packets_bytes(k) == o.node_num_batches(k) * (K - r) * o.len * 4
        assert p.decoded_bytes(k) == comb(K - 1, r) * o.len * 4
    assert p.coded_bytes == o.nround * (r + 1) * p.coded_row_elems * 4
    assert p.out_bytes == Q * B * 4


@pytest.mark.parametrize("K,r,N", [(4, 2, 6), (5, 2, 9), (5, 3, 8), (6, 1, 6), (6, 4, 10)])
def test_jobs_plan_matches_oracle_plan(K, r, N):
    Q, B = K, 6
    p = ccdc.Plan(K, r, N, Q, B, "int32", jobs=True)
    o = Oracle(K, r, N, Q, B, "int32", mode="paper")
    assert (p.J, p.num_batches, p.num_groups, p.files_per_batch) == (o.J, o.nbatch, o.nround, o.b)
    for b in range(o.nbatch):
        nodes, f0, job = p.batch(b)
        assert nodes == o.batch_nodes(b) and job == o.batch_job(b) and f0 == o.batch_files(b)[0]
    for g in range(o.nround):
        assert p.group(g) == o.round_group(g) and p.group_batches(g) == o.round_batches(g)
    # Theorem 1, from the library's own bit count (r | B here or padded: compare to s)
    assert p.coded_bits == o.nround * (r + 1) * 32 * o.s
    assert p.out_bytes == o.J * Q * B * 4


def test_expected_bits_of_the_five_workloads():
    expect = {(4, 2, 12, 4, 256): 49_152, (10, 3, 480, 10, 4096): 36_718_080,
              (16, 4, 1820, 16, 16384): 2_862_612_480, (20, 2, 190, 20, 1_280_000): 70_041_600_000,
              (8, 3, 112, 8, 1024): 3_064_320}
    for shape, bits in expect.items():
        assert ccdc.Plan(*shape, "float32").coded_bits == bits


def test_storage_and_replication():
    K, r, N, Q, B = 6, 3, 40, 6, 4
    p = ccdc.Plan(K, r, N, Q, B, "int32")
    seen = {}
    for k in range(K):
        files = p.node_files(k)
        assert len(files) * K == r * N
        for n in files:
            seen.setdefault(n, []).append(k)
    assert sorted(seen) == list(range(N))
    assert all(len(v) == r and v == p.batch_of_file(n) for n, v in seen.items())
    assert [p.batch(b)[0] for b in range(p.num_batches)] == [list(c) for c in combinations(range(K), r)]


@pytest.mark.parametrize("K,r,N", [(4, 2, 8), (6, 1, 12), (5, 2, 10), (8, 3, 16), (5, 4, 10), (20, 2, 190)])
def test_compression_plan(K, r, N):
    """Appendix placement: m = ceil(1/mu) batches, node k stores batch k mod m, at most
    mu*N files per node; unicast bit count = (ceil(1/mu)-1) * Q * T."""
    from fractions import Fraction

    Q, B = K, 8
    p = ccdc.Plan(K, r, N, Q, B, "float32", compression=True)
    m = -(-K // r)
    assert p.num_batches == m and p.num_groups == 0 and p.J == 1
    assert Fraction(p.coded_bits, Q * 32 * B) == m - 1
    seen = set()
    for k in range(K):
        files = p.node_files(k)
        assert len(files) * K <= r * N and p.partition_bytes(k) == len(files) * Q * B * 4
        assert p.node_batches(k) == [k % m]
        assert p.decoded_bytes(k) == (m - 1) * (Q // K) * B * 4
        for n in files:
            assert k in p.batch_of_file(n)
        seen.update(files)
    assert seen == set(range(N))
    assert p.coded_bytes == 0 and p.workspace_bytes == 0
    with pytest.raises(ccdc.CcdcError):
        ccdc.Plan(5, 2, 11, 5, 8, "float32", compression=True)      # mu*N not an integer


@pytest.mark.parametrize("K,r,N,world,jobs", [(4, 2, 12, 2, False), (6, 3, 40, 3, False), (8, 3, 112, 4, False),
                                              (4, 2, 6, 2, True), (6, 2, 9, 3, True)])
def test_node_sharded_plans_agree_on_the_gathered_layout(K, r, N, world, jobs):
    """Every rank's plan places coded row (round, a) at the same position of the
    gathered buffer; the rows a rank sends fill exactly its own slice, in order."""
    Q, B = K, 8
    plans = [ccdc.Plan(K, r, N, Q, B, "int32", jobs=jobs, shard=(rk, world)) for rk in range(world)]
    full = ccdc.Plan(K, r, N, Q, B, "int32", jobs=jobs)
    rows = full.num_groups * (r + 1)
    pos = [[pl.coded_row_position(g, a) for g in range(full.num_groups) for a in range(r + 1)] for pl in plans]
    assert all(p == pos[0] for p in pos) and sorted(pos[0]) == list(range(rows))
    per = rows // world
    for rk, pl in enumerate(plans):
        assert pl.coded_send_bytes == per * pl.coded_row_elems * 4 and pl.coded_bytes == full.coded_bytes
        mine = [pos[0][g * (r + 1) + a] for g in range(full.num_groups) for a, k in enumerate(full.group(g))
                if k // (K // world) == rk]
        assert mine == list(range(rk * per, (rk + 1) * per))
        assert [pl.node_is_local(k) for k in range(K)] == [k // (K // world) == rk for k in range(K)]
        assert pl.coded_bits == full.coded_bits        # what crosses between the GPUs is the multicast load
    with pytest.raises(ccdc.CcdcError):
        ccdc.Plan(6, 2, 15, 6, 8, "int32", shard=(0, 4))     # world must divide K


@pytest.mark.parametrize("K,r,N,gamma", [(4, 2, 6, 2), (5, 2, 9, 3), (5, 3, 8, 2)])
def test_gamma_groups_repeat_the_jobs_plan(K, r, N, gamma):
    """J = gamma * C(K, r+1) jobs: group g is the oracle's J-job plan with every batch, round,
    job and file id moved on by g groups; the multicast bits are gamma times one group's, so the
    load per J*Q*T is still Theorem 1."""
    from fractions import Fraction

    Q, B = K, 6
    p = ccdc.Plan(K, r, N, Q, B, "int32", jobs=True, gamma=gamma)
    o = Oracle(K, r, N, Q, B, "int32", mode="paper")
    assert (p.J, p.num_batches, p.num_groups, p.files_per_batch) == (gamma * o.J, gamma * o.nbatch, gamma * o.nround, o.b)
    for g in range(gamma):
        for b in range(o.nbatch):
            nodes, f0, job = p.batch(g * o.nbatch + b)
            assert nodes == o.batch_nodes(b) and job == g * o.J + o.batch_job(b)
            assert f0 == g * o.J * N + o.batch_files(b)[0]
        for rd in range(o.nround):
            assert p.group(g * o.nround + rd) == o.round_group(rd)
            assert p.group_batches(g * o.nround + rd) == [g * o.nbatch + x for x in o.round_batches(rd)]
    assert p.coded_bits == gamma * o.nround * (r + 1) * 32 * o.s
    assert Fraction(p.coded_bits, p.J * Q * 32 * B) == Fraction((K - r) * (r + 1), K * r) * Fraction(r * o.s, o.len)
    assert p.out_bytes == gamma * o.J * Q * B * 4
    for k in range(K):
        assert p.partition_bytes(k) == gamma * o.node_num_files(k) * Q * B * 4
    with pytest.raises(ccdc.CcdcError):
        ccdc.Plan(K, r, N, Q, B, "int32", jobs=True, gamma=0)
    with pytest.raises(ValueError):
        ccdc.Plan(K, r, comb(K, r), Q, B, "int32", gamma=2)


@pytest.mark.parametrize("K,r,Q,B,world", [(4, 2, 4, 16, 2), (6, 3, 12, 30, 5), (10, 2, 10, 64, 4), (5, 1, 5, 12, 3)])
def test_value_shards_partition_every_segment(K, r, Q, B, world):
    """Rank g owns sub-range g of every segment: the ranks' position maps are disjoint, cover the
    packet, keep a word inside its segment and at the same offset in every segment."""
    length = (Q // K) * B
    s = length // r
    w = s // world
    seen = []
    for rank in range(world):
        b_local = ccdc.value_shard(K, r, Q, B, rank, world)
        assert b_local * (Q // K) == r * w
        pos = [ccdc.value_shard_position(K, r, Q, B, rank, world, x) for x in range(r * w)]
        assert ccdc.value_shard_position(K, r, Q, B, rank, world, r * w) == -1
        for x, full in enumerate(pos):
            i, off = divmod(x, w)
            assert full // s == i and full % s == rank * w + off
        seen += pos
    assert sorted(seen) == list(range(length))
    for bad in ((K, r, Q, B + 1, 0, world), (K, r, Q, B, world, world), (K, r, Q, B, 0, 7 * s + 1)):
        with pytest.raises(ccdc.CcdcError) as e:
            ccdc.value_shard(*bad)
        assert e.value.status == ccdc.EINVAL


def test_decode_shape_queries_and_override():
    """The planner's launch shape of the fused decode, for the five workloads, and its override."""
    shapes = {(4, 2, 12, 4, 256): (128, 1), (16, 4, 1820, 16, 16384): (1024, 19), (20, 2, 190, 20, 1_280_000): (512, 1)}
    for shape, want in shapes.items():
        p = ccdc.Plan(*shape, "float32")
        assert (p.decode_threads, p.decode_chunks) == want, shape
        assert (p.workspace_bytes > 0) == (p.decode_chunks > 1) and not p.decode_cluster
    p = ccdc.Plan(10, 3, 480, 10, 4096, "float32")
    assert p.decode_threads == 128 and 1 < p.decode_chunks <= 8
    assert p.decode_cluster and p.workspace_bytes == 0      # the chunks meet in a thread-block cluster
    p.tune_decode(128, 6)
    assert p.decode_chunks == 6 and p.decode_cluster and p.workspace_bytes == 0
    p.tune_decode(128, 12)
    assert p.decode_chunks == 12 and not p.decode_cluster and p.workspace_bytes == 12 * 10 * 4096 * 4
    for threads, chunks in ((256, 6), (128, 0), (128, 121)):
        with pytest.raises(ccdc.CcdcError) as e:
            p.tune_decode(threads, chunks)
        assert e.value.status == ccdc.EINVAL
    assert ccdc.last_gather_kernel() == "" or "k_gather" in ccdc.last_gather_kernel()


def test_bench_byte_counts_agree_with_the_plan():
    """The benchmark's algorithmic byte counts against the plan's own sizes, and its DRAM-traffic
    table: an entry applies only to the kernel sources it was measured on and scales with B."""
    import sys

    sys.path.insert(0, str(ROOT))
    import bench
    from paper_1805_01993_b200.inputs import CONFIGS

    for name in ("cfg1", "cfg2", "cfg3", "cfg4", "cfg5"):
        w = CONFIGS[name]
        p = ccdc.Plan(w.K, w.r, w.N, w.Q, w.B, w.dtype)
        by = bench.algorithmic_bytes(w.K, w.r, w.N, w.Q, w.B)
        assert by["coded_write"] * 8 == p.coded_bits
        stored = sum(p.partition_bytes(k) for k in range(w.K))
        assert stored == w.r * w.N * w.Q * w.B * 4
        # every node reads, of every stored file, its own function's value and the K-r outside nodes' values
        assert by["iv_read"] == stored // w.Q * (w.Q // w.K) * (w.K - w.r + 1)
        assert by["total"] == by["encode_kernel"] + by["decode_kernel"]
    w = CONFIGS["jobs20"]
    p = ccdc.Plan(w.K, w.r, w.N, w.Q, w.B, w.dtype, jobs=True)
    by = bench.algorithmic_bytes(w.K, w.r, w.N, w.Q, w.B, J=p.J, rounds=p.num_groups)
    assert by["coded_write"] * 8 == p.coded_bits
    assert bench.measured_traffic(CONFIGS["cfg1"], "k_decode_reduce") == (None, None)
    full, kind = bench.measured_traffic(CONFIGS["cfg4"], "k_decode_reduce")
    if full is not None:                                    # the table matches the current kernel sources
        half, _ = bench.measured_traffic(CONFIGS["cfg4"].scaled(640000), "k_decode_reduce")
        assert "scaled" in kind and half == pytest.approx(full / 2)
        assert 0.8 < full / by_of("cfg4")["decode_kernel"] < 1.1
        assert bench.measured_traffic(CONFIGS["cfg4"], "k_gather(encode)") == (None, None)


def by_of(name):
    import bench
    from paper_1805_01993_b200.inputs import CONFIGS

    w = CONFIGS[name]
    return bench.algorithmic_bytes(w.K, w.r, w.N, w.Q, w.B)
