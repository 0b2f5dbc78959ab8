"""Parity of the CUDA path with the CPU oracle, through the C ABI.

Same seeded inputs on both sides.  int32: every packet, coded word, decoded word
and output bit-exact.  fp32: coded packets bit-exact (the pre-combining order is
fixed: files ascending, starting from the first file's value); outputs within
1e-5 * sum_n |v_{q,n}| element-wise, the tolerance the method's evaluation
states, since the fused path may add the per-batch terms in another grouping.
"""
from math import comb

import numpy as np
import pytest

from oracle.ccdc_oracle import Oracle
from paper_1805_01993_b200.inputs import CONFIGS, values_numpy, values_torch

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

FP32_RTOL = 1e-5
CANARY = 0x5A5A5A5A


@pytest.fixture(scope="module")
def ccdc():
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    from paper_1805_01993_b200 import build, ccdc as mod

    build.build_library()
    mod.lib()
    return mod


def guarded(n_words, dtype, pad=64):
    """tensor of n words with canary words on both sides; returns (whole, view)."""
    whole = torch.full((n_words + 2 * pad,), CANARY, dtype=torch.int32, device="cuda")
    return whole, whole[pad:pad + n_words].view(dtype)


def canaries_intact(whole, n_words, pad=64):
    w = whole.cpu().numpy().view(np.uint32)
    return bool((w[:pad] == CANARY).all() and (w[pad + n_words:] == CANARY).all())


def bits(t):
    return t.detach().cpu().contiguous().numpy().view(np.uint32)


def assert_outputs(out_gpu, o, dtype):
    ref = o.reduce()
    got = out_gpu.cpu().numpy().reshape(ref.shape)
    if dtype == "int32":
        assert np.array_equal(got, ref)
        assert np.array_equal(got, o.direct())
        return
    s64, a64 = o.direct()
    err = np.abs(got.astype(np.float64) - ref.astype(np.float64))
    assert np.all(err <= FP32_RTOL * a64 + 1e-30), float((err / (a64 + 1e-30)).max())
    assert np.all(np.abs(got - s64) <= FP32_RTOL * a64 + 1e-30)


def run_case(ccdc, K, r, N, Q, B, dtype, jobs=False, seed=1, std=1.0, tune=None, family=None):
    plan = ccdc.Plan(K, r, N, Q, B, dtype, jobs=jobs)
    if family is not None:
        plan.tune_family(family)
    if tune:
        plan.tune_decode(*tune)
    o = Oracle(K, r, N, Q, B, dtype, mode="paper" if jobs else "single")
    v = values_numpy(plan.J * N, Q, B, dtype, seed=seed, std=std)
    o.load_values(v)
    o.shuffle()
    tdt = plan.torch_dtype
    part = plan.alloc_partitions()
    plan.fill_partitions(part, torch.from_numpy(v).cuda())
    s, sp, L = plan.segment_elems, plan.coded_row_elems, plan.packet_elems
    rows = plan.num_groups * (r + 1)
    ref_coded = o.coded().reshape(rows, s)

    # ---- stepwise path -------------------------------------------------
    packets = plan.alloc_packets()
    decoded = plan.alloc_decoded()
    coded_w, coded = guarded(rows * sp, tdt)
    out_w, out = guarded(plan.J * Q * B, tdt)
    plan.combine(part, packets)
    plan.encode(packets, coded)
    plan.decode(packets, coded, decoded)
    plan.reduce(part, decoded, out)
    torch.cuda.synchronize()
    for k in range(K):
        assert np.array_equal(bits(packets[k]).reshape(-1, L), o.packets(k)), f"packets of node {k}"
        assert np.array_equal(bits(decoded[k]).reshape(-1, L), o.decoded(k)), f"decoded of node {k}"
    assert np.array_equal(bits(coded).reshape(rows, sp)[:, :s], ref_coded)
    assert canaries_intact(coded_w, rows * sp) and canaries_intact(out_w, plan.J * Q * B)
    assert_outputs(out, o, dtype)
    # the stepwise reduce adds the batches in the oracle's order: same bits
    assert np.array_equal(bits(out).reshape(-1, B), o.reduce().view(np.uint32))

    # ---- fused path ------------------------------------------------------
    coded_w2, coded2 = guarded(rows * sp, tdt)
    out_w2, out2 = guarded(plan.J * Q * B, tdt)
    ws_words = plan.workspace_bytes // 4
    ws_w, ws = guarded(ws_words, tdt)
    plan.shuffle(part, coded2, out2, ws if ws_words else None)
    torch.cuda.synchronize()
    assert np.array_equal(bits(coded2).reshape(rows, sp)[:, :s], ref_coded)
    assert canaries_intact(coded_w2, rows * sp) and canaries_intact(out_w2, plan.J * Q * B)
    assert canaries_intact(ws_w, ws_words)
    assert_outputs(out2, o, dtype)
    if plan.decode_chunks == 1:          # the batch loop is not split: the oracle's order of additions
        assert np.array_equal(bits(out2).reshape(-1, B), o.reduce().view(np.uint32))
    assert plan.coded_bits == o.coded_bits
    plan.shuffle_status()
    return plan


# K, r, N, Q, B: r = 1, r = K-1, several files per batch, Q/K > 1, r does not
# divide the packet, B < r, vector widths 1 / 2 / 4, several tiles + ragged tail
SHAPES = [
    (3, 2, 6, 3, 8),
    (3, 1, 3, 3, 5),
    (4, 2, 12, 4, 6),
    (4, 3, 8, 4, 9),
    (4, 1, 8, 8, 3),
    (5, 2, 20, 5, 7),
    (5, 3, 10, 10, 5),
    (5, 4, 5, 5, 2),
    (6, 3, 40, 6, 4),
    (6, 2, 15, 12, 3),
    (4, 2, 12, 4, 2 * (3 * 2048 + 20)),     # vec 4, 4 tiles per segment, ragged tail
    (5, 3, 20, 5, 3 * (2 * 1024 + 6)),      # vec 2
    (5, 3, 10, 5, 3 * 2049 + 1),            # vec 1, r does not divide B
    (6, 5, 12, 6, 7001),                    # r = K-1, one round
    (7, 3, 35, 14, 1000),                   # Q/K = 2
    (32, 1, 32, 32, 40),                    # the largest K, r = 1
    (32, 31, 32, 32, 70),                   # the largest K, r = K-1: one round of 32 members
    (12, 6, 924, 12, 8),                    # 924 batches, 792 rounds of 7
    (9, 5, 252, 9, 1030),                   # r = 5: general (run-time r) decode path, b = 2
    (6, 2, 15, 6, 40000),                   # b = 1, long values: lean gather + deep-load decode
    (4, 2, 54, 4, 1100),                    # b = 9: batch sums in groups of four files plus a remainder
    (3, 1, 30, 3, 2100),                    # b = 10, r = 1: one operand, eight files' loads in flight
    (5, 3, 50, 5, 777),                     # b = 5, three operands
    (5, 4, 15, 5, 1300),                    # b = 3, four operands
    (6, 2, 15, 6, 65544),                   # b = 1, segments of 32 772 words: the 512-thread form of the fused encode
    (4, 2, 6, 8, 6 * 1366 + 2),             # Q/K = 2, b = 1, ragged
    (6, 2, 105, 6, 3000),                   # b = 7: two groups of files per operand (4 + 3)
    (5, 1, 45, 5, 2200),                    # b = 9, r = 1: three groups, no cancel operand
]


@pytest.mark.parametrize("dtype", ["int32", "float32"])
@pytest.mark.parametrize("K,r,N,Q,B", SHAPES)
def test_single_job_matches_oracle(ccdc, K, r, N, Q, B, dtype):
    run_case(ccdc, K, r, N, Q, B, dtype, seed=K * 10 + r)


@pytest.mark.parametrize("dtype", ["int32", "float32"])
@pytest.mark.parametrize("K,r,N,Q,B", [(4, 2, 6, 4, 8), (5, 2, 9, 5, 37), (5, 3, 8, 10, 6), (6, 1, 6, 6, 5),
                                       (6, 4, 10, 6, 4100), (5, 2, 21, 5, 2060)])     # the last: 7 files per batch
def test_jobs_plan_matches_oracle(ccdc, K, r, N, Q, B, dtype):
    """The scheme as stated for J = C(K, r+1) jobs (stages 1 and 2)."""
    run_case(ccdc, K, r, N, Q, B, dtype, jobs=True, seed=3)


def bulk_copy_family_serves(K, r, N, Q, B):
    length = (Q // K) * B
    return length % 4 == 0 and (-(-length // r)) % 2 == 0


@pytest.mark.parametrize("dtype", ["int32", "float32"])
@pytest.mark.parametrize("K,r,N,Q,B", SHAPES + [(10, 3, 480, 10, 4096), (8, 3, 112, 8, 1024), (4, 2, 12, 4, 256),
                                               (6, 2, 15, 6, 4 * 2048 + 2), (5, 3, 10, 5, 3 * 4098)])
def test_bulk_copy_family_matches_oracle(ccdc, K, r, N, Q, B, dtype):
    """The fused encode and decode as bulk-copy pipelines (kernel family 1): same coded words, same
    outputs; shapes the family cannot serve (rows not 16-byte aligned, odd segments) are refused."""
    if not bulk_copy_family_serves(K, r, N, Q, B):
        with pytest.raises(ccdc.CcdcError) as e:
            ccdc.Plan(K, r, N, Q, B, dtype).tune_family(1)
        assert e.value.status == ccdc.ESIZE
        return
    plan = run_case(ccdc, K, r, N, Q, B, dtype, seed=K + r, family=1)
    assert plan.kernel_family == 1
    assert "k_stream<encode" in ccdc.last_gather_kernel() and "k_stream<decode" in ccdc.last_decode_kernel()


@pytest.mark.parametrize("dtype", ["int32", "float32"])
@pytest.mark.parametrize("K,r,N,Q,B", [(4, 2, 6, 4, 8), (5, 2, 9, 5, 36), (6, 4, 10, 6, 4104), (5, 2, 21, 5, 2060)])
def test_bulk_copy_family_on_the_jobs_plan(ccdc, K, r, N, Q, B, dtype):
    plan = run_case(ccdc, K, r, N, Q, B, dtype, jobs=True, seed=5, family=1)
    assert "k_stream<decode" in ccdc.last_decode_kernel()


def test_cfg1_full(ccdc):
    w = CONFIGS["cfg1"]
    plan = run_case(ccdc, w.K, w.r, w.N, w.Q, w.B, w.dtype)
    assert plan.coded_bits == 49_152


def test_cfg2_full(ccdc):
    w = CONFIGS["cfg2"]
    plan = run_case(ccdc, w.K, w.r, w.N, w.Q, w.B, w.dtype)
    assert plan.coded_bits == 36_718_080 and plan.decode_chunks > 1 and plan.decode_cluster
    assert "cluster" in ccdc.last_decode_kernel()


def test_cfg3_short_values(ccdc):
    w = CONFIGS["cfg3"].scaled(512)
    plan = run_case(ccdc, w.K, w.r, w.N, w.Q, w.B, w.dtype)
    assert plan.workspace_bytes > 0


def test_cfg4_short_values(ccdc):
    w = CONFIGS["cfg4"].scaled(6000)
    run_case(ccdc, w.K, w.r, w.N, w.Q, w.B, w.dtype, std=w.std)


def test_cfg3_structure_exhaustive_1024_thread_decode(ccdc):
    """K=16, r=4, N=1820, Q=16 with values of 8208 elements: segments of 2052 words select the
    1024-thread block of the fused decode, the launch shape of the full-size workload; every coded
    word, packet and output against the oracle."""
    w = CONFIGS["cfg3"].scaled(8208)
    plan = run_case(ccdc, w.K, w.r, w.N, w.Q, w.B, w.dtype)
    assert plan.decode_threads == 1024 and plan.decode_chunks > 1
    assert "threads=1024" in ccdc.last_decode_kernel() and "cancel=3" in ccdc.last_decode_kernel()
    full = ccdc.Plan(w.K, w.r, w.N, w.Q, CONFIGS["cfg3"].B, w.dtype)
    assert (full.decode_threads, full.decode_chunks) == (plan.decode_threads, plan.decode_chunks)


def test_cfg4_structure_exhaustive_wide_encode(ccdc):
    """K=20, r=2, N=190, Q=20 with values of 65 544 elements: one-file rows of 32 772 words select the
    512-thread form of the fused encode with several tiles per block and a ragged last tile, the
    launch shape of the full-size workload; every coded word, packet and output against the oracle."""
    w = CONFIGS["cfg4"].scaled(65544)
    full = ccdc.Plan(w.K, w.r, w.N, w.Q, CONFIGS["cfg4"].B, w.dtype)
    assert (full.decode_threads, full.decode_chunks) == (512, 1)
    plan = run_case(ccdc, w.K, w.r, w.N, w.Q, w.B, w.dtype, std=w.std, tune=(512, 1))   # the full size's decode shape
    assert "operands=2,files=1,vectors=2,threads=512" in ccdc.last_gather_kernel()
    assert "threads=512,cancel=1,files=1,chunks=1" in ccdc.last_decode_kernel()


def test_cfg5_shuffle_shape(ccdc):
    w = CONFIGS["cfg5"]
    plan = run_case(ccdc, w.K, w.r, w.N, w.Q, w.B, w.dtype)
    assert plan.coded_bits == 3_064_320


@pytest.mark.parametrize("chunks", [4, 12])
def test_shuffle_replayed_from_a_cuda_graph(ccdc, chunks):
    """The two launches of ccdc_shuffle (plus the final pass of a split loop) captured in a CUDA graph and
    replayed on new inputs give the oracle's coded packets and outputs: small jobs are launch-bound and
    are meant to be run this way."""
    K, r, N, Q, B, dtype = 10, 3, 480, 10, 96, "float32"          # the K = 10 structure, short values, split loop
    plan = ccdc.Plan(K, r, N, Q, B, dtype)
    plan.tune_decode(plan.decode_threads, chunks)
    if chunks > 8:
        assert plan.workspace_bytes > 0                            # three launches: encode, decode, sum of the partial sums
    else:
        assert plan.decode_cluster and plan.workspace_bytes == 0   # two launches, the second one clustered
    part = plan.alloc_partitions()
    coded, out, ws = plan.alloc(plan.coded_bytes), plan.alloc(plan.out_bytes), plan.alloc(plan.workspace_bytes)
    v0 = values_numpy(N, Q, B, dtype, seed=31)
    plan.fill_partitions(part, torch.from_numpy(v0).cuda())
    plan.shuffle(part, coded, out, ws)                            # tables uploaded, attributes set
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            plan.shuffle(part, coded, out, ws)
    torch.cuda.current_stream().wait_stream(side)
    s, sp = plan.segment_elems, plan.coded_row_elems
    for seed in (32, 33):
        v = values_numpy(N, Q, B, dtype, seed=seed)
        plan.fill_partitions(part, torch.from_numpy(v).cuda())
        coded.zero_(); out.zero_()
        graph.replay()
        torch.cuda.synchronize()
        o = Oracle(K, r, N, Q, B, dtype)
        o.load_values(v)
        o.shuffle()
        assert np.array_equal(bits(coded).reshape(-1, sp)[:, :s], o.coded().reshape(-1, s))
        assert_outputs(out, o, dtype)


def test_special_float_patterns_survive_coding(ccdc):
    """-0.0, infinities and NaN payloads are carried bit for bit when b = 1."""
    K, r, N, Q, B = 4, 2, 6, 4, 8
    v = values_numpy(N, Q, B, "float32", seed=2)
    v.view(np.uint32)[0, 3, 0] = 0x80000000
    v.view(np.uint32)[1, 2, 1] = 0x7F800000
    v.view(np.uint32)[2, 0, 2] = 0x7FC12345
    plan = ccdc.Plan(K, r, N, Q, B, "float32")
    o = Oracle(K, r, N, Q, B, "float32")
    o.load_values(v)
    o.shuffle()
    part = plan.alloc_partitions()
    plan.fill_partitions(part, torch.from_numpy(v).cuda())
    coded = plan.alloc(plan.coded_bytes)
    out = plan.alloc(plan.out_bytes)
    plan.shuffle(part, coded, out, None)
    packets, decoded = plan.alloc_packets(), plan.alloc_decoded()
    plan.combine(part, packets)
    plan.decode(packets, coded, decoded)
    torch.cuda.synchronize()
    assert np.array_equal(bits(coded).reshape(-1, plan.coded_row_elems)[:, :plan.segment_elems],
                          o.coded().reshape(-1, plan.segment_elems))
    for k in range(K):
        assert np.array_equal(bits(decoded[k]).reshape(-1, B), o.decoded(k))


@pytest.mark.parametrize("dtype", ["int32", "float32"])
@pytest.mark.parametrize("K,r,N,Q,B", [(4, 2, 8, 4, 64), (6, 1, 12, 12, 33), (5, 2, 10, 5, 2 * 2048 + 12),
                                       (8, 3, 16, 8, 1000), (5, 4, 10, 5, 7), (10, 2, 50, 10, 4096)])
def test_compression_only_matches_oracle(ccdc, K, r, N, Q, B, dtype):
    """The appendix's compression-only shuffle (comparator): every unicast packet and
    every output bit-exact (same addition order on both sides), bits = ceil(1/mu)-1."""
    from oracle.ccdc_oracle import compression_only

    v = values_numpy(N, Q, B, dtype, seed=K + r)
    ref_out, ref_recv, ref_bits, files = compression_only(K, r, N, Q, B, dtype, v)
    plan = ccdc.Plan(K, r, N, Q, B, dtype, compression=True)
    assert plan.coded_bits == ref_bits
    assert [len(plan.node_files(k)) for k in range(K)] == files
    part = plan.alloc_partitions()
    plan.fill_partitions(part, torch.from_numpy(v).cuda())
    recv = plan.alloc_decoded()
    out_w, out = guarded(Q * B, plan.torch_dtype)
    plan.compression_shuffle(part, recv, out)
    torch.cuda.synchronize()
    for k in range(K):
        assert np.array_equal(bits(recv[k]).reshape(ref_recv.shape[1], -1), ref_recv[k])
    assert np.array_equal(bits(out).reshape(Q, B), ref_out.view(np.uint32))
    assert canaries_intact(out_w, Q * B)
    # the coded steps refuse such a plan
    with pytest.raises(ccdc.CcdcError) as e:
        plan.encode_fused(part, out)
    assert e.value.status == ccdc.ESTATE
    with pytest.raises(ccdc.CcdcError) as e:
        ccdc.Plan(K, r, comb(K, r) * 2, Q, B, dtype).compression_shuffle(part, recv, out)
    assert e.value.status == ccdc.ESTATE


@pytest.mark.parametrize("dtype", ["int32", "float32"])
@pytest.mark.parametrize("K,r,N,Q,B,world,jobs", [(4, 2, 12, 4, 300, 2, False), (6, 3, 40, 6, 2049, 3, False),
                                                  (8, 3, 112, 8, 1024, 4, False), (10, 3, 480, 10, 512, 2, False),
                                                  (4, 2, 6, 4, 100, 2, True), (6, 2, 9, 12, 64, 3, True)])
def test_node_sharded_ranks_emulated_on_one_gpu(ccdc, K, r, N, Q, B, world, jobs, dtype):
    """K/world logical nodes per GPU: every rank encodes the coded rows its nodes send,
    the send buffers are gathered rank-major (here a concatenation stands in for the
    all-gather; the ranks run one after the other, none waits for another), and every
    rank decodes for its own nodes.  Coded rows and outputs against the oracle."""
    full = ccdc.Plan(K, r, N, Q, B, dtype, jobs=jobs)
    o = Oracle(K, r, N, Q, B, dtype, mode="paper" if jobs else "single")
    v = values_numpy(full.J * N, Q, B, dtype, seed=K + world)
    o.load_values(v)
    o.shuffle()
    vt = torch.from_numpy(v).cuda()
    plans = [ccdc.Plan(K, r, N, Q, B, dtype, jobs=jobs, shard=(rk, world)) for rk in range(world)]
    parts, sends = [], []
    for pl in plans:
        part = pl.alloc_partitions()
        pl.fill_partitions(part, vt)
        send_w, send = guarded(pl.coded_send_bytes // 4, pl.torch_dtype)
        pl.encode_fused(part, send)
        torch.cuda.synchronize()
        assert canaries_intact(send_w, pl.coded_send_bytes // 4)
        parts.append(part); sends.append(send)
    coded = torch.cat(sends)                                  # the all-gather
    assert coded.numel() * 4 == full.coded_bytes
    s, sp = full.segment_elems, full.coded_row_elems
    got = bits(coded).reshape(-1, sp)[:, :s]
    ref = o.coded().reshape(-1, s)
    order = [plans[0].coded_row_position(g, a) for g in range(full.num_groups) for a in range(r + 1)]
    assert np.array_equal(got[order], ref)
    out = torch.full((full.J * Q * B,), 7, dtype=full.torch_dtype, device="cuda")
    for pl, part in zip(plans, parts):
        ws = pl.alloc(pl.workspace_bytes)
        pl.decode_reduce(part, coded, out, ws)
    torch.cuda.synchronize()
    assert_outputs(out, o, dtype)
    with pytest.raises(ccdc.CcdcError) as e:
        plans[0].shuffle(parts[0], coded, out, None)
    assert e.value.status == ccdc.ESTATE
    # the encode that stores straight into every rank's buffer (here: `world` buffers on one GPU)
    if r <= 4:
        guards = [guarded(full.coded_bytes // 4, full.torch_dtype) for _ in range(world)]
        peers = [gview for _, gview in guards]
        for pl, part in zip(plans, parts):
            pl.encode_fused_peers(part, peers)
        torch.cuda.synchronize()                              # stands in for the ranks' synchronisation
        for whole, gview in guards:
            assert canaries_intact(whole, full.coded_bytes // 4)
            assert np.array_equal(bits(gview).reshape(-1, sp)[:, :s], got)
        out2 = torch.full_like(out, 7)
        for rk, (pl, part) in enumerate(zip(plans, parts)):
            pl.decode_reduce(part, peers[rk], out2, pl.alloc(pl.workspace_bytes))
        torch.cuda.synchronize()
        assert torch.equal(out2, out)


def test_bad_arguments_are_refused(ccdc):
    plan = ccdc.Plan(4, 2, 12, 4, 64, "int32")
    part = plan.alloc_partitions()
    coded = plan.alloc(plan.coded_bytes)
    out = plan.alloc(plan.out_bytes)
    before = ccdc.num_kernel_launches()
    with pytest.raises(ccdc.CcdcError) as e:
        plan.shuffle(part[:3] + [None], coded, out, None)
    assert e.value.status == ccdc.EINVAL
    with pytest.raises(ccdc.CcdcError):
        plan.shuffle(part, coded[1:], out, None)            # misaligned
    bigplan = ccdc.Plan(10, 3, 480, 10, 64, "int32")
    bigplan.tune_decode(bigplan.decode_threads, 12)
    assert bigplan.workspace_bytes > 0
    bp = bigplan.alloc_partitions()
    with pytest.raises(ccdc.CcdcError):
        bigplan.shuffle(bp, bigplan.alloc(bigplan.coded_bytes), bigplan.alloc(bigplan.out_bytes), None)
    assert ccdc.num_kernel_launches() == before
    plan.shuffle(part, coded, out, None)
    torch.cuda.synchronize()
    assert ccdc.num_kernel_launches() == before + 2


def sampled_full_size_check(ccdc, w, offsets_per_segment=48, seed=5):
    """Full-size run in the benchmark's launch configuration, compared with the
    oracle on a sub-problem: the same element offsets inside every segment form
    an exact instance of the scheme with a shorter value (every step acts
    element-wise along a segment), so the oracle can produce those coded words
    and outputs one by one.  Requires r | B and Q = K."""
    assert w.Q == w.K and w.B % w.r == 0
    plan = ccdc.Plan(w.K, w.r, w.N, w.Q, w.B, w.dtype)
    s = plan.segment_elems
    rng = np.random.default_rng(seed)
    # first and last word of a tile and of a block's span for every tile the two launches use at these
    # shapes (the fused encode: 256 or 512 threads x 4 words x 2 vectors, 32 tiles per block; the fused
    # decode: 512 or 1024 threads x 4 words), and of the ragged last tile and span
    fixed = [0, 1, 3, s - 1, s - 4, s // 2]
    for tile in (2048, 4096):
        span = 32 * tile
        for edge in (tile, 2 * tile, span, (s - 1) // tile * tile, (s - 1) // span * span):
            fixed += [edge - 1, edge]
    fixed = [x for x in fixed if 0 <= x < s]
    offs = np.unique(np.concatenate([np.array(fixed), rng.integers(0, s, offsets_per_segment)]))
    m = len(offs)
    index = np.concatenate([i * s + offs for i in range(w.r)])
    idx_t = torch.from_numpy(index).cuda()

    part = plan.alloc_partitions()
    sampled = plan.fill_partitions_streaming(
        part, values_torch(w.N, w.Q, w.B, w.dtype, "cuda", seed=seed, std=w.std), idx_t)
    coded = plan.alloc(plan.coded_bytes)
    out = plan.alloc(plan.out_bytes)
    ws = plan.alloc(plan.workspace_bytes) if plan.workspace_bytes else None
    plan.shuffle(part, coded, out, ws)
    torch.cuda.synchronize()

    o = Oracle(w.K, w.r, w.N, w.Q, w.r * m, w.dtype)
    o.load_values(sampled.numpy())
    o.shuffle()
    assert o.s == m
    rows = plan.num_groups * (w.r + 1)
    got_coded = coded.view(rows, plan.coded_row_elems).index_select(1, torch.from_numpy(offs).cuda())
    assert np.array_equal(bits(got_coded), o.coded().reshape(rows, m))
    got_out = out.view(w.Q, w.B).index_select(1, idx_t).cpu().numpy()
    ref = o.reduce()
    s64, a64 = o.direct()
    err = np.abs(got_out.astype(np.float64) - ref.astype(np.float64))
    assert np.all(err <= FP32_RTOL * a64 + 1e-30)
    assert np.all(np.abs(got_out - s64) <= FP32_RTOL * a64 + 1e-30)
    del part, coded, ws
    return plan


def test_cfg3_full_size_sampled(ccdc):
    plan = sampled_full_size_check(ccdc, CONFIGS["cfg3"])
    assert "threads=1024" in ccdc.last_decode_kernel()
    assert plan.coded_bits == 2_862_612_480


def test_cfg4_full_size_sampled(ccdc):
    free, _ = torch.cuda.mem_get_info()
    if free < 60 * 2**30:
        pytest.fail("cfg4 needs about 50 GB of device memory")
    plan = sampled_full_size_check(ccdc, CONFIGS["cfg4"], offsets_per_segment=24)
    assert "threads=512" in ccdc.last_gather_kernel() and "threads=512" in ccdc.last_decode_kernel()
    assert plan.coded_bits == 70_041_600_000


@pytest.mark.parametrize("dtype", ["int32", "float32"])
@pytest.mark.parametrize("K,r,N,Q,B", [(4, 2, 12, 4, 300), (10, 3, 480, 10, 96), (6, 3, 20, 12, 2049)])
def test_shuffle_from_host_buffers(ccdc, K, r, N, Q, B, dtype):
    """ccdc_shuffle_host: Map results in pinned host memory, outputs back in host memory, copies and
    the two launches on one stream; outputs and the coded rows left on the device against the oracle."""
    plan = ccdc.Plan(K, r, N, Q, B, dtype)
    o = Oracle(K, r, N, Q, B, dtype)
    v = values_numpy(N, Q, B, dtype, seed=77)
    o.load_values(v)
    o.shuffle()
    row = Q * B
    host_part = []
    for k in range(K):
        files = plan.node_files(k)
        h = torch.empty(len(files) * row, dtype=plan.torch_dtype).pin_memory()
        h.view(-1, row).copy_(torch.from_numpy(v.reshape(N, row)[files]))
        host_part.append(h)
    host_out = torch.full((Q * B,), 7, dtype=plan.torch_dtype).pin_memory()
    part = plan.alloc_partitions()
    coded_w, coded = guarded(plan.coded_bytes // 4, plan.torch_dtype)
    out_w, out = guarded(Q * B, plan.torch_dtype)
    ws = plan.alloc(plan.workspace_bytes)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for _ in range(2):          # the second call finds the first one's data everywhere
            plan.shuffle_host(host_part, host_out, part, coded, out, ws if ws.numel() else None, stream=stream)
    stream.synchronize()
    s, sp = plan.segment_elems, plan.coded_row_elems
    assert np.array_equal(bits(coded).reshape(-1, sp)[:, :s], o.coded().reshape(-1, s))
    assert canaries_intact(coded_w, plan.coded_bytes // 4) and canaries_intact(out_w, Q * B)
    assert_outputs(host_out, o, dtype)
    assert torch.equal(host_out, out.cpu())
    for k in range(K):
        assert torch.equal(part[k].cpu(), host_part[k])


@pytest.mark.parametrize("dtype", ["int32", "float32"])
@pytest.mark.parametrize("K,r,N,Q,B,jobs", [(4, 2, 12, 4, 300, False), (6, 3, 20, 12, 2049, False), (5, 2, 9, 5, 64, True)])
def test_shuffle_from_host_files(ccdc, K, r, N, Q, B, jobs, dtype):
    """ccdc_shuffle_host_files: every file in host memory once; the library places the r replicas
    (one host-to-device copy per file, device-to-device for the other holders) and shuffles."""
    plan = ccdc.Plan(K, r, N, Q, B, dtype, jobs=jobs)
    o = Oracle(K, r, N, Q, B, dtype, mode="paper" if jobs else "single")
    v = values_numpy(plan.J * N, Q, B, dtype, seed=78)
    o.load_values(v)
    o.shuffle()
    host_values = torch.from_numpy(v).pin_memory()
    host_out = torch.full((plan.J * Q * B,), 7, dtype=plan.torch_dtype).pin_memory()
    part = plan.alloc_partitions()
    for p_ in part:
        p_.fill_(3)
    coded, out = plan.alloc(plan.coded_bytes), plan.alloc(plan.out_bytes)
    ws = plan.alloc(plan.workspace_bytes)
    plan.shuffle_host_files(host_values, host_out, part, coded, out, ws if ws.numel() else None)
    torch.cuda.synchronize()
    ref_part = plan.alloc_partitions()
    plan.fill_partitions(ref_part, torch.from_numpy(v).cuda())
    for k in range(K):
        assert torch.equal(part[k], ref_part[k]), f"partition of node {k}"
    s, sp = plan.segment_elems, plan.coded_row_elems
    assert np.array_equal(bits(coded).reshape(-1, sp)[:, :s], o.coded().reshape(-1, s))
    assert_outputs(host_out, o, dtype)


@pytest.mark.parametrize("K,r,N,Q,B,jobs", [(5, 2, 10, 5, 1000, False), (10, 3, 480, 10, 64, False),
                                            (4, 2, 12, 8, 37, False), (5, 2, 9, 5, 50, True)])
def test_words_written_by_the_encode_are_the_multicast_bits(ccdc, K, r, N, Q, B, jobs):
    """Definition 1 counted on the device: the coded buffer starts full of a word no coded word can
    equal (Map values below 2**20, so every sum and XOR stays below 2**31; the mark has bit 31 set);
    after the fused encode the words that changed, times 32, are the plan's multicast bit count."""
    plan = ccdc.Plan(K, r, N, Q, B, "int32", jobs=jobs)
    v = (values_numpy(plan.J * N, Q, B, "int32", seed=9).view(np.uint32) >> 12).view(np.int32)
    part = plan.alloc_partitions()
    plan.fill_partitions(part, torch.from_numpy(v).cuda())
    mark = -0x7A5A5A5B      # bit 31 set
    coded = torch.full((plan.coded_bytes // 4,), mark, dtype=torch.int32, device="cuda")
    plan.encode_fused(part, coded)
    torch.cuda.synchronize()
    written = int((coded != mark).sum().item())
    assert written * 32 == plan.coded_bits
    o = Oracle(K, r, N, Q, B, "int32", mode="paper" if jobs else "single")
    o.load_values(v)
    o.shuffle()
    assert written * 32 == o.coded_bits


@pytest.mark.parametrize("dtype", ["int32", "float32"])
def test_decode_shape_overrides_keep_parity(ccdc, dtype):
    """ccdc_plan_tune_decode: every allowed launch shape of the fused decode gives the oracle's outputs."""
    for (K, r, N, Q, B), shapes in (((10, 3, 480, 10, 96), [(128, c) for c in (1, 2, 7, 15, 120)]),
                                    ((6, 2, 15, 6, 9000), [(512, 1), (512, 3), (1024, 2), (1024, 15)])):
        o = Oracle(K, r, N, Q, B, dtype)
        v = values_numpy(N, Q, B, dtype, seed=K)
        o.load_values(v)
        o.shuffle()
        for threads, chunks in shapes:
            plan = ccdc.Plan(K, r, N, Q, B, dtype)
            plan.tune_decode(threads, chunks)
            assert (plan.decode_threads, plan.decode_chunks) == (threads, chunks)
            part = plan.alloc_partitions()
            plan.fill_partitions(part, torch.from_numpy(v).cuda())
            coded = plan.alloc(plan.coded_bytes)
            out_w, out = guarded(Q * B, plan.torch_dtype)
            ws_w, ws = guarded(plan.workspace_bytes // 4, plan.torch_dtype)
            assert (plan.workspace_bytes > 0) == (chunks > 1 and not plan.decode_cluster)
            assert plan.decode_cluster == (threads == 128 and 2 <= chunks <= 8)
            for _ in range(2):      # the counters of the split loop must be back at zero for the second call
                plan.shuffle(part, coded, out, ws if plan.workspace_bytes else None)
            torch.cuda.synchronize()
            assert canaries_intact(out_w, Q * B) and canaries_intact(ws_w, plan.workspace_bytes // 4)
            assert_outputs(out, o, dtype)
            assert f"threads={threads}" in ccdc.last_decode_kernel() and f"chunks={chunks}" in ccdc.last_decode_kernel()
            with pytest.raises(ccdc.CcdcError) as e:
                plan.tune_decode(threads, chunks)           # the tables are on the device now
            assert e.value.status == ccdc.ESTATE
    bad = ccdc.Plan(10, 3, 480, 10, 96, dtype)
    for threads, chunks in ((512, 4), (128, 0), (128, 121)):
        with pytest.raises(ccdc.CcdcError) as e:
            bad.tune_decode(threads, chunks)
        assert e.value.status == ccdc.EINVAL


@pytest.mark.parametrize("dtype", ["int32", "float32"])
@pytest.mark.parametrize("K,r,N,Q,B", [(3, 1, 30, 3, 2100), (4, 2, 54, 4, 1100), (5, 3, 50, 5, 774), (5, 4, 15, 5, 1304),
                                       (6, 2, 30, 12, 514)])
def test_clustered_decode_for_every_operand_count(ccdc, K, r, N, Q, B, dtype):
    """Splits of 2, 5 and 8 chunks whose partial sums meet in a thread-block cluster, for r = 1..4, 64- and
    128-bit accesses, ragged tails: outputs against the oracle, no workspace touched."""
    o = Oracle(K, r, N, Q, B, dtype)
    v = values_numpy(N, Q, B, dtype, seed=r)
    o.load_values(v)
    o.shuffle()
    for chunks in (2, 5, 8):
        plan = ccdc.Plan(K, r, N, Q, B, dtype)
        if chunks > plan.num_batches:
            continue
        plan.tune_decode(plan.decode_threads, chunks)
        assert plan.decode_cluster and plan.workspace_bytes == 0, (K, r, chunks)
        part = plan.alloc_partitions()
        plan.fill_partitions(part, torch.from_numpy(v).cuda())
        coded = plan.alloc(plan.coded_bytes)
        out_w, out = guarded(Q * B, plan.torch_dtype)
        plan.shuffle(part, coded, out, None)
        torch.cuda.synchronize()
        assert canaries_intact(out_w, Q * B)
        assert_outputs(out, o, dtype)
        assert "cluster" in ccdc.last_decode_kernel() and f"chunks={plan.decode_chunks}" in ccdc.last_decode_kernel()


@pytest.mark.parametrize("K,r,N,Q,B,chunks", [(6, 2, 15, 6, 3000, 0), (10, 3, 480, 10, 64, 0), (10, 3, 480, 10, 64, 12),
                                              (8, 4, 70, 8, 4096, 0)])
def test_back_to_back_steps_on_the_same_buffers(ccdc, K, r, N, Q, B, chunks):
    """Forty shuffles in a row on one stream without a synchronise, the inputs swapped between two sets
    before every step: each kernel may be scheduled while its predecessor drains (programmatic dependent
    launch), so a read or write placed before its dependency wait would show here.  The last two steps'
    coded rows and outputs are compared with the oracle."""
    dtype = "int32"
    plan = ccdc.Plan(K, r, N, Q, B, dtype)
    if chunks:
        plan.tune_decode(plan.decode_threads, chunks)
    sets, refs = [], []
    for seed in (1, 2):
        v = values_numpy(N, Q, B, dtype, seed=seed)
        o = Oracle(K, r, N, Q, B, dtype)
        o.load_values(v)
        o.shuffle()
        refs.append((o.coded().copy(), o.reduce().copy()))
        p = plan.alloc_partitions()
        plan.fill_partitions(p, torch.from_numpy(v).cuda())
        sets.append(p)
    part = plan.alloc_partitions()
    coded, out = plan.alloc(plan.coded_bytes), plan.alloc(plan.out_bytes)
    ws = plan.alloc(plan.workspace_bytes)
    keep = {}
    s, sp = plan.segment_elems, plan.coded_row_elems
    for step in range(40):
        which = step % 2
        for dst, src in zip(part, sets[which]):
            dst.copy_(src, non_blocking=True)
        plan.shuffle(part, coded, out, ws if ws.numel() else None)
        if step >= 38:
            keep[which] = (coded.clone(), out.clone())
    torch.cuda.synchronize()
    for which in (0, 1):
        c, o_ = keep[which]
        assert np.array_equal(bits(c).reshape(-1, sp)[:, :s], refs[which][0].reshape(-1, s))
        assert np.array_equal(o_.cpu().numpy().reshape(refs[which][1].shape), refs[which][1])
    plan.shuffle_status()


def random_shapes(seed, count):
    """`count` parameter sets of the scheme drawn from a seeded generator: K up to 12, every r, 1 to 9 files
    per batch, Q/K up to 3, value lengths from 1 to 24 000 words, one job or the J-job setting, both
    dtypes; some with the bulk-copy kernels, some with a drawn launch shape of the fused decode."""
    import random

    rng = random.Random(seed)
    while count > 0:
        jobs = rng.random() < 0.2
        K = rng.randint(3, 6 if jobs else 12)
        r = rng.randint(1, K - 1)
        if jobs:
            N = rng.randint(1, 4) * (r + 1)
            if comb(K, r + 1) > 60 or N < K:
                continue
        else:
            if comb(K, r) > 500:
                continue
            N = rng.choice([1, 1, 2, 3, 4, 5, 7, 9]) * comb(K, r)
        Q = K * rng.choice([1, 1, 1, 2, 3])
        kind = rng.random()
        B = rng.randint(1, 40) if kind < 0.3 else rng.randint(41, 3000) if kind < 0.7 else rng.randint(3000, 24000)
        if (comb(K, r + 1) if jobs else 1) * N * Q * B > 12_000_000:
            continue
        dtype = rng.choice(["int32", "float32"])
        family = 1 if rng.random() < 0.3 and bulk_copy_family_serves(K, r, N, Q, B) else None
        shape = (rng.random() < 0.5, rng.random() < 0.5, rng.randint(1, 16))    # override?, short blocks?, chunks
        yield K, r, N, Q, B, dtype, jobs, family, shape
        count -= 1


@pytest.mark.parametrize("seed", [11, 12, 13, 14])
def test_random_shapes_match_oracle(ccdc, seed):
    """Thirty drawn parameter sets per seed, each through the stepwise and the fused path against the oracle."""
    for case, (K, r, N, Q, B, dtype, jobs, family, (override, short, chunks)) in enumerate(random_shapes(seed, 30)):
        tune = None
        if family is None and override:
            probe = ccdc.Plan(K, r, N, Q, B, dtype, jobs=jobs)
            threads = probe.decode_threads if probe.decode_threads == 128 else (1024 if short else 512)
            try:
                probe.tune_decode(threads, chunks)
                tune = (threads, chunks)
            except ccdc.CcdcError as e:         # more chunks than terms in the batch loop
                assert e.status == ccdc.EINVAL
        try:
            run_case(ccdc, K, r, N, Q, B, dtype, jobs=jobs, seed=seed * 100 + case, tune=tune, family=family)
        except AssertionError as e:
            raise AssertionError(f"{(K, r, N, Q, B, dtype, jobs, family, tune)}: {e}") from e


@pytest.mark.parametrize("seed", [21, 22])
def test_random_shapes_through_the_other_entry_points(ccdc, seed):
    """Twenty-five drawn parameter sets per seed through the compression-only comparator, the node-sharded
    plans (all ranks on this GPU, one after the other) and the two entries that start from host memory."""
    import random

    rng = random.Random(seed)
    done = 0
    while done < 25:
        what = rng.choice(["comparator", "node shards", "host files", "host buffers"])
        dtype = rng.choice(["int32", "float32"])
        K = rng.randint(3, 10)
        r = rng.randint(1, K - 1)
        Q = K * rng.choice([1, 1, 2])
        kind = rng.random()
        B = rng.randint(1, 40) if kind < 0.3 else rng.randint(41, 3000) if kind < 0.7 else rng.randint(3000, 12000)
        jobs = what in ("node shards", "host files") and rng.random() < 0.3
        if what == "comparator":
            N = rng.randint(K, 60)
            if (r * N) % K or N - (-(-K // r) - 1) * (r * N // K) < 1:
                continue
        elif jobs:
            N = rng.randint(1, 3) * (r + 1)
            if K > 6 or comb(K, r + 1) > 40 or N < K:
                continue
        else:
            if comb(K, r) > 260:
                continue
            N = rng.choice([1, 2, 3, 4]) * comb(K, r)
        if (comb(K, r + 1) if jobs else 1) * N * Q * B > 6_000_000:
            continue
        try:
            if what == "comparator":
                test_compression_only_matches_oracle(ccdc, K, r, N, Q, B, dtype)
            elif what == "node shards":
                worlds = [w for w in range(2, K + 1) if K % w == 0]
                test_node_sharded_ranks_emulated_on_one_gpu(ccdc, K, r, N, Q, B, rng.choice(worlds), jobs, dtype)
            elif what == "host files":
                test_shuffle_from_host_files(ccdc, K, r, N, Q, B, jobs, dtype)
            else:
                test_shuffle_from_host_buffers(ccdc, K, r, N, Q, B, dtype)
        except AssertionError as e:
            raise AssertionError(f"{what} {(K, r, N, Q, B, dtype, jobs)}: {e}") from e
        done += 1


def test_jobs20_structure_short_values(ccdc):
    """The paper's own setting at the benchmark's scale of nodes -- K=20, r=2, J = C(20,3) = 1140 jobs of
    21 files, 7 per batch, stage 1 and 17 stage-2 rounds per subset -- with short values: every coded
    word, packet and output against the oracle, and the load of Theorem 1."""
    from fractions import Fraction

    w = CONFIGS["jobs20"].scaled(96)
    plan = run_case(ccdc, w.K, w.r, w.N, w.Q, w.B, w.dtype, jobs=True, std=w.std)
    assert plan.J == 1140 and plan.files_per_batch == 7 and plan.num_groups == 1140 * 18
    assert Fraction(plan.coded_bits, plan.J * w.Q * 32 * w.B) == Fraction(27, 20)       # (1-mu)(mu K+1)/(mu K) = 1.35
    assert "files=4" in ccdc.last_decode_kernel()


def test_bench_line_contract(ccdc):
    """`python bench.py --workload cfg1`: one JSON line with every key the measurement contract names."""
    import json
    import subprocess
    import sys
    from pathlib import Path

    root = Path(__file__).resolve().parent.parent
    res = subprocess.run([sys.executable, str(root / "bench.py"), "--workload", "cfg1", "--steps", "5", "--warmup", "3"],
                         capture_output=True, text=True, timeout=900, cwd=str(root))
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "roofline", "cpu_baseline", "e2e", "gpu_launches", "clocks"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 5 and d["warmup"] == 3 and d["dtype"] == "i32"
    assert d["config"]["workload"] == "cfg1" and d["vs_baseline"] is None and d["value"] > 0
    for key in ("bound", "achieved", "peak", "unit", "frac", "frac_nominal", "traffic", "algorithmic_gbs"):
        assert key in d["roofline"], key
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] == 1 and d["cpu_baseline"]["value"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] == 12 * 4 * 256 * 4 and d["e2e"]["d2h_bytes_per_step"] == 4 * 256 * 4
    assert d["gpu_launches"] >= 2 * 5
