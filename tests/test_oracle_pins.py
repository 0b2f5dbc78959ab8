"""Pins of the CPU oracle to things other than itself.

Each test ties a part of ``oracle/ccdc_oracle.c`` to what the paper or plain
mathematics fixes: the direct sum of Eq. (1), the decode guarantee of
Section IV, the loads the paper prints for its two worked examples, Theorem 1,
the per-round packet size, the storage constraint, the closed forms for plain
CDC and combining, and special cases that collapse to something elementary.
"""
from fractions import Fraction
from itertools import combinations
from math import comb

import numpy as np
import pytest

from oracle.ccdc_oracle import Oracle, map_linear_regression
from paper_1805_01993_b200.inputs import values_numpy, round_to_bf16


def read_golden(path):
    """``key value...`` lines of a golden text fixture -> list of (key, [tokens])."""
    rows = []
    for line in path.read_text().splitlines():
        line = line.strip()
        if line and not line.startswith("#"):
            tok = line.split()
            rows.append((tok[0], tok[1:]))
    return rows


def golden_scalar(rows, key):
    return Fraction([t for k, t in rows if k == key][0][0])


# shapes that exercise: r = 1, r = K-1, several files per batch, several
# functions per node, a packet length that r does not divide, B < r
TINY = [
    # K, r, N, Q, B
    (3, 2, 6, 3, 8),
    (3, 1, 3, 3, 5),
    (4, 2, 12, 4, 6),
    (4, 3, 8, 4, 9),
    (4, 1, 8, 8, 3),
    (5, 2, 20, 5, 7),      # r does not divide len = 7
    (5, 3, 10, 10, 5),     # Q/K = 2, len = 10, r = 3
    (5, 4, 5, 5, 2),       # B < r: empty trailing segments
    (6, 3, 40, 6, 4),
    (6, 2, 15, 12, 3),
]


# ---------------------------------------------------------------- Eq. (1)
@pytest.mark.parametrize("K,r,N,Q,B", TINY)
def test_int32_outputs_equal_direct_sum(K, r, N, Q, B):
    """Every Reduce output is the wrapped sum of its N Map values (Eq. (1))."""
    v = values_numpy(N, Q, B, "int32", seed=K * 100 + r)
    o = Oracle(K, r, N, Q, B, "int32")
    out = o.run(v)
    # the definition, with numpy: sum over the file axis in 64 bits, wrap to 32
    expect = (v.astype(np.int64).sum(axis=0) & 0xFFFFFFFF).astype(np.uint32).view(np.int32)
    assert np.array_equal(out, expect)
    assert np.array_equal(o.direct(), expect)


@pytest.mark.parametrize("K,r,N,Q,B", TINY)
def test_fp32_outputs_close_to_direct_sum(K, r, N, Q, B):
    """fp32: within N rounding errors of the binary64 sum, relative to sum |v|."""
    v = values_numpy(N, Q, B, "float32", seed=7 + K)
    o = Oracle(K, r, N, Q, B, "float32")
    out = o.run(v)
    s64 = v.astype(np.float64).sum(axis=0)
    a64 = np.abs(v.astype(np.float64)).sum(axis=0)
    assert np.all(np.abs(out - s64) <= N * 2.0 ** -24 * a64 + 1e-30)
    ds, da = o.direct()
    assert np.allclose(ds, s64, rtol=1e-14, atol=1e-14) and np.allclose(da, a64, rtol=1e-14)


def test_fp32_summation_order_is_batches_then_files():
    """The fp32 result is the left-to-right sum of per-batch sums, batches in
    lexicographic order, files ascending inside a batch -- checked with numpy
    float32 scalars on a case where the order changes the rounding."""
    K, r, N, Q, B = 4, 2, 18, 4, 3
    v = (values_numpy(N, Q, B, "float32", seed=3) * np.float32(1e4)).astype(np.float32)
    v[::3] *= np.float32(1e-4)          # mixed magnitudes: order matters
    o = Oracle(K, r, N, Q, B, "float32")
    out = o.run(v)
    b = N // comb(K, r)
    expect = np.zeros((Q, B), dtype=np.float32)
    for q in range(Q):
        for e in range(B):
            acc = np.float32(0)
            for p in range(comb(K, r)):
                t = v[p * b, q, e]
                for f in range(1, b):
                    t = np.float32(t + v[p * b + f, q, e])
                acc = np.float32(acc + t)
            expect[q, e] = acc
    assert np.array_equal(out.view(np.uint32), expect.view(np.uint32))
    naive = v.sum(axis=0, dtype=np.float32)
    assert not np.array_equal(naive.view(np.uint32), expect.view(np.uint32)), \
        "case too easy: the order did not matter"


def test_linearity_int32():
    """The whole scheme is linear over Z/2^32: out(u + v) = out(u) + out(v)."""
    K, r, N, Q, B = 5, 2, 20, 5, 6
    u = values_numpy(N, Q, B, "int32", seed=1)
    v = values_numpy(N, Q, B, "int32", seed=2)
    w = (u.view(np.uint32) + v.view(np.uint32)).view(np.int32)
    o = Oracle(K, r, N, Q, B, "int32")
    a = o.run(u).view(np.uint32).copy()
    b = o.run(v).view(np.uint32).copy()
    c = o.run(w).view(np.uint32).copy()
    assert np.array_equal(a + b, c)


# ------------------------------------------------------- decode guarantee
@pytest.mark.parametrize("K,r,N,Q,B", TINY)
def test_every_receiver_recovers_its_packets(K, r, N, Q, B):
    """Section IV: from X_{k'} node k recovers V_{K\\{k},k'} -- the oracle's
    shuffle reports any packet that differs from what its senders built."""
    for dt in ("int32", "float32"):
        v = values_numpy(N, Q, B, dt, seed=11)
        o = Oracle(K, r, N, Q, B, dt)
        o.load_values(v)
        assert o.shuffle_status() == 0
        # decoded packets equal the packet built at a node that stores the batch
        for k in range(K):
            dec = o.decoded(k)
            rounds = [ro for ro in range(o.nround) if k in o.round_group(ro)]
            assert len(rounds) == comb(K - 1, r) == dec.shape[0]
            for i, ro in enumerate(rounds):
                S = o.round_group(ro)
                p = o.round_batches(ro)[S.index(k)]
                P = o.batch_nodes(p)
                assert sorted(P + [k]) == S
                files = o.batch_files(p)
                per = Q // K
                acc = v[files[0], k * per:(k + 1) * per].copy()
                for f in files[1:]:
                    acc = acc + v[f, k * per:(k + 1) * per]
                assert np.array_equal(dec[i], acc.reshape(-1).view(np.uint32))


def test_disagreeing_replicas_are_detected():
    """Planted fault: if one replica of a value differs, cancellation leaves a
    residue and the decode check must fire."""
    K, r, N, Q, B = 4, 2, 12, 4, 6
    v = values_numpy(N, Q, B, "int32", seed=5)
    o = Oracle(K, r, N, Q, B, "int32")
    o.load_values(v)
    assert o.shuffle_status() == 0
    # node 0, first stored file, function 3 (needed by node 3), element 2
    o.poke_node(0, 3 * B + 2, 0x00010000)
    assert o.shuffle_status() == -10


def test_damaged_broadcast_is_detected():
    K, r, N, Q, B = 4, 2, 12, 4, 6
    v = values_numpy(N, Q, B, "float32", seed=5)
    o = Oracle(K, r, N, Q, B, "float32")
    o.load_values(v)
    assert o.shuffle_status() == 0
    assert o.redecode_status() == 0
    o.poke_log(4, 0x1)
    assert o.redecode_status() == -10


def test_xor_of_coded_packet_with_side_information():
    """A coded packet is exactly the XOR of r labelled segments: recomputed here
    from the raw values with numpy for every round of a small instance."""
    K, r, N, Q, B = 5, 3, 20, 5, 7           # s = 3, last segment has 1 element
    v = values_numpy(N, Q, B, "int32", seed=9)
    o = Oracle(K, r, N, Q, B, "int32")
    o.load_values(v)
    o.shuffle()
    coded = o.coded()
    b, s, L = o.b, o.s, o.len
    assert (b, s, L) == (2, 3, 7)
    subsets = list(combinations(range(K), r))
    for g, S in enumerate(combinations(range(K), r + 1)):
        assert list(S) == o.round_group(g)
        for a, sender in enumerate(S):
            x = np.zeros(s, dtype=np.uint32)
            for t in S:
                if t == sender:
                    continue
                P = tuple(m for m in S if m != t)
                p = subsets.index(P)
                pkt = v[p * b:(p + 1) * b, t].astype(np.int64).sum(axis=0) & 0xFFFFFFFF
                pad = np.zeros(r * s, dtype=np.uint32)
                pad[:L] = pkt.astype(np.uint32)
                i = P.index(sender)
                x ^= pad[i * s:(i + 1) * s]
            assert np.array_equal(coded[g, a], x)


# ------------------------------------------------------------- placement
@pytest.mark.parametrize("K,r,N,Q,B", TINY)
def test_placement_storage_and_replication(K, r, N, Q, B):
    """Section IV-A with one job: every node stores mu*N = r*N/K files, every
    file sits on exactly r nodes, every batch label is a distinct r-subset."""
    o = Oracle(K, r, N, Q, B, "int32")
    labels = [tuple(o.batch_nodes(p)) for p in range(o.nbatch)]
    assert labels == list(combinations(range(K), r))
    holders = {n: set() for n in range(N)}
    for p, P in enumerate(labels):
        for n in o.batch_files(p):
            holders[n].update(P)
    assert all(len(h) == r for h in holders.values())
    for k in range(K):
        assert o.node_num_files(k) * K == r * N
    # every batch reaches every outside node in exactly one round
    for p, P in enumerate(labels):
        for k in range(K):
            ro = o.recv_round(p, k)
            assert (ro == -1) == (k in P)
            if ro >= 0:
                assert o.round_group(ro) == sorted(P + (k,))


def test_paper_mode_storage_is_mu_J_N():
    """Section IV-A: each node stores mu*J*N files; job j lives on K_j only."""
    for K, r, N in [(4, 2, 6), (5, 2, 9), (5, 3, 8), (6, 1, 6)]:
        o = Oracle(K, r, N, K, 2, "int32", mode="paper")
        J = comb(K, r + 1)
        assert o.J == J and o.nbatch == J * (r + 1) and o.nround == J * (K - r)
        for k in range(K):
            assert Fraction(o.node_num_files(k)) == Fraction(r, K) * J * N
        homes = list(combinations(range(K), r + 1))
        for p in range(o.nbatch):
            assert set(o.batch_nodes(p)) < set(homes[o.batch_job(p)])


def test_motivating_example_placement_structure(golden_dir):
    """Section II: nodes store {1,2,3,4}, {3,4,5,6}, {5,6,1,2}.  Batch labels are
    free up to renaming files, so compare what is invariant: files per node and
    the number of files each pair of nodes shares."""
    rows = read_golden(golden_dir / "motivating_example_k3.txt")
    paper = {int(t[0]): set(map(int, t[1:])) for k, t in rows if k == "node"}
    K = int(golden_scalar(rows, "K"))
    N, Q = int(golden_scalar(rows, "N")), int(golden_scalar(rows, "Q"))
    per_node = int(golden_scalar(rows, "files_per_node"))
    r = per_node * K // N
    o = Oracle(K, r, N, Q, 4, "int32")
    ours = {k + 1: set() for k in range(K)}
    for p in range(o.nbatch):
        for k in o.batch_nodes(p):
            ours[k + 1].update(n + 1 for n in o.batch_files(p))
    assert all(len(ours[k]) == per_node == len(paper[k]) for k in paper)
    for a, b in combinations(sorted(paper), 2):
        assert len(ours[a] & ours[b]) == len(paper[a] & paper[b])
    assert set().union(*ours.values()) == set().union(*paper.values())


# ------------------------------------------------------ loads the paper prints
def test_motivating_example_loads(golden_dir):
    """Section II: uncoded 6, compression 3, CDC 3, compressed CDC 3/2, all in
    units of T; each coded packet is half an intermediate value."""
    rows = read_golden(golden_dir / "motivating_example_k3.txt")
    K, N, Q = (int(golden_scalar(rows, k)) for k in ("K", "N", "Q"))
    B = 16
    T = 32 * B
    o = Oracle(K, 2, N, Q, B, "int32")
    o.run(values_numpy(N, Q, B, "int32"))
    assert Fraction(o.coded_bits, T) == golden_scalar(rows, "load_compressed_cdc")
    assert Fraction(o.bits_uncoded, T) == golden_scalar(rows, "load_uncoded")
    assert Fraction(o.bits_combining, T) == golden_scalar(rows, "load_compression")
    assert Fraction(o.bits_plain_cdc, T) == golden_scalar(rows, "load_cdc")
    assert Fraction(32 * o.s, T) == golden_scalar(rows, "coded_packet_fraction")
    assert o.nround == 1 and o.coded().shape == (1, 3, B // 2)


def test_running_example_loads(golden_dir):
    """Section IV example: 3/32 for stage 1, 3/32 for stage 2 in one subset,
    3/4 in total, against J*Q*T; the plain-CDC formula gives 3/2 and the
    compression formula 1 for the same K, mu, N."""
    rows = read_golden(golden_dir / "running_example_k4.txt")
    K, r, J, N, Q = (int(golden_scalar(rows, k)) for k in ("K", "r", "J", "N", "Q"))
    B = 8
    T = 32 * B
    o = Oracle(K, r, N, Q, B, "int32", mode="paper")
    assert o.J == J
    v = values_numpy(J * N, Q, B, "int32")
    out = o.run(v)
    per_round = Fraction((r + 1) * 32 * o.s, J * Q * T)
    assert per_round == golden_scalar(rows, "load_stage1") == golden_scalar(rows, "load_stage2")
    assert o.nround == comb(K, r + 1) * 2          # stage 1 + one stage-2 round per subset
    assert Fraction(o.coded_bits, J * Q * T) == golden_scalar(rows, "load_total")
    mu = Fraction(r, K)
    assert (1 - mu) * N / (mu * K) == golden_scalar(rows, "load_cdc")
    assert (1 if mu >= Fraction(1, 2) else -(-1 // mu) - 1) == golden_scalar(rows, "load_compression")
    # outputs: J independent jobs, each the direct sum of its own files
    expect = (v.astype(np.int64).reshape(J, N, Q, B).sum(axis=1) & 0xFFFFFFFF)
    assert np.array_equal(out.view(np.uint32), expect.astype(np.uint32).reshape(J * Q, B))


def test_running_example_placement_and_final_reduction(golden_dir):
    """Section IV example: job 1's batches on nodes {1,2,3} are {1,2},{1,3},{2,3}
    with two files each; node 1 completes jobs 1, 2, 3 inside the subsets
    {1,2,3}, {1,2,4}, {1,3,4} and receives in each a two-file partial sum of
    job 4 (which lives on {2,3,4})."""
    rows = read_golden(golden_dir / "running_example_k4.txt")
    K, r, N, Q = (int(golden_scalar(rows, k)) for k in ("K", "r", "N", "Q"))
    o = Oracle(K, r, N, Q, 4, "int32", mode="paper")
    paper_batches = {}
    for k, t in rows:
        if k == "batch":
            c = t.index(":")
            paper_batches[tuple(int(x) for x in t[:c])] = [int(x) for x in t[c + 1:]]
    ours = {tuple(n + 1 for n in o.batch_nodes(p)): o.batch_files(p)
            for p in range(o.nbatch) if o.batch_job(p) == 0}
    assert set(ours) == set(paper_batches)
    assert all(len(ours[P]) == len(paper_batches[P]) for P in ours)
    assert sorted(n + 1 for f in ours.values() for n in f) == sorted(
        n for f in paper_batches.values() for n in f)
    homes = list(combinations(range(1, K + 1), r + 1))
    for k, t in rows:
        if k != "node1":
            continue
        S = tuple(int(x) for x in t[1:4])
        done_job, partial_job = int(t[5]), int(t[7])
        assert homes[done_job - 1] == S
        # rounds in this subset where node 1 is a receiver
        got = []
        for ro in range(o.nround):
            if tuple(n + 1 for n in o.round_group(ro)) == S:
                p = o.round_batches(ro)[0]          # node 1 is the smallest member
                got.append((o.batch_job(p) + 1, tuple(n + 1 for n in o.batch_nodes(p))))
        assert sorted(j for j, _ in got) == sorted([done_job, partial_job])
        for j, P in got:
            assert set(P) == set(S) - {1}
            assert set(P) < set(homes[j - 1])
    assert o.b == int(golden_scalar(rows, "partial_files"))


@pytest.mark.parametrize("K", [3, 4, 5, 6, 7])
def test_theorem1_load(K):
    """Theorem 1: L = (1-mu)(mu K+1)/(mu K) for mu K in {1..K-1}, J = C(K, mu K+1),
    counted from the packets the oracle actually broadcasts."""
    for r in range(1, K):
        B = 2 * r                                  # r | len: no padding
        N = r + 1
        N *= -(-K // N)                            # K <= N, (r+1) | N
        o = Oracle(K, r, N, K, B, "int32", mode="paper")
        o.run(values_numpy(o.J * N, K, B, "int32", seed=K))
        mu = Fraction(r, K)
        assert Fraction(o.coded_bits, o.J * K * 32 * B) == (1 - mu) * (mu * K + 1) / (mu * K)
        # per round: mu K + 1 packets of (Q/K) T / (mu K) bits
        assert o.coded().shape == (o.nround, r + 1, B // r)
        assert o.nround == comb(K, r + 1) * (K - r)


@pytest.mark.parametrize("K,r,N,Q,B", TINY)
def test_single_job_bit_count_and_comparators(K, r, N, Q, B):
    """One job over all r-subsets: C(K,r+1) rounds of r+1 packets of s words.
    When r | len this is C(K-1,r)/r in units of Q*T, equals the plain-CDC
    formula with N replaced by the number of batches, and equals Theorem 1 when
    divided by the C(K,r)/(r+1) job-equivalents it carries.  On the same
    placement combining alone costs r times, plain CDC b times and uncoded
    unicast r*b times as much."""
    o = Oracle(K, r, N, Q, B, "int32")
    o.run(values_numpy(N, Q, B, "int32"))
    Gs, L = comb(K, r + 1), (Q // K) * B
    s = -(-L // r)
    assert o.s == s and o.len == L and o.b * comb(K, r) == N
    assert o.coded_bits == Gs * (r + 1) * 32 * s
    ideal = Fraction(Gs * (r + 1) * 32 * L, r)
    assert Fraction(o.coded_bits) == ideal * Fraction(r * s, L)
    QT = Q * 32 * B
    mu = Fraction(r, K)
    assert ideal / QT == Fraction(comb(K - 1, r), r)
    assert ideal / QT == (1 - mu) * comb(K, r) / (mu * K)              # L_CDC with N -> #batches
    assert ideal / QT / Fraction(comb(K, r), r + 1) == (1 - mu) * (mu * K + 1) / (mu * K)
    assert o.bits_combining == Gs * (r + 1) * 32 * L
    assert o.bits_combining == r * ideal
    assert o.bits_uncoded == r * o.b * ideal
    assert o.bits_plain_cdc == o.b * o.coded_bits
    # plain CDC load formula (1-mu) N / (mu K), in units of Q*T
    assert Fraction(o.b) * ideal / QT == (1 - mu) * N / (mu * K)


def test_expected_bits_of_the_five_workloads():
    """Multicast bit counts of the five evaluation shapes, from
    Gs*(r+1)*32*ceil(len/r); the large ones are run with B scaled down by a
    factor that keeps r | B, since the count is linear in the segment length."""
    expect = {  # name: (K, r, N, Q, B, bits)
        "cfg1": (4, 2, 12, 4, 256, 49_152),
        "cfg2": (10, 3, 480, 10, 4096, 36_718_080),
        "cfg3": (16, 4, 1820, 16, 16384, 2_862_612_480),
        "cfg4": (20, 2, 190, 20, 1_280_000, 70_041_600_000),
        "cfg5": (8, 3, 112, 8, 1024, 3_064_320),
    }
    for name, (K, r, N, Q, B, bits) in expect.items():
        scale = {"cfg3": 1024, "cfg4": 160_000, "cfg2": 1, "cfg1": 1, "cfg5": 1}[name]
        if name == "cfg2":
            # full K, r, N, Q with a short value: checks the padded-segment count
            o = Oracle(K, r, N, Q, 16, "int32")
            o.run(values_numpy(N, Q, 16, "int32"))
            assert o.coded_bits == comb(K, r + 1) * (r + 1) * 32 * 6
            assert comb(K, r + 1) * (r + 1) * 32 * (-(-B // r)) == bits
            continue
        Bs = B // scale
        o = Oracle(K, r, N, Q, Bs, "int32")
        o.run(values_numpy(N, Q, Bs, "int32"))
        if (B % r) == 0:
            assert o.coded_bits * scale == bits
        else:
            assert o.coded_bits == bits


# ---------------------------------------------------------- special cases
def test_r1_is_unicast_of_precombined_packets():
    """r = 1: one segment, nothing to XOR with: each coded packet is the
    pre-combined packet itself and its only receiver is the other member."""
    K, r, N, Q, B = 4, 1, 8, 4, 5
    v = values_numpy(N, Q, B, "int32", seed=21)
    o = Oracle(K, r, N, Q, B, "int32")
    o.run(v)
    coded = o.coded()
    for g, (a, c) in enumerate(combinations(range(K), 2)):
        # sender a holds batch {a}: files 2a, 2a+1; the packet is for node c
        for sender, recv, slot in ((a, c, 0), (c, a, 1)):
            pkt = (v[2 * sender:2 * sender + 2, recv].astype(np.int64).sum(axis=0) & 0xFFFFFFFF)
            assert np.array_equal(coded[g, slot], pkt.astype(np.uint32))
    assert o.coded_bits == o.bits_combining


def test_single_job_on_r_plus_1_nodes_is_stage_1():
    """K = r+1: the one-job plan and the paper's plan are the same scheme
    (one subset, stage 1 only): identical broadcast logs and outputs."""
    for K, N, B in [(3, 6, 8), (4, 8, 9), (5, 10, 4)]:
        r = K - 1
        v = values_numpy(N, K, B, "float32", seed=K)
        a = Oracle(K, r, N, K, B, "float32")
        b = Oracle(K, r, N, K, B, "float32", mode="paper")
        oa, ob = a.run(v), b.run(v)
        assert b.J == 1 and b.nround == 1
        assert np.array_equal(a.coded(), b.coded())
        assert np.array_equal(oa.view(np.uint32), ob.view(np.uint32))


def test_one_file_per_batch_passes_bits_through():
    """b = 1: combining is the identity, so fp32 payloads (including -0.0, inf,
    NaN patterns) travel through XOR coding and decoding unchanged."""
    K, r, N, Q, B = 4, 2, 6, 4, 4
    v = values_numpy(N, Q, B, "float32", seed=2)
    v.view(np.uint32)[0, 3, 0] = 0x80000000      # -0.0
    v.view(np.uint32)[1, 2, 1] = 0x7F800000      # +inf
    v.view(np.uint32)[2, 0, 2] = 0x7FC12345      # a NaN payload
    o = Oracle(K, r, N, Q, B, "float32")
    o.load_values(v)
    assert o.shuffle_status() == 0
    for k in range(K):
        dec = o.decoded(k)
        rounds = [ro for ro in range(o.nround) if k in o.round_group(ro)]
        for i, ro in enumerate(rounds):
            p = o.round_batches(ro)[o.round_group(ro).index(k)]
            assert np.array_equal(dec[i], v[p, k].view(np.uint32))
    assert o.coded_bits == o.bits_plain_cdc


def test_invalid_parameters_are_refused():
    for bad in [(4, 0, 12, 4, 8), (4, 4, 12, 4, 8), (4, 2, 3, 4, 8), (4, 2, 13, 4, 8),
                (4, 2, 12, 6, 8), (4, 2, 12, 4, 0), (1, 1, 4, 1, 4)]:
        with pytest.raises(ValueError):
            Oracle(*bad, "int32")
    with pytest.raises(ValueError):
        Oracle(4, 2, 7, 4, 8, "int32", mode="paper")     # (r+1) must divide N


# -------------------------------------------------------------- Map oracle
def test_map_linear_regression_small_exact():
    """X^T (X w - y) on integers small enough to be exact, against hand loops."""
    rng = np.random.default_rng(0)
    m, d, Q = 5, 8, 4
    X = rng.integers(-3, 4, size=(m, d)).astype(np.float32)
    w = rng.integers(-2, 3, size=d).astype(np.float32)
    y = rng.integers(-5, 6, size=m).astype(np.float32)
    g = map_linear_regression(X, w, y, Q)
    expect = np.zeros(d)
    for i in range(m):
        resid = sum(float(X[i, j]) * float(w[j]) for j in range(d)) - float(y[i])
        for j in range(d):
            expect[j] += float(X[i, j]) * resid
    assert g.shape == (Q, d // Q)
    assert np.array_equal(g.reshape(-1), expect.astype(np.float32))


def test_map_linear_regression_is_the_gradient():
    """g is the gradient of 0.5*||X w - y||^2: central differences in binary64."""
    rng = np.random.default_rng(1)
    m, d = 16, 12
    X = round_to_bf16(rng.standard_normal((m, d)).astype(np.float32))
    w = round_to_bf16(rng.standard_normal(d).astype(np.float32))
    y = rng.standard_normal(m).astype(np.float32)
    g = map_linear_regression(X, w, y, 3).reshape(-1).astype(np.float64)
    f = lambda ww: 0.5 * np.sum((X.astype(np.float64) @ ww - y.astype(np.float64)) ** 2)
    h = 1e-5
    for j in range(d):
        e = np.zeros(d); e[j] = h
        fd = (f(w.astype(np.float64) + e) - f(w.astype(np.float64) - e)) / (2 * h)
        assert abs(fd - g[j]) <= 1e-5 * max(1.0, abs(g[j]))


# ------------------------------------------------ compression-only comparator
@pytest.mark.parametrize("K,r,N", [(4, 2, 8), (6, 2, 12), (6, 1, 12), (5, 2, 10), (7, 3, 14), (8, 3, 16),
                                   (6, 4, 12), (10, 3, 20), (5, 4, 10)])
def test_compression_only_load_and_result(K, r, N):
    """Appendix: with mu = r/K the compression-only scheme sends ceil(1/mu)-1 packets
    of one value per function, L = ceil(1/mu)-1 (which is 1 for mu >= 1/2), every
    node stores at most mu*N files and every output is the direct sum of Eq. (1)."""
    from oracle.ccdc_oracle import compression_only

    Q, B = 2 * K, 6
    for dt in ("int32", "float32"):
        v = values_numpy(N, Q, B, dt, seed=K + r)
        out, recv, bits, files = compression_only(K, r, N, Q, B, dt, v)
        mu = Fraction(r, K)
        m = -(-K // r)
        expect_L = (-(-1 // mu) - 1) if mu < Fraction(1, 2) else 1
        assert m - 1 == expect_L or mu >= Fraction(1, 2)
        assert Fraction(bits, Q * 32 * B) == m - 1
        if mu <= Fraction(1, 2):
            assert Fraction(bits, Q * 32 * B) == -(-1 // mu) - 1
        else:
            assert Fraction(bits, Q * 32 * B) == 1
        assert all(f <= mu * N for f in files) and recv.shape == (K, m - 1, (Q // K) * B)
        if dt == "int32":
            expect = (v.astype(np.int64).sum(axis=0) & 0xFFFFFFFF).astype(np.uint32).view(np.int32)
            assert np.array_equal(out, expect)
        else:
            s64 = v.astype(np.float64).sum(axis=0)
            a64 = np.abs(v.astype(np.float64)).sum(axis=0)
            assert np.all(np.abs(out - s64) <= N * 2.0 ** -24 * a64)


def test_compression_only_running_example(golden_dir):
    """Remark after the K=4 example: combining alone sends 4 pre-combined packets,
    one for each node, per job: L = 4/4 = 1."""
    from oracle.ccdc_oracle import compression_only

    rows = read_golden(golden_dir / "running_example_k4.txt")
    K, r, N, Q = (int(golden_scalar(rows, k)) for k in ("K", "r", "N", "Q"))
    B = 4
    out, recv, bits, files = compression_only(K, r, N, Q, B, "int32", values_numpy(N, Q, B, "int32"))
    assert recv.shape[0] * recv.shape[1] == 4
    assert Fraction(bits, Q * 32 * B) == golden_scalar(rows, "load_compression")


@pytest.mark.parametrize("mode", ["single", "paper"])
@pytest.mark.parametrize("dtype", ["int32", "float32"])
def test_every_step_acts_word_by_word_along_a_segment(mode, dtype):
    """Section IV-B: sums, XORs and cancellations combine words at equal positions of equal-size
    segments only.  So the same sub-range of every segment is itself an instance of the scheme:
    shuffling the sliced values gives the slices of the coded packets and of the outputs (the property
    the value-dimension sharding over several GPUs rests on).  Checked on the oracle alone."""
    K, r, Q, B = 5, 2, 10, 12                   # Q/K = 2: packets of 24 words, segments of 12
    N = 9 if mode == "paper" else 20
    per = Q // K
    full = Oracle(K, r, N, Q, B, dtype, mode=mode)
    v = values_numpy(full.J * N, Q, B, dtype, seed=17)
    out = full.run(v)
    coded = full.coded()                        # [round][sender][s]
    s = full.s
    for lo, hi in ((0, 4), (4, 12), (5, 7)):
        w = hi - lo
        pos = np.concatenate([np.arange(i * s + lo, i * s + hi) for i in range(r)])
        assert (r * w) % per == 0
        b_local = r * w // per
        packets = v.reshape(full.J * N, K, per * B)
        local = np.ascontiguousarray(packets[:, :, pos]).reshape(full.J * N, Q, b_local)
        part = Oracle(K, r, N, Q, b_local, dtype, mode=mode)
        got = part.run(local)
        assert part.s == w
        assert np.array_equal(part.coded(), coded[:, :, lo:hi])
        want = out.reshape(full.J * K, per * B)[:, pos].reshape(got.shape)
        assert np.array_equal(got.view(np.uint32), np.ascontiguousarray(want).view(np.uint32))
        assert part.coded_bits * s == full.coded_bits * w


# ---------------------------------------------- drawn parameter sets, both settings
@pytest.mark.parametrize("seed", [1, 2, 3])
def test_drawn_parameter_sets_obey_the_definition_and_the_load(seed):
    """Forty parameter sets per seed (K up to 8, every r, several files per batch, Q/K up to 3, value lengths
    that r does or does not divide; one job or J = C(K, r+1) jobs): every output is the wrapped sum of
    Eq. (1) written with numpy, every receiver decodes (the shuffle reports nothing), the multicast bits are
    rounds x (r+1) packets x 32 s, and, where r divides the packet, the J-job load is Theorem 1's."""
    import random

    rng = random.Random(seed)
    done = 0
    while done < 40:
        paper = rng.random() < 0.4
        K = rng.randint(2, 6 if paper else 8)
        r = rng.randint(1, K - 1)
        per = rng.choice([1, 1, 2, 3])
        B = rng.randint(1, 24)
        if paper:
            N = rng.randint(1, 3) * (r + 1)
            if N < K or comb(K, r + 1) > 40:
                continue
            J, rounds, b = comb(K, r + 1), comb(K, r + 1) * (K - r), N // (r + 1)
        else:
            b = rng.randint(1, 4)
            N = b * comb(K, r)
            if N < K:
                continue
            J, rounds = 1, comb(K, r + 1)
        Q = per * K
        v = values_numpy(J * N, Q, B, "int32", seed=seed * 1000 + done)
        o = Oracle(K, r, N, Q, B, "int32", mode="paper" if paper else "single")
        o.load_values(v)
        assert o.shuffle_status() == 0, (K, r, N, Q, B, paper)
        out = o.reduce().reshape(J, Q, B)
        expect = (v.reshape(J, N, Q, B).astype(np.int64).sum(axis=1) & 0xFFFFFFFF).astype(np.uint32).view(np.int32)
        assert np.array_equal(out, expect), (K, r, N, Q, B, paper)
        s = -(-(per * B) // r)
        assert (o.J, o.nround, o.b, o.s) == (J, rounds, b, s)
        assert o.coded_bits == rounds * (r + 1) * 32 * s
        if paper and (per * B) % r == 0:
            mu = Fraction(r, K)
            assert Fraction(o.coded_bits, J * Q * 32 * B) == (1 - mu) * (mu * K + 1) / (mu * K)
        done += 1
