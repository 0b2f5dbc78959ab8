#!/usr/bin/env python
"""Benchmark of the compressed-CDC shuffle on B200.

A step is one pass of the whole shuffle path (pre-combine + encode, then
decode + cancel + reduce) over one batch of synthetic Map outputs that is
already resident in device memory.  The workload is the distributed-SGD
gradient shape (K=20, r=2, N=190, Q=20, 1.28 M floats per value, about 39 GB of
intermediate values held across the 20 logical nodes), far larger than L2.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints one JSON line.  ``value`` is intermediate-value GB/s: the bytes of Map
output every node has to read for the shuffle, divided by the time of a step.
With N > 1 (torchrun) every rank runs an independent job of the same shape
(weak scaling, no collective on the data path).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

from paper_1805_01993_b200.inputs import CONFIGS, DEFAULT_SEED, values_numpy, values_torch  # noqa: E402

METRIC = "shuffle GB/s (combine+encode+decode+reduce)"
UNIT = "GB/s"

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per launch of the dominant kernel of a
# workload, from the ncu captures summarised under profiles/ (file named per entry).  A capture taken
# at a shorter value length is scaled by the value length (every byte the kernel moves grows in
# proportion to it) and the line says "scaled".  An entry is only valid for the kernel sources it was
# measured on (hash over the files listed); otherwise the line reports null.
NCU_TRAFFIC = {
    # workload: (kernel, sources sha256, value elements of the capture, DRAM bytes of that launch, profile)
    "cfg4": ("k_decode_reduce", "60a405a7a0446a11b9ca011cd2614cde98348f8b6d7edb13cf7d7d80c5b447b3",
             128000, 3541666520.0, "profiles/ncu_cfg4_small.md"),
    "cfg3": ("k_decode_reduce", "60a405a7a0446a11b9ca011cd2614cde98348f8b6d7edb13cf7d7d80c5b447b3",
             8208, 3113737120.0, "profiles/ncu_cfg3_small.md"),
    "jobs20": ("k_decode_reduce", "60a405a7a0446a11b9ca011cd2614cde98348f8b6d7edb13cf7d7d80c5b447b3",
             1024, 2256910400.0, "profiles/ncu_jobs20_small.md"),
    "cfg2": ("k_decode_reduce", "60a405a7a0446a11b9ca011cd2614cde98348f8b6d7edb13cf7d7d80c5b447b3",
             4096, 144492544.0, "profiles/ncu_cfg2_full.md"),
    "compression:cfg4": ("k_gather(combine)+k_reduce", "60a405a7a0446a11b9ca011cd2614cde98348f8b6d7edb13cf7d7d80c5b447b3",
             128000, 2141599280.0, "profiles/ncu_compression_small.md"),
    "cfg5": ("k_map", "a7427ce9fd62495f5562f015e6406acaf19ca4a6b7c5b8c4ef81d0fa3406c4a7",
             1024, 2826514184.0, "profiles/k_map_cluster_cfg5.md"),
}
TRAFFIC_SOURCES = {
    "k_decode_reduce": ("ccdc_kernels.cu", "ccdc_internal.h", "ccdc_plan.cpp"),
    "k_gather(encode)": ("ccdc_kernels.cu", "ccdc_internal.h", "ccdc_plan.cpp"),
    "k_gather(combine)+k_reduce": ("ccdc_kernels.cu", "ccdc_internal.h", "ccdc_plan.cpp"),
    "k_map": ("ccdc_map_cluster.cu", "ccdc_map_cluster.h"),
}


def sources_hash(kernel):
    import hashlib

    h = hashlib.sha256()
    for f in TRAFFIC_SOURCES[kernel]:
        h.update((ROOT / "paper_1805_01993_b200" / "csrc" / f).read_bytes())
    return h.hexdigest()


def measured_traffic(w, kernel, prefix=""):
    """(DRAM bytes per launch of `kernel` on workload w, how they were obtained) or (None, None)."""
    base = prefix + w.name.split("[")[0]
    entry = NCU_TRAFFIC.get(base)
    if not entry or entry[0] != kernel or sources_hash(kernel) != entry[1]:
        return None, None
    _, _, elems, dram_bytes, profile = entry
    if elems == w.B:
        return dram_bytes, f"ncu capture of this launch ({profile})"
    return dram_bytes * w.B / elems, f"scaled by {w.B}/{elems} from an ncu capture at B={elems} ({profile})"


# ---------------------------------------------------------------- byte counts
def algorithmic_bytes(K, r, N, Q, B, J=1, rounds=None):
    """Bytes the method must move, node-faithful (each logical node's reads count;
    pre-combined packets are recomputed, never stored)."""
    from math import comb

    length = (Q // K) * B
    s = -(-length // r)
    b = N // comb(K, r) if J == 1 else N // (r + 1)
    rounds = comb(K, r + 1) if rounds is None else rounds
    packets = rounds * (r + 1)                       # (round, receiver) pairs
    enc_iv = packets * length * b * 4                # each packet built once, a segment per sender
    dec_cancel = packets * (r - 1) * length * b * 4  # the other r-1 segments at each receiver
    local = r * J * N * length * 4                   # own function's values
    coded_w = packets * s * 4
    coded_r = r * coded_w
    out = J * Q * B * 4
    return {
        "iv_read": enc_iv + dec_cancel + local,
        "encode_kernel": enc_iv + coded_w,
        "decode_kernel": dec_cancel + local + coded_r + out,
        "coded_write": coded_w,
        "total": enc_iv + dec_cancel + local + coded_w + coded_r + out,
    }


# ---------------------------------------------------------------- multi-rank
def rank_seed(rank: int) -> int:
    """Every rank runs an independent job of the same shape: its own input seed."""
    return DEFAULT_SEED + rank


def max_over_ranks(ms: float, world: int, device):
    """Slowest rank's time (the job is done when the last rank is)."""
    import torch
    import torch.distributed as dist

    t = torch.tensor([ms], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.item()


def whole_job_value(world: int, bytes_per_rank: int, ms_per_step: float) -> float:
    """GB/s over all ranks: every rank moved bytes_per_rank in ms_per_step."""
    return world * bytes_per_rank / (ms_per_step * 1e-3) / 1e9


# ---------------------------------------------------------------- clocks
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None

    def start(self):
        """starts nvidia-smi sampling every 100 ms and waits (up to 3 s) for its first sample, so that a
        short timed region is not over before the sampler is up."""
        import threading

        self.lines = []
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100", "-i", str(self.index)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return

        def pump():
            for line in self.proc.stdout:
                self.lines.append(line)

        self.reader = threading.Thread(target=pump, daemon=True)
        self.reader.start()
        t0 = time.perf_counter()
        while not self.lines and time.perf_counter() - t0 < 3.0:
            time.sleep(0.02)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)                    # one more sample after the timed region's last kernel
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            self.proc.wait()
        self.reader.join(timeout=2)
        text = "".join(self.lines)
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in text.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power)}


def host_cpu():
    """model name and core counts of the host the oracle is timed on."""
    model = "unknown"
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("model name"):
                model = line.split(":", 1)[1].strip()
                break
    except OSError:
        pass
    try:
        usable = len(os.sched_getaffinity(0))
    except AttributeError:
        usable = os.cpu_count()
    return {"cpu_model": model, "host_cores": os.cpu_count(), "host_cores_usable": usable}


SAMPLE_REASON = ("value length shortened so that the single-threaded oracle finishes in the seconds "
                 "the benchmark allows; every step is element-wise along the value, so the rate does not depend on it")


# ---------------------------------------------------------------- oracle legs
def oracle_sample_shape(w, target_seconds):
    """Same K, r, N, Q with the value shortened so one oracle pass takes about
    ``target_seconds`` on one core; calibrated on a very short value first."""
    from oracle.ccdc_oracle import Oracle

    per_elem = None
    probe_B = w.r * 64
    for _ in range(2):      # second pass: a value long enough to leave the caches, about a second of work
        o = Oracle(w.K, w.r, w.N, w.Q, probe_B, w.dtype, mode="paper" if w.jobs else "single")
        o.load_values(values_numpy(o.J * w.N, w.Q, probe_B, w.dtype, std=w.std))
        t0 = time.perf_counter()
        o.shuffle(); o.reduce()
        per_elem = (time.perf_counter() - t0) / probe_B
        nxt = int(min(1.0, target_seconds) / per_elem) // (4 * w.r) * (4 * w.r)
        if nxt <= probe_B or nxt >= w.B:
            break
        probe_B = nxt
    B = int(target_seconds / per_elem) // (4 * w.r) * (4 * w.r)
    return max(4 * w.r, min(B, w.B))


def make_oracle(w, B):
    """The oracle on the workload's structure at value length B, Map outputs placed."""
    from oracle.ccdc_oracle import Oracle

    o = Oracle(w.K, w.r, w.N, w.Q, B, w.dtype, mode="paper" if w.jobs else "single")
    o.load_values(values_numpy(o.J * w.N, w.Q, B, w.dtype, std=w.std))
    return o


def time_oracle(o):
    """One oracle pass (shuffle + reduce; the copy of the Map outputs into the
    node memories is not part of the shuffle and is not timed)."""
    t0 = time.perf_counter()
    o.shuffle(); o.reduce()
    return time.perf_counter() - t0


def sample_bytes(w, B):
    """algorithmic bytes of the workload's structure at value length B."""
    from math import comb

    if w.jobs:
        J = comb(w.K, w.r + 1)
        return algorithmic_bytes(w.K, w.r, w.N, w.Q, B, J=J, rounds=J * (w.K - w.r))
    return algorithmic_bytes(w.K, w.r, w.N, w.Q, B)


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    total_budget = 150.0
    B = oracle_sample_shape(w, total_budget / (args.steps + args.warmup))
    o = make_oracle(w, B)
    for _ in range(args.warmup):
        time_oracle(o)
    t = [time_oracle(o) for _ in range(args.steps)]
    per_step = sum(t) / len(t)
    by = sample_bytes(w, B)
    value = by["iv_read"] / per_step / 1e9
    sample = f"{w.name} with B={B} of {w.B} elements per value (same K, r, N, Q), one pass per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32" if w.dtype == "float32" else "i32",
        "data": "synthetic", "config": {"workload": w.name, "K": w.K, "r": w.r, "N": w.N, "Q": w.Q, "B": w.B},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample,
                         "sample_reason": SAMPLE_REASON if B < w.B else "full size", **host_cpu()},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ---------------------------------------------------------------- CUDA arm
def run_ours(args, w):
    import torch
    import torch.distributed as dist

    from paper_1805_01993_b200 import build as lib_build
    from paper_1805_01993_b200 import ccdc

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        lib_build.build_library()
    if world > 1:
        dist.barrier()
    ccdc.lib()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # --shard-nodes: ONE job over all GPUs, K/N logical nodes per GPU, coded rows exchanged by an
    # all-gather between the two launches (strong scaling).  Default: one independent job per GPU.
    sharded = bool(args.shard_nodes) and world > 1
    if sharded and (w.map_rows or w.K % world):
        raise RuntimeError("--shard-nodes needs a shuffle-only workload and a GPU count that divides K")
    # --shard-values: ONE job over all GPUs, every GPU owning one sub-range of every segment: each rank
    # runs the whole scheme on values of B/N elements, nothing is exchanged (strong scaling).
    value_sharded = bool(args.shard_values) and world > 1
    full_B = w.B
    if value_sharded:
        if sharded or w.map_rows:
            raise RuntimeError("--shard-values is for the shuffle-only workloads and excludes --shard-nodes")
        w = w.scaled(ccdc.value_shard(w.K, w.r, w.Q, w.B, rank, world))
    plan = ccdc.Plan(w.K, w.r, w.N, w.Q, w.B, w.dtype, jobs=w.jobs, shard=(rank, world) if sharded else None)
    if args.family is not None:
        plan.tune_family(args.family)
    if args.decode_chunks:
        plan.tune_decode(plan.decode_threads, args.decode_chunks)
    plan.upload()
    part = plan.alloc_partitions(dev)
    coded = plan.alloc(plan.coded_bytes, dev)
    out = plan.alloc(plan.out_bytes, dev)
    ws = plan.alloc(plan.workspace_bytes, dev)
    by = algorithmic_bytes(w.K, w.r, w.N, w.Q, w.B, J=plan.J, rounds=plan.num_groups)
    stream = torch.cuda.current_stream()
    stages = []
    map_bytes = 0
    if w.map_rows:
        # linear-regression workload: the partitions are produced by the Map, which is
        # part of the step (job time = Map + shuffle); files drawn on the device
        gen = torch.Generator(device=dev)
        gen.manual_seed(rank_seed(rank))
        d = w.Q * w.B
        canon = torch.randn((w.N, w.map_rows, d), generator=gen, device=dev).to(torch.bfloat16)
        # y_n = X_n w* + 0.01 N(0,1), as the workload states (drawn on the device; one file at a time)
        w_star = torch.randn(d, generator=gen, device=dev)
        ycan = torch.stack([canon[n].float() @ w_star for n in range(w.N)])
        ycan += 0.01 * torch.randn((w.N, w.map_rows), generator=gen, device=dev)
        files_x = [canon[plan.node_files(k)].contiguous() for k in range(w.K)]
        files_y = [ycan[plan.node_files(k)].contiguous() for k in range(w.K)]
        del canon, ycan
        wvec = torch.randn(d, generator=gen, device=dev).to(torch.bfloat16)
        map_ws = torch.empty(plan.map_workspace_bytes(w.map_rows) // 4, dtype=torch.float32, device=dev)
        map_bytes = sum(t.numel() * 2 for t in files_x) + sum(plan.partition_bytes(k) for k in range(w.K))
        stages.append(("k_map",
                       lambda: plan.map(files_x, files_y, wvec, w.map_rows, part, map_ws)))
    else:
        # every rank is an independent job of the same shape: its own seed
        plan.fill_partitions_streaming(part, values_torch(plan.J * w.N, w.Q, w.B, w.dtype, dev, seed=rank_seed(rank),
                                                          std=w.std))
    wire = None
    if sharded:
        # Definition 1 counts a multicast once; between GPUs a coded row has to reach every OTHER GPU
        # that hosts one of its receivers.  The all-gather (and the peer stores) deliver every row to
        # all world-1 other GPUs.
        per = w.K // world
        needed = 0
        for g in range(plan.num_groups):
            members = plan.group(g)
            for a, sender in enumerate(members):
                needed += len({k // per for k in members if k != sender} - {sender // per})
        row_bytes = plan.segment_elems * 4
        wire = {"multicast_bytes": plan.coded_bits // 8,
                "wire_bytes_per_step": plan.num_groups * (w.r + 1) * row_bytes * (world - 1),
                "needed_wire_bytes_per_step": needed * row_bytes,
                "exchange": "peer stores by the encode kernel" if args.peer_stores else "NCCL all-gather of the send buffers"}
    if sharded and args.peer_stores:
        # every rank's coded buffer opened in every process; the encode kernel stores each row it
        # produces into all of them, an all-reduce of one word orders the ranks before the decode
        mine = ccdc.PeerBuffer.create(plan.coded_bytes)
        handles = [None] * world
        dist.all_gather_object(handles, mine.handle)
        peers = [mine if d == rank else ccdc.PeerBuffer.open(handles[d], plan.coded_bytes) for d in range(world)]
        coded = mine
        token = torch.zeros(1, device=dev)
        stages.append(("k_gather(encode)", lambda: plan.encode_fused_peers(part, peers)))
        stages.append(("all_gather(coded rows)", lambda: dist.all_reduce(token)))
    elif sharded:
        send = plan.alloc(plan.coded_send_bytes, dev)
        stages.append(("k_gather(encode)", lambda: plan.encode_fused(part, send)))
        stages.append(("all_gather(coded rows)", lambda: dist.all_gather_into_tensor(coded, send)))
    else:
        stages.append(("k_gather(encode)", lambda: plan.encode_fused(part, coded)))
    stages.append(("k_decode_reduce", lambda: plan.decode_reduce(part, coded, out, ws)))
    share = world if sharded else 1                      # a rank's part of the job
    stage_bytes = {"k_map": map_bytes, "k_gather(encode)": by["encode_kernel"] // share,
                   "k_decode_reduce": by["decode_kernel"] // share,
                   "all_gather(coded rows)": by["coded_write"] * (world - 1) // max(world, 1)}
    input_bytes = sum(plan.partition_bytes(k) for k in range(w.K)) + map_bytes
    # inputs that fit in L2 (126 MB) would be served from it on every repeat: between steps 512 MB are
    # written, then another 512 MB are read; the read pass pushes the dirty lines the write leaves in L2
    # out to memory, so that the step starts with a cold AND clean L2 instead of paying for their write-back
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev) if input_bytes < (1 << 30) else None
    drain = torch.zeros(128 << 20, dtype=torch.int32, device=dev) if flush is not None else None

    def flush_l2():
        flush.zero_()
        drain.sum()

    def one_step(events=None):
        if flush is not None:
            flush_l2()
        for i, (_, fn) in enumerate(stages):
            if events is not None:
                events[i].record(stream)
            fn()
        if events is not None:
            events[len(stages)].record(stream)

    for _ in range(args.warmup):
        one_step()
    barrier()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(len(stages) + 1)] for _ in range(args.steps)]
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = ccdc.num_kernel_launches()
    barrier()
    start.record(stream)
    for i in range(args.steps):
        one_step(ev[i])
    end.record(stream)
    barrier()
    launches = ccdc.num_kernel_launches() - launches0
    clocks = sampler.stop() if rank == 0 else None
    if w.map_rows:
        plan.map_status(w.map_rows, map_ws)     # raises if a bounded wait inside the Map ran out: no number then
    # with a flush between steps the bracket would include it: sum the steps instead
    elapsed_ms = start.elapsed_time(end) if flush is None else sum(e[0].elapsed_time(e[-1]) for e in ev)
    stage_ms = {name: statistics.mean(e[i].elapsed_time(e[i + 1]) for e in ev) for i, (name, _) in enumerate(stages)}
    enc_ms, dec_ms = stage_ms["k_gather(encode)"], stage_ms["k_decode_reduce"]
    ms_per_step = max_over_ranks(elapsed_ms, world, dev) / args.steps
    # Small jobs, and the Map job with its short shuffle, are launch-bound (a step is a handful of kernels,
    # most of a few microseconds): replay the
    # step's launches as ONE CUDA graph, which is how a caller would run such a job repeatedly.  The
    # stage times above stay those of the eager launches.
    launch_mode, eager_ms = "eager launches", ms_per_step
    if (flush is not None or w.map_rows) and world == 1:
        try:
            torch.cuda.synchronize()
            eager_out = out.clone()                 # the replays must reproduce the eager step bit for bit
            side = torch.cuda.Stream(device=dev)
            side.wait_stream(stream)
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(graph, stream=side):
                    for _, fn in stages:
                        fn()
            stream.wait_stream(side)
            g_ms = []
            for i in range(args.warmup + args.steps):
                if flush is not None:
                    flush_l2()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                graph.replay()
                b.record(stream)
                torch.cuda.synchronize()
                if i >= args.warmup:
                    g_ms.append(a.elapsed_time(b))
            if not torch.equal(out, eager_out):
                raise RuntimeError("graph replay and eager launches disagree")
            if w.map_rows:
                plan.map_status(w.map_rows, map_ws)
            launches += len(g_ms) * (launches // max(args.steps, 1))
            ms_per_step, launch_mode = sum(g_ms) / len(g_ms), "one CUDA graph replay per step"
        except ccdc.CcdcError:
            raise
        except Exception as exc:            # capture refused: keep the eager number
            launch_mode = f"eager launches (graph capture failed: {type(exc).__name__})"
    # node shards: `by` is the whole job's; value shards: `by` is this rank's 1/world of the job
    value = whole_job_value(1 if sharded else world, by["iv_read"], ms_per_step)

    # ---- end to end through the host-buffer entry point ------------------
    e2e = None
    try:
        if args.skip_e2e:
            raise RuntimeError("--skip-e2e")
        if sharded or value_sharded:
            raise RuntimeError("host-buffer leg is defined for the unsharded workloads")
        import psutil

        if w.map_rows:
            # job from host buffers: the files, y and w are copied in, Map + shuffle, outputs copied out
            host_x = [t.cpu().pin_memory() for t in files_x]
            host_y = [t.cpu().pin_memory() for t in files_y]
            host_w = wvec.cpu().pin_memory()
            host_out = torch.empty(out.numel(), dtype=out.dtype, pin_memory=True)
            h2d = sum(t.numel() * t.element_size() for t in host_x + host_y) + host_w.numel() * 2
            e2e_steps = max(1, min(args.steps, 3))

            def job():
                plan.job_host(host_x, host_y, host_w, w.map_rows, host_out, files_x, files_y, wvec, part, coded, out,
                              map_ws, ws)
            job()                                                               # warm-up
            barrier()
            s2, e2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s2.record(stream)
            for _ in range(e2e_steps):
                job()
            e2.record(stream)
            barrier()
            e2e_ms = max_over_ranks(s2.elapsed_time(e2), world, dev) / e2e_steps
            e2e = {"value": whole_job_value(world, by["iv_read"], e2e_ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
                   "d2h_bytes_per_step": plan.out_bytes, "steps": e2e_steps, "ms_per_step": e2e_ms}
            assert torch.equal(host_out, out.cpu())

        else:
            # every file's Map results sit in pinned host memory once; the library copies each to the device once
            # and places its r replicas device to device (ccdc_shuffle_host_files)
            need = plan.J * w.N * w.Q * w.B * 4 + plan.out_bytes
            if psutil.virtual_memory().available > 1.5 * need * min(world, 8) + (8 << 30):
                host_values = torch.empty((plan.J * w.N, w.Q, w.B), dtype=out.dtype, pin_memory=True)
                for n, t in values_torch(plan.J * w.N, w.Q, w.B, w.dtype, dev, seed=rank_seed(rank), std=w.std):
                    host_values[n].copy_(t)
                host_out = torch.empty(out.numel(), dtype=out.dtype, pin_memory=True)
                e2e_steps = max(1, min(args.steps, 3))
                plan.shuffle_host_files(host_values, host_out, part, coded, out, ws)      # warm-up
                barrier()
                s2, e2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                s2.record(stream)
                for _ in range(e2e_steps):
                    plan.shuffle_host_files(host_values, host_out, part, coded, out, ws)
                e2.record(stream)
                barrier()
                e2e_ms = max_over_ranks(s2.elapsed_time(e2), world, dev) / e2e_steps
                e2e = {"value": whole_job_value(world, by["iv_read"], e2e_ms), "unit": UNIT,
                       "h2d_bytes_per_step": need - plan.out_bytes, "d2h_bytes_per_step": plan.out_bytes,
                       "steps": e2e_steps, "ms_per_step": e2e_ms, "entry": "ccdc_shuffle_host_files",
                       "note": "every file copied to the device once, its r replicas placed device to device"}
                assert torch.equal(host_out, out.cpu())
                del host_values
            else:
                e2e = {"value": None, "unit": UNIT, "skipped": "not enough free host memory for pinned copies"}
    except Exception as exc:            # the device-resident number must still be reported
        e2e = {"value": None, "unit": UNIT, "skipped": f"{type(exc).__name__}: {exc}"}

    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    peaks_file = ROOT / "MEASURED_PEAKS.json"
    if peaks_file.exists():
        peak, peak_kind = json.loads(peaks_file.read_text())["hbm_gbs"], "measured"
    else:
        peak, peak_kind = 6650.0, "fallback"
    # the dominant kernel of the step (the exchange between GPUs is reported beside it, not as a kernel)
    top = max((n for n in stage_ms if not n.startswith("all_gather")), key=stage_ms.get)
    NOMINAL = 8000.0                                    # GB/s, the B200's nominal HBM3e rate
    algorithmic_gbs = stage_bytes[top] / (stage_ms[top] * 1e-3) / 1e9
    others = {n: {"achieved": stage_bytes[n] / (stage_ms[n] * 1e-3) / 1e9,
                  "frac": stage_bytes[n] / (stage_ms[n] * 1e-3) / 1e9 / peak,
                  "frac_nominal": stage_bytes[n] / (stage_ms[n] * 1e-3) / 1e9 / NOMINAL, "ms_per_launch": stage_ms[n]}
              for n in stage_ms if n != top}
    traffic, traffic_kind = measured_traffic(w, top)
    # with a DRAM byte count for this kernel the achieved rate is DRAM bytes over time (bytes served
    # from L2 do not count as HBM traffic); the algorithmic rate stays beside it
    achieved = (traffic if traffic else stage_bytes[top]) / (stage_ms[top] * 1e-3) / 1e9

    cpu = None
    if world == 1 and not args.skip_cpu_baseline:
        Bs = oracle_sample_shape(w, 15.0)
        secs = time_oracle(make_oracle(w, Bs))
        bs = sample_bytes(w, Bs)
        cpu = {"value": bs["iv_read"] / secs / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": f"{w.name} with B={Bs} of {w.B} elements per value (same K, r, N, Q), one pass, "
                         f"{secs:.1f} s",
               "sample_reason": SAMPLE_REASON if Bs < w.B else "full size", **host_cpu()}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "strong" if (sharded or value_sharded) else "weak",
        "vs_baseline": None, "dtype": "f32" if w.dtype == "float32" else "i32", "data": "synthetic",
        "config": {"workload": w.name, "parallelism": f"nodes sharded over {world} GPUs, {wire['exchange']}" if sharded
                   else f"one job, every segment cut into {world} sub-ranges, one per GPU, no exchange (B={full_B})" if value_sharded
                   else f"{world} independent job(s), one per GPU", "K": w.K, "r": w.r, "N": w.N, "Q": w.Q, "B": w.B,
                   **({"wire": wire} if wire else {}),
                   "l2": (f"inputs ({input_bytes / 1e9:.1f} GB) larger than L2, no flush" if flush is None else
                          f"inputs ({input_bytes / 1e9:.3f} GB) fit in L2: 512 MB written, then 512 MB read, between steps; steps timed one by one"),
                   "step": "Map + shuffle (job time)" if w.map_rows else "shuffle", "jobs_per_gpu": plan.J,
                   "kernels": {"encode": ccdc.last_gather_kernel(), "decode": ccdc.last_decode_kernel()},
                   "launch": launch_mode, **({"eager_ms_per_step": eager_ms} if launch_mode.startswith("one") else {}),
                   **({"map_kernel": ccdc.map_last_kernel()} if w.map_rows else {}),
                   "load_per_JQT": plan.coded_bits / (plan.J * w.Q * 32 * w.B),
                   "coded_bits": plan.coded_bits, "iv_bytes_per_step": by["iv_read"],
                   "algorithmic_bytes_per_step": by["total"] + map_bytes,
                   "hbm_frac_whole_step": (by["total"] + map_bytes) / (ms_per_step * 1e-3) / 1e9 / peak,
                   "hbm_frac_whole_step_nominal": (by["total"] + map_bytes) / (ms_per_step * 1e-3) / 1e9 / NOMINAL},
        "roofline": {"bound": "hbm", "kernel": top, "achieved": achieved, "peak": peak,
                     "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                     "frac_nominal": achieved / NOMINAL, "nominal_peak": NOMINAL,
                     "achieved_kind": "DRAM bytes (ncu) / time" if traffic else "algorithmic bytes / time",
                     "algorithmic_gbs": algorithmic_gbs, "algorithmic_frac": algorithmic_gbs / peak,
                     "algorithmic_bytes": stage_bytes[top], "traffic": traffic, "traffic_kind": traffic_kind,
                     "ms_per_launch": stage_ms[top], "other_kernels": others},
        "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches, "clocks": clocks,
    }
    print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_compression(args, w):
    """Comparator: the appendix's compression-only shuffle on the same workload shape
    (unicast of pre-combined packets, no coding).  Same JSON contract; `config.scheme`
    says what ran."""
    import torch

    from paper_1805_01993_b200 import build as lib_build
    from paper_1805_01993_b200 import ccdc

    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        raise RuntimeError("the comparator runs on one GPU")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    lib_build.build_library()
    plan = ccdc.Plan(w.K, w.r, w.N, w.Q, w.B, w.dtype, compression=True)
    plan.upload()
    part = plan.alloc_partitions(dev)
    plan.fill_partitions_streaming(part, values_torch(w.N, w.Q, w.B, w.dtype, dev, seed=DEFAULT_SEED, std=w.std))
    recv = plan.alloc_decoded(dev)
    out = plan.alloc(plan.out_bytes, dev)
    m = plan.num_batches
    ln = plan.packet_elems * 4
    nfiles = [len(plan.node_files(k)) for k in range(w.K)]
    full, last = plan.files_per_batch, w.N - (m - 1) * plan.files_per_batch
    sent = sum((last if t == m - 1 else full) for k in range(w.K) for t in range(m) if t != k % m)
    iv_read = (sent + sum(nfiles)) * ln                       # batches pre-combined for others + own batch
    total = iv_read + 2 * w.K * (m - 1) * ln + plan.out_bytes   # + packets written and read + outputs
    stream = torch.cuda.current_stream()
    for _ in range(args.warmup):
        plan.compression_shuffle(part, recv, out)
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    time.sleep(0.3)
    l0 = ccdc.num_kernel_launches()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record(stream)
    for _ in range(args.steps):
        plan.compression_shuffle(part, recv, out)
    b.record(stream)
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / args.steps
    peaks_file = ROOT / "MEASURED_PEAKS.json"
    peak = json.loads(peaks_file.read_text())["hbm_gbs"] if peaks_file.exists() else 6650.0
    traffic, traffic_kind = measured_traffic(w, "k_gather(combine)+k_reduce", prefix="compression:")
    print(json.dumps({
        "metric": METRIC, "value": iv_read / (ms * 1e-3) / 1e9, "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32" if w.dtype == "float32" else "i32", "data": "synthetic",
        "config": {"workload": w.name, "scheme": "compression-only (appendix), comparator", "K": w.K, "r": w.r,
                   "N": w.N, "Q": w.Q, "B": w.B, "batches": m, "unicast_bits": plan.coded_bits,
                   "load_per_QT": plan.coded_bits / (w.Q * 32 * w.B), "iv_bytes_per_step": iv_read,
                   "algorithmic_bytes_per_step": total},
        "roofline": {"bound": "hbm", "kernel": "k_gather(combine)+k_reduce", "achieved": total / (ms * 1e-3) / 1e9,
                     "peak": peak, "unit": "GB/s", "frac": total / (ms * 1e-3) / 1e9 / peak, "frac_nominal": total / (ms * 1e-3) / 1e9 / 8000.0,
                     "achieved_kind": "algorithmic bytes / time", "traffic": traffic, "traffic_kind": traffic_kind},
        "cpu_baseline": None, "e2e": None, "gpu_launches": ccdc.num_kernel_launches() - l0,
        "clocks": sampler.stop(),
    }))


def run_load_table(args):
    """One JSON line per workload: the multicast words the fused encode really wrote (counted on the
    device: the coded buffer starts full of a mark, the partitions hold zeros, so every word written
    is a zero), times 32, beside the plan's count and the paper's loads -- Theorem 1, the plain CDC
    load and the compression-only load of Eq. (2) -- in the paper's normalisation (bits / (J Q T))."""
    import torch
    from fractions import Fraction
    from math import ceil, comb

    from paper_1805_01993_b200 import build as lib_build
    from paper_1805_01993_b200 import ccdc

    lib_build.build_library()
    torch.cuda.set_device(0)
    for name in sorted(CONFIGS):
        w = CONFIGS[name]
        plan = ccdc.Plan(w.K, w.r, w.N, w.Q, w.B, w.dtype, jobs=w.jobs)
        part = [torch.zeros(plan.partition_bytes(k) // 4, dtype=plan.torch_dtype, device="cuda") for k in range(w.K)]
        coded = torch.full((plan.coded_bytes // 4,), -0x7A5A5A5B, dtype=torch.int32, device="cuda")
        plan.encode_fused(part, coded.view(plan.torch_dtype))
        torch.cuda.synchronize()
        written = int((coded != -0x7A5A5A5B).sum().item())
        del part, coded
        torch.cuda.empty_cache()
        mu = Fraction(w.r, w.K)
        T = 32 * w.B
        # one job over all K nodes carries C(K,r)/(r+1) of the paper's jobs (a paper job has r+1 batches)
        jobs_eq = Fraction(plan.J) if w.jobs else Fraction(comb(w.K, w.r), w.r + 1)
        theorem1 = (1 - mu) * (w.r + 1) / w.r
        length = (w.Q // w.K) * w.B
        pad = Fraction(w.r * plan.segment_elems, length)      # zero extension when r does not divide the packet
        print(json.dumps({
            "workload": name, "K": w.K, "r": w.r, "N": w.N, "Q": w.Q, "B": w.B, "jobs": plan.J,
            "coded_bits_counted_on_device": written * 32, "coded_bits_plan": plan.coded_bits,
            "load_measured": float(Fraction(written * 32) / (jobs_eq * w.Q * T)),
            "load_theorem1": float(theorem1), "segment_padding_factor": float(pad),
            "measured_over_theorem1": float(Fraction(written * 32) / (jobs_eq * w.Q * T) / theorem1),
            # plain CDC on a paper job of r+1 batches of b files, (1-mu) N / (mu K) with N = (r+1) b: no combining
            "load_cdc": float(theorem1 * plan.files_per_batch),
            "load_compression_eq2": float(ceil(1 / mu) - 1 if mu < Fraction(1, 2) else 1),
            "normalisation": "bits / (J Q T); a single job over all K nodes counts as C(K,r)/(r+1) jobs"}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="cfg4", choices=sorted(CONFIGS))
    ap.add_argument("--value-elems", type=int, default=0,
                    help="shorten every value to this many elements (profiling captures on a small case)")
    ap.add_argument("--scheme", choices=["ccdc", "compression"], default="ccdc",
                    help="compression = the appendix's compression-only shuffle, as a comparator")
    ap.add_argument("--shard-nodes", action="store_true",
                    help="with N > 1 GPUs: one job, K/N logical nodes per GPU, coded rows all-gathered (strong scaling)")
    ap.add_argument("--peer-stores", action="store_true",
                    help="with --shard-nodes: the encode kernel stores its rows into every GPU's coded buffer (peer mappings) "
                         "instead of an all-gather")
    ap.add_argument("--shard-values", action="store_true",
                    help="with N > 1 GPUs: one job, every GPU owns one sub-range of every segment, no exchange (strong scaling)")
    ap.add_argument("--load-table", action="store_true",
                    help="print, per workload, the multicast bits counted on the device against the paper's loads, and exit")
    ap.add_argument("--family", type=int, choices=[0, 1], default=None,
                    help="kernel family override: 0 = loads through registers, 1 = bulk-copy pipelines (default: the planner's choice)")
    ap.add_argument("--decode-chunks", type=int, default=0, help="override the split of the fused decode's batch loop")
    ap.add_argument("--skip-e2e", action="store_true", help="leave out the host-buffer leg")
    ap.add_argument("--skip-cpu-baseline", action="store_true", help="leave out the oracle timing leg")
    args = ap.parse_args()
    w = CONFIGS[args.workload]
    if args.value_elems:
        w = w.scaled(args.value_elems)
    if args.load_table:
        run_load_table(args)
    elif args.impl == "reference":
        run_reference(args, w)
    elif args.scheme == "compression":
        run_compression(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
