"""Seeded synthetic inputs: Map outputs v_{q,n} and linear-regression files.

This module holds no part of the method (no placement, no sums, no coding): it
only draws numbers.  Both the CUDA path and the CPU checks are fed from here, so
that they see identical values.

Two generators:

* ``values_numpy`` -- host side, counter based: the numbers of value (file n,
  function q) come from ``numpy``'s Philox bit generator keyed with
  ``(seed, n * 2**20 + q)``, so any (n, q) can be regenerated alone.
* ``values_torch`` -- device side, for sizes that are too large to draw on the
  host: one seeded ``torch.Generator`` stream per file.

The five named workloads are the shapes the method is evaluated on:
  cfg1  K=4  r=2 N=12   Q=4  B=256      int32 uniform over all 2**32 words
  cfg2  K=10 r=3 N=480  Q=10 B=4096     fp32 N(0,1)
  cfg3  K=16 r=4 N=1820 Q=16 B=16384    fp32 N(0,1)
  cfg4  K=20 r=2 N=190  Q=20 B=1280000  fp32 N(0, variance 1e-3): a 25.6 M-entry
        gradient per file cut into 20 slices
  cfg5  K=8  r=3 N=112  Q=8  B=1024     fp32, produced by the linear-regression
        Map from files X_n (512 x 8192, bf16-representable), y_n, and w
plus ``jobs20``: the paper's J = C(K, r+1) parallel jobs at K=20, r=2 (1140 jobs of 21
files each, B=10240), sized like cfg4.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np

DEFAULT_SEED = 20180501


@dataclass(frozen=True)
class Workload:
    name: str
    K: int
    r: int
    N: int
    Q: int
    B: int
    dtype: str            # "int32" | "float32"
    std: float = 1.0      # standard deviation of the normal draws (fp32 only)
    map_rows: int = 0     # linear-regression workload: rows m of X_n (0 = no Map)
    jobs: bool = False    # the scheme as stated for J = C(K, r+1) jobs (stages 1 and 2); N is per job

    @property
    def map_cols(self) -> int:
        return self.Q * self.B

    def scaled(self, B: int) -> "Workload":
        """Same structure with a different value length."""
        return replace(self, name=f"{self.name}[B={B}]", B=B)


CONFIGS = {
    "cfg1": Workload("cfg1", 4, 2, 12, 4, 256, "int32"),
    "cfg2": Workload("cfg2", 10, 3, 480, 10, 4096, "float32"),
    "cfg3": Workload("cfg3", 16, 4, 1820, 16, 16384, "float32"),
    "cfg4": Workload("cfg4", 20, 2, 190, 20, 1280000, "float32", std=float(np.sqrt(1e-3))),
    "cfg5": Workload("cfg5", 8, 3, 112, 8, 1024, "float32", map_rows=512),
    # the paper's own multi-job setting at the scale of cfg4: J = C(20,3) = 1140 jobs of 21 files,
    # 2394 files (1.96 GB) per node, load (1-mu)(mu K+1)/(mu K) = 1.35
    "jobs20": Workload("jobs20", 20, 2, 21, 20, 10240, "float32", std=float(np.sqrt(1e-3)), jobs=True),
}


def _rng(seed: int, n: int, q: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed, n * (1 << 20) + q]))


def values_numpy(N: int, Q: int, B: int, dtype: str, seed: int = DEFAULT_SEED,
                 std: float = 1.0) -> np.ndarray:
    """Map outputs ``[N][Q][B]`` drawn on the host, one Philox stream per (n, q)."""
    if dtype == "int32":
        out = np.empty((N, Q, B), dtype=np.uint32)
        for n in range(N):
            for q in range(Q):
                out[n, q] = _rng(seed, n, q).integers(0, 1 << 32, size=B, dtype=np.uint32)
        return out.view(np.int32)
    out = np.empty((N, Q, B), dtype=np.float32)
    for n in range(N):
        for q in range(Q):
            out[n, q] = _rng(seed, n, q).standard_normal(B, dtype=np.float32) * np.float32(std)
    return out


def values_torch(N: int, Q: int, B: int, dtype: str, device, seed: int = DEFAULT_SEED,
                 std: float = 1.0, files=None):
    """Generator of ``(n, tensor [Q][B])`` drawn on ``device``, one seeded stream per file."""
    import torch

    gen = torch.Generator(device=device)
    for n in (range(N) if files is None else files):
        gen.manual_seed(seed * 1000003 + n)
        if dtype == "int32":
            t = torch.randint(-(1 << 31), 1 << 31, (Q, B), generator=gen, device=device,
                              dtype=torch.int64).to(torch.int32)
        else:
            t = torch.randn((Q, B), generator=gen, device=device, dtype=torch.float32)
            if std != 1.0:
                t *= std
        yield n, t


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """float32 array rounded to the nearest bfloat16 (ties to even), kept as float32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """upper 16 bits of float32 values that are already bfloat16-representable."""
    return (np.ascontiguousarray(x, dtype=np.float32).view(np.uint32) >> 16).astype(np.uint16)


def regression_files(N: int, rows: int, cols: int, seed: int = DEFAULT_SEED, noise: float = 0.01):
    """Linear-regression files: ``X`` [N][rows][cols] (bf16-representable float32),
    ``y`` [N][rows] float32 with ``y_n = X_n w* + noise * N(0,1)`` evaluated in
    binary64, and the current iterate ``w`` [cols] (bf16-representable float32)."""
    g = np.random.Generator(np.random.Philox(key=[seed, (1 << 62) + 1]))
    w_star = g.standard_normal(cols, dtype=np.float32)
    w = round_to_bf16(g.standard_normal(cols, dtype=np.float32))
    X = np.empty((N, rows, cols), dtype=np.float32)
    y = np.empty((N, rows), dtype=np.float32)
    for n in range(N):
        gn = np.random.Generator(np.random.Philox(key=[seed, (1 << 62) + 2 + n]))
        X[n] = round_to_bf16(gn.standard_normal((rows, cols), dtype=np.float32))
        e = gn.standard_normal(rows)
        y[n] = (X[n].astype(np.float64) @ w_star.astype(np.float64) + noise * e).astype(np.float32)
    return X, y, w
