"""ctypes front end of the CPU oracle (``ccdc_oracle.c``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the CPU-baseline leg of
the benchmark import this; the CUDA library and its Python binding never do.
The C file is compiled on first use with gcc (strict IEEE binary32, no fused
contraction) into ``oracle/_build/``.

Also here, in plain numpy: the Map of the linear-regression workload,
``g = X^T (X w - y)`` accumulated in binary64 (Section III, Map phase: an
arbitrary per-file function g_q; the gradient slices are its Q outputs).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "ccdc_oracle.c"
_BUILD = _HERE / "_build"
_LIB = _BUILD / "libccdc_oracle.so"

I32, F32 = 0, 1


def build(force: bool = False) -> Path:
    """Compile the oracle if the shared object is missing or older than its source."""
    if not force and _LIB.exists() and _LIB.stat().st_mtime >= _SRC.stat().st_mtime:
        return _LIB
    _BUILD.mkdir(exist_ok=True)
    tmp = _BUILD / f"libccdc_oracle.{os.getpid()}.so"
    cmd = ["gcc", "-std=c11", "-O2", "-fPIC", "-shared", "-ffp-contract=off", "-fno-fast-math",
           "-Wall", "-Wextra", "-o", str(tmp), str(_SRC), "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(str(build()))
    P, I, L = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64
    sig = {
        "oracle_new_single": (P, [I, I, L, I, L, I]),
        "oracle_new_paper": (P, [I, I, L, I, L, I]),
        "oracle_free": (None, [P]),
        "oracle_num_jobs": (L, [P]),
        "oracle_num_batches": (L, [P]),
        "oracle_num_rounds": (L, [P]),
        "oracle_files_per_batch": (L, [P]),
        "oracle_packet_elems": (L, [P]),
        "oracle_segment_elems": (L, [P]),
        "oracle_node_num_batches": (L, [P, I]),
        "oracle_node_num_files": (L, [P, I]),
        "oracle_batch_job": (L, [P, L]),
        "oracle_batch_first_file": (L, [P, L]),
        "oracle_recv_round": (L, [P, L, I]),
        "oracle_batch_nodes": (None, [P, L, P]),
        "oracle_round_group": (None, [P, L, P]),
        "oracle_round_batches": (None, [P, L, P]),
        "oracle_load_values": (I, [P, P]),
        "oracle_shuffle": (I, [P]),
        "oracle_redecode": (I, [P]),
        "oracle_poke_node": (None, [P, I, L, ctypes.c_uint32]),
        "oracle_poke_log": (None, [P, L, ctypes.c_uint32]),
        "oracle_coded_bits": (L, [P]),
        "oracle_copy_coded": (None, [P, P]),
        "oracle_copy_packets": (None, [P, I, P]),
        "oracle_copy_decoded": (None, [P, I, P]),
        "oracle_reduce": (I, [P, P]),
        "oracle_direct_i32": (None, [P, P, P]),
        "oracle_direct_f64": (None, [P, P, P, P]),
        "oracle_bits_uncoded": (L, [P]),
        "oracle_bits_combining": (L, [P]),
        "oracle_bits_plain_cdc": (L, [P]),
        "oracle_compression_run": (L, [I, I, L, I, L, I, P, P, P, P]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    _lib = lib
    return lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


class Oracle:
    """One instance of the scheme on K logical nodes.

    ``mode="single"``: one job spread over every size-r subset of the nodes.
    ``mode="paper"``: J = C(K, r+1) jobs, stages 1 and 2, as Section IV states it.
    Values are handed over as an array ``[J*N][Q][B]`` of int32 or float32.
    """

    def __init__(self, K, r, N, Q, B, dtype, mode="single"):
        lib = _load()
        self.K, self.r, self.N, self.Q, self.B = K, r, N, Q, B
        self.dtype = {"int32": I32, "float32": F32, I32: I32, F32: F32}[dtype]
        self.np_dtype = np.int32 if self.dtype == I32 else np.float32
        new = lib.oracle_new_paper if mode == "paper" else lib.oracle_new_single
        self._h = new(K, r, N, Q, B, self.dtype)
        if not self._h:
            raise ValueError(f"invalid parameters K={K} r={r} N={N} Q={Q} B={B} mode={mode}")
        self.J = lib.oracle_num_jobs(self._h)
        self.nbatch = lib.oracle_num_batches(self._h)
        self.nround = lib.oracle_num_rounds(self._h)
        self.b = lib.oracle_files_per_batch(self._h)
        self.len = lib.oracle_packet_elems(self._h)
        self.s = lib.oracle_segment_elems(self._h)
        self._values = None

    def __del__(self):
        if getattr(self, "_h", None):
            _load().oracle_free(self._h)
            self._h = None

    # ---- plan queries -------------------------------------------------
    def batch_nodes(self, p):
        out = np.zeros(self.r, dtype=np.int32)
        _load().oracle_batch_nodes(self._h, p, _ptr(out))
        return out.tolist()

    def batch_job(self, p):
        return _load().oracle_batch_job(self._h, p)

    def batch_files(self, p):
        f0 = _load().oracle_batch_first_file(self._h, p)
        return list(range(f0, f0 + self.b))

    def round_group(self, ro):
        out = np.zeros(self.r + 1, dtype=np.int32)
        _load().oracle_round_group(self._h, ro, _ptr(out))
        return out.tolist()

    def round_batches(self, ro):
        out = np.zeros(self.r + 1, dtype=np.int64)
        _load().oracle_round_batches(self._h, ro, _ptr(out))
        return out.tolist()

    def recv_round(self, p, k):
        return _load().oracle_recv_round(self._h, p, k)

    def node_num_files(self, k):
        return _load().oracle_node_num_files(self._h, k)

    def node_num_batches(self, k):
        return _load().oracle_node_num_batches(self._h, k)

    # ---- the scheme ---------------------------------------------------
    def load_values(self, v: np.ndarray):
        v = np.ascontiguousarray(v)
        assert v.dtype == self.np_dtype, (v.dtype, self.np_dtype)
        assert v.shape == (self.J * self.N, self.Q, self.B), v.shape
        self._values = v
        rc = _load().oracle_load_values(self._h, _ptr(v))
        if rc:
            raise MemoryError(f"oracle_load_values: {rc}")

    def shuffle(self):
        rc = _load().oracle_shuffle(self._h)
        if rc:
            raise RuntimeError(f"oracle_shuffle failed: {rc}")

    def shuffle_status(self):
        """as ``shuffle`` but returns the oracle's status code instead of raising."""
        return _load().oracle_shuffle(self._h)

    def redecode_status(self):
        """decode every round again from the broadcast log as it stands."""
        return _load().oracle_redecode(self._h)

    def poke_node(self, k, word, mask):
        """fault planting: flip bits of one word of node k's private memory."""
        _load().oracle_poke_node(self._h, k, word, mask)

    def poke_log(self, word, mask):
        """fault planting: flip bits of one word of the broadcast log."""
        _load().oracle_poke_log(self._h, word, mask)

    @property
    def coded_bits(self):
        return _load().oracle_coded_bits(self._h)

    def coded(self):
        out = np.zeros((self.nround, self.r + 1, self.s), dtype=np.uint32)
        _load().oracle_copy_coded(self._h, _ptr(out))
        return out

    def packets(self, k):
        n = self.node_num_batches(k) * (self.K - self.r)
        out = np.zeros((n, self.len), dtype=np.uint32)
        _load().oracle_copy_packets(self._h, k, _ptr(out))
        return out

    def decoded(self, k):
        n = sum(1 for ro in range(self.nround) if k in self.round_group(ro))
        out = np.zeros((n, self.len), dtype=np.uint32)
        _load().oracle_copy_decoded(self._h, k, _ptr(out))
        return out

    def reduce(self):
        out = np.zeros((self.J * self.Q, self.B), dtype=np.uint32)
        rc = _load().oracle_reduce(self._h, _ptr(out))
        if rc:
            raise RuntimeError(f"oracle_reduce failed: {rc}")
        return out.view(self.np_dtype)

    def run(self, v):
        """load, shuffle, reduce; returns the outputs [J*Q][B]."""
        self.load_values(v)
        self.shuffle()
        return self.reduce()

    # ---- direct evaluation of Eq. (1) ---------------------------------
    def direct(self, v=None):
        v = self._values if v is None else np.ascontiguousarray(v)
        if self.dtype == I32:
            out = np.zeros((self.J * self.Q, self.B), dtype=np.uint32)
            _load().oracle_direct_i32(self._h, _ptr(v), _ptr(out))
            return out.view(np.int32)
        s = np.zeros((self.J * self.Q, self.B), dtype=np.float64)
        a = np.zeros_like(s)
        _load().oracle_direct_f64(self._h, _ptr(v), _ptr(s), _ptr(a))
        return s, a

    # ---- comparator bit counts on the same placement -------------------
    @property
    def bits_uncoded(self):
        return _load().oracle_bits_uncoded(self._h)

    @property
    def bits_combining(self):
        return _load().oracle_bits_combining(self._h)

    @property
    def bits_plain_cdc(self):
        return _load().oracle_bits_plain_cdc(self._h)


def compression_only(K, r, N, Q, B, dtype, v):
    """The compression-only scheme of the paper's appendix (one job, mu = r/K).

    Returns ``(out [Q][B], recv [K][m-1][len], bits, files_at_node [K])``.
    """
    lib = _load()
    dt = {"int32": I32, "float32": F32}[dtype]
    npdt = np.int32 if dt == I32 else np.float32
    v = np.ascontiguousarray(v)
    assert v.dtype == npdt and v.shape == (N, Q, B)
    m = -(-K // r)
    ln = (Q // K) * B
    out = np.zeros((Q, B), dtype=np.uint32)
    recv = np.zeros((K, m - 1, ln), dtype=np.uint32)
    files = np.zeros(K, dtype=np.int64)
    bits = lib.oracle_compression_run(K, r, N, Q, B, dt, _ptr(v), _ptr(out), _ptr(recv), _ptr(files))
    if bits < 0:
        raise ValueError(f"invalid parameters K={K} r={r} N={N} Q={Q} B={B}")
    return out.view(npdt), recv, bits, files.tolist()


def map_linear_regression(X: np.ndarray, w: np.ndarray, y: np.ndarray, Q: int) -> np.ndarray:
    """Map of one file for the linear-regression workload.

    ``X`` [m][d] (values exactly representable in bfloat16, given as float32),
    ``w`` [d] (likewise), ``y`` [m] float32.  Returns the Q intermediate values
    ``[Q][d/Q]`` = the partial gradient ``X^T (X w - y)`` cut into Q contiguous
    slices, evaluated in binary64 and rounded once to float32.
    """
    Xd = X.astype(np.float64)
    u = Xd @ w.astype(np.float64) - y.astype(np.float64)
    g = Xd.T @ u
    return g.astype(np.float32).reshape(Q, -1)
