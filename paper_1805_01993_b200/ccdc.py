"""Python binding of the C-ABI library ``libccdc.so`` (declared in ``include/ccdc.h``).

Argument marshalling only: every step of the shuffle runs in the library's CUDA
kernels.  PyTorch supplies device memory and streams.  The function names are
those of the C ABI; ``Plan`` wraps a ``ccdc_plan_t`` and offers the same calls as
methods taking torch tensors.

There is no fallback: if the shared library has not been built (see
``paper_1805_01993_b200.build``) importing a symbol from here raises.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

_LIB_PATH = Path(__file__).resolve().parent / "libccdc.so"
_lib = None

I32, F32 = 0, 1
OK, EINVAL, ENOMEM, ECUDA, ESIZE, ESTATE = 0, -1, -2, -3, -4, -5
MAX_K = 32

_P, _I, _LL, _SZ = ctypes.c_void_p, ctypes.c_int, ctypes.c_longlong, ctypes.c_size_t
_PP = ctypes.POINTER(ctypes.c_void_p)

# name -> (restype, argtypes); mirrors include/ccdc.h
SIGNATURES = {
    "ccdc_plan": (_I, [_I, _I, _LL, _I, _LL, _I, _PP]),
    "ccdc_plan_jobs": (_I, [_I, _I, _LL, _I, _LL, _I, _PP]),
    "ccdc_plan_jobs_gamma": (_I, [_I, _I, _LL, _I, _LL, _I, _I, _PP]),
    "ccdc_plan_compression": (_I, [_I, _I, _LL, _I, _LL, _I, _PP]),
    "ccdc_plan_sharded": (_I, [_I, _I, _LL, _I, _LL, _I, _I, _I, _I, _PP]),
    "ccdc_plan_coded_row_position": (_LL, [_P, _LL, _I]),
    "ccdc_plan_node_is_local": (_I, [_P, _I]),
    "ccdc_coded_send_bytes": (_SZ, [_P]),
    "ccdc_plan_destroy": (None, [_P]),
    "ccdc_plan_upload": (_I, [_P]),
    "ccdc_plan_kernel_family": (_I, [_P]),
    "ccdc_plan_tune_family": (_I, [_P, _I]),
    "ccdc_shuffle_status": (_I, [_P]),
    "ccdc_plan_decode_threads": (_I, [_P]),
    "ccdc_plan_decode_chunks": (_I, [_P]),
    "ccdc_plan_decode_cluster": (_I, [_P]),
    "ccdc_plan_tune_decode": (_I, [_P, _I, _I]),
    "ccdc_plan_num_jobs": (_LL, [_P]),
    "ccdc_plan_num_batches": (_LL, [_P]),
    "ccdc_plan_num_groups": (_LL, [_P]),
    "ccdc_plan_files_per_batch": (_LL, [_P]),
    "ccdc_plan_batch_files": (_LL, [_P, _LL]),
    "ccdc_plan_packet_elems": (_LL, [_P]),
    "ccdc_plan_segment_elems": (_LL, [_P]),
    "ccdc_plan_coded_row_elems": (_LL, [_P]),
    "ccdc_plan_coded_bits": (_LL, [_P]),
    "ccdc_plan_batch_of_file": (_I, [_P, _LL, _P]),
    "ccdc_plan_batch": (_I, [_P, _LL, _P, _P, _P]),
    "ccdc_plan_group": (_I, [_P, _LL, _P]),
    "ccdc_plan_group_batches": (_I, [_P, _LL, _P]),
    "ccdc_plan_node_batches": (_LL, [_P, _I, _P]),
    "ccdc_partition_bytes": (_SZ, [_P, _I]),
    "ccdc_packets_bytes": (_SZ, [_P, _I]),
    "ccdc_decoded_bytes": (_SZ, [_P, _I]),
    "ccdc_coded_bytes": (_SZ, [_P]),
    "ccdc_out_bytes": (_SZ, [_P]),
    "ccdc_workspace_bytes": (_SZ, [_P]),
    "ccdc_map_workspace_bytes": (_SZ, [_P, _LL]),
    "ccdc_map": (_I, [_P, _PP, _PP, _P, _LL, _PP, _P, _P]),
    "ccdc_map_status": (_I, [_P, _LL, _P]),
    "ccdc_map_last_kernel": (ctypes.c_char_p, []),
    "ccdc_combine": (_I, [_P, _PP, _PP, _P]),
    "ccdc_encode": (_I, [_P, _PP, _P, _P]),
    "ccdc_decode": (_I, [_P, _PP, _P, _PP, _P]),
    "ccdc_reduce": (_I, [_P, _PP, _PP, _P, _P]),
    "ccdc_encode_fused": (_I, [_P, _PP, _P, _P]),
    "ccdc_decode_reduce": (_I, [_P, _PP, _P, _P, _P, _P]),
    "ccdc_encode_fused_peers": (_I, [_P, _PP, _PP, _P]),
    "ccdc_shuffle": (_I, [_P, _PP, _P, _P, _P, _P]),
    "ccdc_static_scratch_bytes": (_SZ, []),
    "ccdc_decode_reduce_static": (_I, [_P, _PP, _P, _P, _P]),
    "ccdc_compression_shuffle": (_I, [_P, _PP, _PP, _P, _P]),
    "ccdc_shuffle_host": (_I, [_P, _PP, _P, _PP, _P, _P, _P, _P]),
    "ccdc_shuffle_host_files": (_I, [_P, _P, _P, _PP, _P, _P, _P, _P]),
    "ccdc_job_host": (_I, [_P, _PP, _PP, _P, _LL, _P, _PP, _PP, _P, _PP, _P, _P, _P, _P, _P]),
    "ccdc_value_shard": (_I, [_I, _I, _I, _LL, _I, _I, ctypes.POINTER(ctypes.c_longlong)]),
    "ccdc_value_shard_position": (_LL, [_I, _I, _I, _LL, _I, _I, _LL]),
    "ccdc_value_shard_copy": (_I, [_I, _I, _I, _LL, _I, _I, _I, _P, _P, _LL, _P]),
    "ccdc_peer_buffer_create": (_I, [_SZ, _PP, _P]),
    "ccdc_peer_buffer_open": (_I, [_P, _PP]),
    "ccdc_peer_buffer_close": (_I, [_P]),
    "ccdc_peer_buffer_destroy": (_I, [_P]),
    "ccdc_peer_buffer_copy": (_I, [_P, _P, _SZ, _P]),
    "ccdc_strerror": (ctypes.c_char_p, [_I]),
    "ccdc_last_cuda_error": (_I, []),
    "ccdc_num_kernel_launches": (_I, []),
    "ccdc_last_gather_kernel": (ctypes.c_char_p, []),
    "ccdc_last_decode_kernel": (ctypes.c_char_p, []),
}


class CcdcError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().ccdc_strerror(status).decode()
        if status == ECUDA:
            msg += f" [cudaError {lib().ccdc_last_cuda_error()}]"
        super().__init__(f"{where}: {msg} ({status})")


def lib():
    """The loaded shared library; raises if it is missing (there is no other path)."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise ImportError(f"{_LIB_PATH} not built: run `python -m paper_1805_01993_b200.build`")
        L = ctypes.CDLL(str(_LIB_PATH))
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _check(status: int, where: str):
    if status != OK:
        raise CcdcError(status, where)


def _ptr_array(tensors):
    arr = (ctypes.c_void_p * len(tensors))()
    for i, t in enumerate(tensors):
        arr[i] = t.data_ptr() if t is not None and t.numel() > 0 else None
    return arr


PEER_HANDLE_BYTES = 64


class PeerBuffer:
    """Device memory that another process can open (``ccdc_peer_buffer_*``).  Quacks like a tensor
    for the step calls (``data_ptr`` / ``numel``).  ``PeerBuffer.create(nbytes)`` allocates on the
    current device and exposes ``handle`` (64 bytes to send to the other ranks);
    ``PeerBuffer.open(handle, nbytes)`` maps another process's buffer."""

    def __init__(self, ptr, nbytes, handle, owner):
        self.ptr, self.nbytes, self.handle, self.owner = ptr, nbytes, handle, owner

    @classmethod
    def create(cls, nbytes):
        ptr = ctypes.c_void_p()
        handle = (ctypes.c_ubyte * PEER_HANDLE_BYTES)()
        _check(lib().ccdc_peer_buffer_create(nbytes, ctypes.byref(ptr), handle), "ccdc_peer_buffer_create")
        return cls(ptr.value, nbytes, bytes(handle), True)

    @classmethod
    def open(cls, handle, nbytes):
        ptr = ctypes.c_void_p()
        buf = (ctypes.c_ubyte * PEER_HANDLE_BYTES).from_buffer_copy(handle)
        _check(lib().ccdc_peer_buffer_open(buf, ctypes.byref(ptr)), "ccdc_peer_buffer_open")
        return cls(ptr.value, nbytes, bytes(handle), False)

    def data_ptr(self):
        return self.ptr

    def numel(self):
        return self.nbytes // 4

    def copy_to(self, tensor, stream=None):
        """copies the buffer into a tensor (device or pinned host) of the same size."""
        _check(lib().ccdc_peer_buffer_copy(tensor.data_ptr(), self.ptr, self.nbytes, _stream_handle(stream)),
               "ccdc_peer_buffer_copy")

    def release(self):
        if self.ptr:
            fn = lib().ccdc_peer_buffer_destroy if self.owner else lib().ccdc_peer_buffer_close
            _check(fn(self.ptr), "ccdc_peer_buffer_release")
            self.ptr = None


def value_shard(K, r, Q, B, rank, world) -> int:
    """value length of rank's shard when every segment is cut into `world` sub-ranges."""
    out = ctypes.c_longlong()
    _check(lib().ccdc_value_shard(K, r, Q, B, rank, world, ctypes.byref(out)), "ccdc_value_shard")
    return out.value


def value_shard_position(K, r, Q, B, rank, world, local_pos) -> int:
    return lib().ccdc_value_shard_position(K, r, Q, B, rank, world, local_pos)


def value_shard_copy(K, r, Q, B, rank, world, to_local, src, dst, rows, stream=None):
    """device copy between the full layout [rows][Q][B] and the rank's [rows][Q][B_local]."""
    _check(lib().ccdc_value_shard_copy(K, r, Q, B, rank, world, int(to_local), src.data_ptr(), dst.data_ptr(), rows,
                                       _stream_handle(stream)), "ccdc_value_shard_copy")


def _stream_handle(stream):
    import torch

    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


class Plan:
    """``ccdc_plan`` / ``ccdc_plan_jobs`` plus the step calls on torch tensors."""

    def __init__(self, K, r, N, Q, B, dtype, jobs: bool = False, compression: bool = False, shard=None, gamma: int = 1):
        self.K, self.r, self.N, self.Q, self.B = K, r, N, Q, B
        self.dtype = {"int32": I32, "float32": F32, I32: I32, F32: F32}[dtype]
        self.jobs = jobs
        h = ctypes.c_void_p()
        fn = lib().ccdc_plan_compression if compression else lib().ccdc_plan_jobs if jobs else lib().ccdc_plan
        self._h = None
        self.shard = shard
        if shard is not None:           # (rank, world): this GPU's share of the logical nodes
            _check(lib().ccdc_plan_sharded(K, r, N, Q, B, self.dtype, int(jobs), shard[0], shard[1], ctypes.byref(h)),
                   "ccdc_plan_sharded")
        elif gamma != 1:
            if not jobs:
                raise ValueError("gamma > 1 belongs to the J-job scheme (jobs=True)")
            _check(lib().ccdc_plan_jobs_gamma(K, r, N, Q, B, self.dtype, gamma, ctypes.byref(h)), "ccdc_plan_jobs_gamma")
        else:
            _check(fn(K, r, N, Q, B, self.dtype, ctypes.byref(h)), "ccdc_plan")
        self._h = h
        L = lib()
        self.J = L.ccdc_plan_num_jobs(h)
        self.num_batches = L.ccdc_plan_num_batches(h)
        self.num_groups = L.ccdc_plan_num_groups(h)
        self.files_per_batch = L.ccdc_plan_files_per_batch(h)
        self.packet_elems = L.ccdc_plan_packet_elems(h)
        self.segment_elems = L.ccdc_plan_segment_elems(h)
        self.coded_row_elems = L.ccdc_plan_coded_row_elems(h)
        self.coded_bits = L.ccdc_plan_coded_bits(h)

    def __del__(self):
        if getattr(self, "_h", None) and _lib is not None:
            _lib.ccdc_plan_destroy(self._h)
            self._h = None

    # ---- queries --------------------------------------------------------
    def batch_of_file(self, n):
        out = (ctypes.c_int * self.r)()
        _check(lib().ccdc_plan_batch_of_file(self._h, n, out), "ccdc_plan_batch_of_file")
        return [k for k in out if k >= 0]

    def batch(self, p):
        nodes = (ctypes.c_int * self.r)()
        f0, job = ctypes.c_longlong(), ctypes.c_longlong()
        _check(lib().ccdc_plan_batch(self._h, p, nodes, ctypes.byref(f0), ctypes.byref(job)), "ccdc_plan_batch")
        return [n for n in nodes if n >= 0], f0.value, job.value

    def group(self, g):
        out = (ctypes.c_int * (self.r + 1))()
        _check(lib().ccdc_plan_group(self._h, g, out), "ccdc_plan_group")
        return list(out)

    def group_batches(self, g):
        out = (ctypes.c_longlong * (self.r + 1))()
        _check(lib().ccdc_plan_group_batches(self._h, g, out), "ccdc_plan_group_batches")
        return list(out)

    def node_batches(self, k):
        n = lib().ccdc_plan_node_batches(self._h, k, None)
        out = (ctypes.c_longlong * max(n, 1))()
        lib().ccdc_plan_node_batches(self._h, k, out)
        return list(out)[:n]

    def partition_bytes(self, k):
        return lib().ccdc_partition_bytes(self._h, k)

    def packets_bytes(self, k):
        return lib().ccdc_packets_bytes(self._h, k)

    def decoded_bytes(self, k):
        return lib().ccdc_decoded_bytes(self._h, k)

    def node_is_local(self, k):
        return bool(lib().ccdc_plan_node_is_local(self._h, k))

    def coded_row_position(self, g, a):
        return lib().ccdc_plan_coded_row_position(self._h, g, a)

    @property
    def kernel_family(self):
        return lib().ccdc_plan_kernel_family(self._h)

    def tune_family(self, family):
        """0: loads through registers; 1: bulk-copy pipelines (before the tables are uploaded)."""
        _check(lib().ccdc_plan_tune_family(self._h, family), "ccdc_plan_tune_family")

    def shuffle_status(self):
        """after a synchronise: raises if a bounded wait inside a kernel ever ran out on this plan."""
        _check(lib().ccdc_shuffle_status(self._h), "ccdc_shuffle_status")

    @property
    def decode_threads(self):
        return lib().ccdc_plan_decode_threads(self._h)

    @property
    def decode_chunks(self):
        return lib().ccdc_plan_decode_chunks(self._h)

    @property
    def decode_cluster(self):
        return bool(lib().ccdc_plan_decode_cluster(self._h))

    def tune_decode(self, threads, chunks):
        """fixes the launch shape of the fused decode (before the tables are uploaded)."""
        _check(lib().ccdc_plan_tune_decode(self._h, threads, chunks), "ccdc_plan_tune_decode")

    @property
    def coded_send_bytes(self):
        return lib().ccdc_coded_send_bytes(self._h)

    @property
    def coded_bytes(self):
        return lib().ccdc_coded_bytes(self._h)

    @property
    def out_bytes(self):
        return lib().ccdc_out_bytes(self._h)

    @property
    def workspace_bytes(self):
        return lib().ccdc_workspace_bytes(self._h)

    def node_files(self, k):
        """global file ids in the order of node k's partition rows."""
        files = []
        for p in self.node_batches(k):
            _, f0, _ = self.batch(p)
            files.extend(range(f0, f0 + lib().ccdc_plan_batch_files(self._h, p)))
        return files

    # ---- device buffers (torch is the allocator) --------------------------
    @property
    def torch_dtype(self):
        import torch

        return torch.int32 if self.dtype == I32 else torch.float32

    def upload(self):
        _check(lib().ccdc_plan_upload(self._h), "ccdc_plan_upload")

    def alloc(self, nbytes, device="cuda"):
        import torch

        return torch.empty(max(nbytes // 4, 0), dtype=self.torch_dtype, device=device)

    def alloc_partitions(self, device="cuda"):
        """one buffer per node (empty for nodes that live on another GPU)."""
        return [self.alloc(self.partition_bytes(k) if self.node_is_local(k) else 0, device) for k in range(self.K)]

    def alloc_packets(self, device="cuda"):
        return [self.alloc(self.packets_bytes(k), device) for k in range(self.K)]

    def alloc_decoded(self, device="cuda"):
        return [self.alloc(self.decoded_bytes(k), device) for k in range(self.K)]

    def fill_partitions(self, part, values):
        """Copies Map outputs ``values`` [J*N][Q][B] (tensor on any device) into the
        node partitions: each node gets a replica of every file it stores."""
        import torch

        row = self.Q * self.B
        flat = values.reshape(-1, row)
        for k in range(self.K):
            if not self.node_is_local(k):
                continue
            idx = torch.as_tensor(self.node_files(k), dtype=torch.long, device=flat.device)
            if idx.numel():
                part[k].view(-1, row).copy_(flat.index_select(0, idx), non_blocking=False)

    def fill_partitions_streaming(self, part, file_iter, sample_index=None):
        """Places files one at a time: ``file_iter`` yields ``(n, tensor [Q][B])`` on
        the partitions' device; each is copied to the r nodes that store file n.
        With ``sample_index`` (1-D long tensor of element positions) also returns
        the sampled values ``[J*N][Q][len(sample_index)]`` on the host."""
        import torch

        row = self.Q * self.B
        where = [{n: i for i, n in enumerate(self.node_files(k))} for k in range(self.K)]
        sampled = None
        if sample_index is not None:
            sampled = torch.empty((self.J * self.N, self.Q, sample_index.numel()), dtype=self.torch_dtype)
        for n, t in file_iter:
            for k in self.batch_of_file(n):
                if not self.node_is_local(k):
                    continue
                i = where[k][n]
                part[k][i * row:(i + 1) * row].copy_(t.reshape(-1))
            if sampled is not None:
                sampled[n] = t.index_select(1, sample_index).cpu()
        return sampled

    # ---- steps ------------------------------------------------------------
    def map_workspace_bytes(self, rows):
        return lib().ccdc_map_workspace_bytes(self._h, rows)

    def map_status(self, rows, workspace):
        """after a synchronise: raises if a wait inside the Map kernel ran out."""
        _check(lib().ccdc_map_status(self._h, rows, workspace.data_ptr()), "ccdc_map_status")

    def map(self, files_x, files_y, w, rows, part, workspace, stream=None):
        """``files_x`` / ``files_y``: per node, bf16 ``[files][rows][Q*B]`` and fp32 ``[files][rows]``."""
        _check(lib().ccdc_map(self._h, _ptr_array(files_x), _ptr_array(files_y), w.data_ptr(), rows,
                              _ptr_array(part), workspace.data_ptr(), _stream_handle(stream)), "ccdc_map")

    def combine(self, part, packets, stream=None):
        _check(lib().ccdc_combine(self._h, _ptr_array(part), _ptr_array(packets), _stream_handle(stream)),
               "ccdc_combine")

    def encode(self, packets, coded, stream=None):
        _check(lib().ccdc_encode(self._h, _ptr_array(packets), coded.data_ptr(), _stream_handle(stream)),
               "ccdc_encode")

    def decode(self, packets, coded, decoded, stream=None):
        _check(lib().ccdc_decode(self._h, _ptr_array(packets), coded.data_ptr(), _ptr_array(decoded),
                                 _stream_handle(stream)), "ccdc_decode")

    def reduce(self, part, decoded, out, stream=None):
        _check(lib().ccdc_reduce(self._h, _ptr_array(part), _ptr_array(decoded), out.data_ptr(),
                                 _stream_handle(stream)), "ccdc_reduce")

    def encode_fused(self, part, coded, stream=None):
        _check(lib().ccdc_encode_fused(self._h, _ptr_array(part), coded.data_ptr(), _stream_handle(stream)),
               "ccdc_encode_fused")

    def encode_fused_peers(self, part, peer_coded, stream=None):
        """``peer_coded``: every rank's full coded buffer as addressable from this GPU."""
        _check(lib().ccdc_encode_fused_peers(self._h, _ptr_array(part), _ptr_array(peer_coded),
                                             _stream_handle(stream)), "ccdc_encode_fused_peers")

    def decode_reduce(self, part, coded, out, workspace=None, stream=None):
        ws = workspace.data_ptr() if workspace is not None and workspace.numel() else None
        _check(lib().ccdc_decode_reduce(self._h, _ptr_array(part), coded.data_ptr(), out.data_ptr(), ws,
                                        _stream_handle(stream)), "ccdc_decode_reduce")

    def compression_shuffle(self, part, recv, out, stream=None):
        _check(lib().ccdc_compression_shuffle(self._h, _ptr_array(part), _ptr_array(recv), out.data_ptr(),
                                              _stream_handle(stream)), "ccdc_compression_shuffle")

    def job_host(self, host_x, host_y, host_w, rows, host_out, dev_x, dev_y, dev_w, part, coded, out, map_workspace,
                 workspace=None, stream=None):
        """Map + shuffle from host tensors (pinned for asynchronous copies) through device staging buffers."""
        _check(lib().ccdc_job_host(self._h, _ptr_array(host_x), _ptr_array(host_y), host_w.data_ptr(), rows,
                                   host_out.data_ptr(), _ptr_array(dev_x), _ptr_array(dev_y), dev_w.data_ptr(),
                                   _ptr_array(part), coded.data_ptr(), out.data_ptr(), map_workspace.data_ptr(),
                                   workspace.data_ptr() if workspace is not None and workspace.numel() else None,
                                   _stream_handle(stream)), "ccdc_job_host")

    def shuffle_host(self, host_part, host_out, part, coded, out, workspace=None, stream=None):
        """``host_part`` / ``host_out``: CPU tensors (pinned for asynchronous copies)."""
        ws = workspace.data_ptr() if workspace is not None and workspace.numel() else None
        _check(lib().ccdc_shuffle_host(self._h, _ptr_array(host_part), host_out.data_ptr(), _ptr_array(part),
                                       coded.data_ptr(), out.data_ptr(), ws, _stream_handle(stream)),
               "ccdc_shuffle_host")

    def shuffle_host_files(self, host_values, host_out, part, coded, out, workspace=None, stream=None):
        """``host_values``: CPU tensor [J*N][Q][B], every file once (pinned for asynchronous copies)."""
        ws = workspace.data_ptr() if workspace is not None and workspace.numel() else None
        _check(lib().ccdc_shuffle_host_files(self._h, host_values.data_ptr(), host_out.data_ptr(), _ptr_array(part),
                                             coded.data_ptr(), out.data_ptr(), ws, _stream_handle(stream)),
               "ccdc_shuffle_host_files")

    def decode_reduce_static(self, part, coded, out, stream=None):
        """``ccdc_decode_reduce`` with the library's built-in scratch: no allocation."""
        _check(lib().ccdc_decode_reduce_static(self._h, _ptr_array(part), coded.data_ptr(), out.data_ptr(),
                                               _stream_handle(stream)), "ccdc_decode_reduce_static")

    def shuffle(self, part, coded, out, workspace=None, stream=None):
        ws = workspace.data_ptr() if workspace is not None and workspace.numel() else None
        _check(lib().ccdc_shuffle(self._h, _ptr_array(part), coded.data_ptr(), out.data_ptr(), ws,
                                  _stream_handle(stream)), "ccdc_shuffle")


def num_kernel_launches() -> int:
    return lib().ccdc_num_kernel_launches()


def last_gather_kernel() -> str:
    """Kernel form of this thread's most recent gather launch (combine, encode, decode, fused encode)."""
    return lib().ccdc_last_gather_kernel().decode()


def last_decode_kernel() -> str:
    """Kernel form of this thread's most recent fused decode launch."""
    return lib().ccdc_last_decode_kernel().decode()


def map_last_kernel() -> str:
    """Name of the kernel the most recent ``Plan.map`` launched."""
    return lib().ccdc_map_last_kernel().decode()
