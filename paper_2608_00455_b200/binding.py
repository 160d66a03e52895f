"""Thin ctypes binding of libdte.so: argument marshalling only.

Every step of the path runs in the CUDA library; torch is used for device
memory and streams.  The names mirror the C ABI (include/dte.h).  There is no
fallback: importing works without a GPU (so that symbols can be checked), but
every compute call needs the library and a CUDA device and raises otherwise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import numpy as np
import torch

from . import build as _build

DTE_OK = 0
DTE_DEV_OVERFLOW, DTE_DEV_BOUNDS, DTE_DEV_TIMEOUT, DTE_DEV_CORRUPT = 1, 2, 4, 8
DTE_CHUNK_PLAIN, DTE_CHUNK_BYTE_PLANES, DTE_CHUNK_DELTA_PLANES = 0, 1, 2
DTE_CHUNK_MAGIC, DTE_CHUNK_HEADER_BYTES, DTE_CHUNK_MAX_ENTRIES = 0x43455444, 32, 1 << 20

SYMBOLS = [
    "dte_layout_create", "dte_layout_destroy", "dte_layout_num_lists", "dte_layout_num_elements",
    "dte_layout_host_workspace_bytes", "dte_derive_constants", "dte_extract_delta", "dte_apply",
    "dte_extract_delta_host", "dte_status_string", "dte_last_error", "dte_layout_last_launch",
    "dte_extract_delta_static", "dte_extract_delta_groups", "dte_layout_num_groups",
    "dte_op_counts", "dte_layout_num_ops", "dte_chunk_count_bound", "dte_chunk_bytes_bound",
    "dte_pack_chunks", "dte_unpack_chunks", "dte_apply_canonical", "dte_extract_delta_push",
    "dte_push_wait", "dte_layout_num_receivers", "dte_layout_receiver_num_ops",
]


class TensorDesc(C.Structure):
    _fields_ = [("shape", C.c_uint64 * 2), ("ndim", C.c_uint32), ("group", C.c_uint32)]


class ShardDesc(C.Structure):
    _fields_ = [("numel", C.c_uint64), ("receiver", C.c_uint32), ("reserved", C.c_uint32)]


class OpDesc(C.Structure):
    _fields_ = [("src_tensor", C.c_uint32), ("dst_shard", C.c_uint32),
                ("src_origin", C.c_uint64 * 2), ("extent", C.c_uint64 * 2),
                ("dst_base", C.c_uint64), ("dst_ld", C.c_uint64), ("dst_origin", C.c_uint64 * 2)]


_OP_DTYPE = np.dtype([("src_tensor", np.uint32), ("dst_shard", np.uint32), ("src_origin", np.uint64, (2,)),
                      ("extent", np.uint64, (2,)), ("dst_base", np.uint64), ("dst_ld", np.uint64),
                      ("dst_origin", np.uint64, (2,))])


class DeltaStruct(C.Structure):
    _fields_ = [("offsets", C.c_void_p), ("values", C.c_void_p), ("capacity", C.c_uint64),
                ("list_ptr", C.c_void_p), ("counters", C.c_void_p)]


class PushTargetStruct(C.Structure):
    _fields_ = [("offsets", C.c_void_p), ("values", C.c_void_p), ("capacity", C.c_uint64),
                ("list_ptr", C.c_void_p), ("op_counts", C.c_void_p), ("status", C.c_void_p)]


class DteError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"dte status {status}: {msg}")
        self.status = status


_lib = None


def library_path() -> str:
    return _build.LIB


def lib() -> C.CDLL:
    """Loads libdte.so, building it first if the sources are newer."""
    global _lib
    if _lib is None:
        path = _build.build()
        L = C.CDLL(path)
        vp, u64, i64, dbl = C.c_void_p, C.c_uint64, C.c_int64, C.c_double
        L.dte_layout_create.argtypes = [vp, C.c_size_t, vp, C.c_size_t, vp, C.c_size_t, C.c_int, C.POINTER(vp)]
        L.dte_layout_create.restype = C.c_int
        L.dte_layout_destroy.argtypes = [vp]
        L.dte_layout_destroy.restype = None
        L.dte_layout_num_lists.argtypes = [vp]
        L.dte_layout_num_lists.restype = C.c_size_t
        L.dte_layout_num_elements.argtypes = [vp]
        L.dte_layout_num_elements.restype = u64
        L.dte_layout_host_workspace_bytes.argtypes = [vp]
        L.dte_layout_host_workspace_bytes.restype = u64
        L.dte_derive_constants.argtypes = [i64, dbl, dbl, dbl, dbl, dbl, vp]
        L.dte_derive_constants.restype = C.c_int
        L.dte_extract_delta.argtypes = [vp, vp, vp, vp, i64, dbl, dbl, dbl, dbl, dbl, vp, vp]
        L.dte_extract_delta.restype = C.c_int
        L.dte_extract_delta_static.argtypes = [vp, vp, vp, vp, i64, dbl, dbl, dbl, dbl, dbl, vp, vp]
        L.dte_extract_delta_static.restype = C.c_int
        L.dte_extract_delta_groups.argtypes = [vp, vp, vp, vp, i64, dbl, dbl, dbl, vp, vp, C.c_size_t, vp, vp]
        L.dte_extract_delta_groups.restype = C.c_int
        L.dte_layout_num_groups.argtypes = [vp]
        L.dte_layout_num_groups.restype = C.c_size_t
        L.dte_op_counts.argtypes = [vp, vp, vp, vp]
        L.dte_op_counts.restype = C.c_int
        L.dte_layout_num_ops.argtypes = [vp]
        L.dte_layout_num_ops.restype = C.c_size_t
        L.dte_chunk_count_bound.argtypes = [C.c_size_t, u64, C.c_uint32]
        L.dte_chunk_count_bound.restype = u64
        L.dte_chunk_bytes_bound.argtypes = [C.c_size_t, u64, C.c_uint32, C.c_uint32]
        L.dte_chunk_bytes_bound.restype = u64
        L.dte_pack_chunks.argtypes = [vp, vp, C.c_uint32, C.c_uint32, vp, u64, vp, u64, vp, vp]
        L.dte_pack_chunks.restype = C.c_int
        L.dte_unpack_chunks.argtypes = [vp, vp, u64, vp, u64, vp, vp]
        L.dte_unpack_chunks.restype = C.c_int
        L.dte_extract_delta_push.argtypes = [vp, vp, vp, vp, i64, dbl, dbl, dbl, dbl, dbl, vp, vp, C.c_size_t, u64, vp]
        L.dte_extract_delta_push.restype = C.c_int
        L.dte_push_wait.argtypes = [vp, u64, C.c_uint32, vp, C.c_int, vp]
        L.dte_push_wait.restype = C.c_int
        L.dte_layout_num_receivers.argtypes = [vp]
        L.dte_layout_num_receivers.restype = C.c_size_t
        L.dte_layout_receiver_num_ops.argtypes = [vp, C.c_uint32]
        L.dte_layout_receiver_num_ops.restype = C.c_size_t
        L.dte_apply_canonical.argtypes = [vp, vp, vp, vp]
        L.dte_apply_canonical.restype = C.c_int
        L.dte_apply.argtypes = [vp, vp, vp, vp]
        L.dte_apply.restype = C.c_int
        L.dte_extract_delta_host.argtypes = [vp, vp, vp, vp, i64, dbl, dbl, dbl, dbl, dbl, vp, u64,
                                             vp, vp, vp, vp, vp, vp]
        L.dte_extract_delta_host.restype = C.c_int
        L.dte_status_string.argtypes = [C.c_int]
        L.dte_status_string.restype = C.c_char_p
        L.dte_last_error.argtypes = []
        L.dte_last_error.restype = C.c_char_p
        L.dte_layout_last_launch.argtypes = [vp, vp]
        L.dte_layout_last_launch.restype = None
        _lib = L
    return _lib


def _check(status: int) -> None:
    if status != DTE_OK:
        L = lib()
        msg = L.dte_last_error().decode() or L.dte_status_string(status).decode()
        raise DteError(status, msg)


def _require_cuda() -> None:
    if not torch.cuda.is_available():
        raise RuntimeError("the delta-transfer path needs a CUDA device; there is no CPU fallback")


def dte_derive_constants(step, lr, beta1, beta2, eps, wd) -> np.ndarray:
    out = np.zeros(5, np.float32)
    _check(lib().dte_derive_constants(int(step), float(lr), float(beta1), float(beta2), float(eps),
                                      float(wd), out.ctypes.data))
    return out


def _ptr_table(tensors: Sequence[Optional[torch.Tensor]], dtype, device=None):
    arr = (C.c_void_p * max(1, len(tensors)))()
    for i, t in enumerate(tensors):
        if t is None:
            arr[i] = None
            continue
        assert t.dtype == dtype and t.is_contiguous(), "tensor dtype / contiguity"
        if device is not None:
            assert t.device == device, f"tensor on {t.device}, layout on {device}"
        arr[i] = t.data_ptr()
    return arr


class Delta:
    """Caller-owned device buffers of one extract result (see dte_delta in dte.h)."""

    def __init__(self, n_lists: int, capacity: int, device):
        dev = torch.device(device)
        self.capacity = int(capacity)
        self.n_lists = int(n_lists)
        self.offsets = torch.empty(max(1, self.capacity), dtype=torch.int32, device=dev)   # uint32 bits
        self.values = torch.empty(max(1, self.capacity), dtype=torch.int16, device=dev)    # bf16 bits
        self.list_ptr = torch.zeros(self.n_lists + 1, dtype=torch.int64, device=dev)
        self.counters = torch.zeros(4, dtype=torch.int64, device=dev)
        self.struct = DeltaStruct(self.offsets.data_ptr(), self.values.data_ptr(), self.capacity,
                                  self.list_ptr.data_ptr(), self.counters.data_ptr())

    @classmethod
    def wrap(cls, list_ptr, offsets: torch.Tensor, values: torch.Tensor) -> "Delta":
        """A delta around lists that already exist on the device (received from a peer or decoded
        from chunks): `list_ptr` host array of n_lists + 1 boundaries, `offsets` int32 / `values`
        int16 device tensors holding list_ptr[-1] entries.  No copy of the entries."""
        lp = np.ascontiguousarray(list_ptr, dtype=np.uint64)
        total = int(lp[-1])
        assert offsets.dtype == torch.int32 and values.dtype == torch.int16
        assert offsets.is_contiguous() and values.is_contiguous() and offsets.device == values.device
        assert offsets.numel() >= total and values.numel() >= total
        self = cls.__new__(cls)
        dev = offsets.device
        self.capacity, self.n_lists = total, lp.size - 1
        # zero-entry deltas still need valid pointers
        self.offsets = offsets if total else torch.empty(1, dtype=torch.int32, device=dev)
        self.values = values if total else torch.empty(1, dtype=torch.int16, device=dev)
        self.list_ptr = torch.from_numpy(lp.astype(np.int64)).to(dev)
        self.counters = torch.tensor([total, 0, 0, 0], dtype=torch.int64, device=dev)
        self.struct = DeltaStruct(self.offsets.data_ptr(), self.values.data_ptr(), self.capacity,
                                  self.list_ptr.data_ptr(), self.counters.data_ptr())
        return self

    # host views (synchronise)
    def total(self) -> int:
        return int(self.counters[0].item())

    def status_bits(self) -> int:
        return int(self.counters[2].item())

    def to_host(self):
        lp = self.list_ptr.cpu().numpy().astype(np.uint64)
        n = min(int(lp[-1]), self.capacity)
        off = self.offsets[:n].cpu().numpy().view(np.uint32)
        val = self.values[:n].cpu().numpy().view(np.uint16)
        return lp, off, val


class Layout:
    """dte_layout handle built from a plan (tensor shapes, shard sizes, operation rows)."""

    def __init__(self, tensor_shapes, shard_numels, ops, device=0, shard_receivers=None, tensor_groups=None):
        _require_cuda()
        self.device = torch.device("cuda", device) if isinstance(device, int) else torch.device(device)
        shapes = [(int(s[0]), int(s[1]) if len(s) > 1 else 1) for s in tensor_shapes]
        self.tensor_shapes = shapes
        self.shard_numels = [int(n) for n in shard_numels]
        T = (TensorDesc * max(1, len(shapes)))()
        for i, (a, b) in enumerate(shapes):
            T[i].shape[0], T[i].shape[1] = a, b
            T[i].ndim = 1 if b == 1 else 2
            T[i].group = int(tensor_groups[i]) if tensor_groups is not None else 0
        S = (ShardDesc * max(1, len(self.shard_numels)))()
        for k, n in enumerate(self.shard_numels):
            S[k].numel = n
            S[k].receiver = int(shard_receivers[k]) if shard_receivers is not None else 0
        ops = np.asarray(ops, dtype=np.int64).reshape(-1, 10)
        # dte_op_desc as a numpy record array (same layout as OpDesc): a plan can have millions of rows
        O = np.zeros(max(1, ops.shape[0]), dtype=_OP_DTYPE)
        if ops.shape[0]:
            O["src_tensor"], O["dst_shard"] = ops[:, 0], ops[:, 1]
            O["src_origin"], O["extent"] = ops[:, 2:4], ops[:, 4:6]
            O["dst_base"], O["dst_ld"], O["dst_origin"] = ops[:, 6], ops[:, 7], ops[:, 8:10]
        assert O.dtype.itemsize == C.sizeof(OpDesc)
        h = C.c_void_p()
        _check(lib().dte_layout_create(T, len(shapes), S, len(self.shard_numels), O.ctypes.data, ops.shape[0],
                                       self.device.index or 0, C.byref(h)))
        self._h = h

    @classmethod
    def from_plan(cls, plan, device=0, tensor_groups=None):
        return cls(plan.tensor_shapes, plan.shard_numels, plan.ops_array(), device, plan.shard_receivers,
                   tensor_groups)

    def close(self):
        if getattr(self, "_h", None):
            lib().dte_layout_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def num_lists(self) -> int:
        return int(lib().dte_layout_num_lists(self._h))

    @property
    def num_groups(self) -> int:
        return int(lib().dte_layout_num_groups(self._h))

    @property
    def num_receivers(self) -> int:
        return int(lib().dte_layout_num_receivers(self._h))

    def receiver_num_ops(self, receiver: int) -> int:
        return int(lib().dte_layout_receiver_num_ops(self._h, int(receiver)))

    @property
    def num_elements(self) -> int:
        return int(lib().dte_layout_num_elements(self._h))

    @property
    def host_workspace_bytes(self) -> int:
        return int(lib().dte_layout_host_workspace_bytes(self._h))

    def last_launch(self):
        out = (C.c_uint64 * 3)()
        lib().dte_layout_last_launch(self._h, out)
        return dict(tiles=int(out[0]), ctas=int(out[1]), kernels=int(out[2]))

    def new_delta(self, capacity: int) -> Delta:
        return Delta(self.num_lists, capacity, self.device)

    def source_tables(self, theta, m, v):
        """Marshal the three pointer tables once (reusable across calls)."""
        return (_ptr_table(theta, torch.float32, self.device), _ptr_table(m, torch.float32, self.device),
                _ptr_table(v, torch.float32, self.device))

    def shard_table(self, shards):
        tabs = []
        for s in shards:
            assert s is None or s.dtype in (torch.bfloat16, torch.int16)
            tabs.append(s)
        arr = (C.c_void_p * max(1, len(tabs)))()
        for i, t in enumerate(tabs):
            arr[i] = None if t is None else t.data_ptr()
            assert t is None or (t.is_contiguous() and t.device == self.device)
        return arr


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


def dte_extract_delta(layout: Layout, tables, step, lr, beta1, beta2, eps, wd, delta: Delta,
                      stream=None) -> None:
    """Enqueue one extract.  `tables` = layout.source_tables(theta, m, v)."""
    th, mm, vv = tables
    _check(lib().dte_extract_delta(layout._h, th, mm, vv, int(step), float(lr), float(beta1),
                                   float(beta2), float(eps), float(wd), C.byref(delta.struct),
                                   _stream_ptr(stream)))


def dte_extract_delta_groups(layout: Layout, tables, step, beta1, beta2, eps, lr, wd, delta: Delta,
                             stream=None) -> None:
    """Extract with one (lr, wd) pair per parameter group (sequences of equal length)."""
    th, mm, vv = tables
    n = len(lr)
    assert len(wd) == n
    lr_a = (C.c_double * n)(*[float(x) for x in lr])
    wd_a = (C.c_double * n)(*[float(x) for x in wd])
    _check(lib().dte_extract_delta_groups(layout._h, th, mm, vv, int(step), float(beta1), float(beta2),
                                          float(eps), lr_a, wd_a, n, C.byref(delta.struct),
                                          _stream_ptr(stream)))


STATIC_MAX_TILES = 65536
STATIC_MAX_CAPACITY = 2097152


def dte_extract_delta_static(layout: Layout, tables, step, lr, beta1, beta2, eps, wd, delta: Delta,
                             stream=None) -> None:
    """dte_extract_delta for callers that must not allocate device memory.

    Same arguments and results; the call's scratch is a fixed array inside the library, so
    it is limited to layouts of at most STATIC_MAX_TILES tiles and deltas of at most
    STATIC_MAX_CAPACITY entries (DteError with status 3 beyond that), and two calls that can
    overlap on one GPU must not be issued.  See dte_extract_delta_static in include/dte.h.
    """
    th, mm, vv = tables
    _check(lib().dte_extract_delta_static(layout._h, th, mm, vv, int(step), float(lr), float(beta1),
                                          float(beta2), float(eps), float(wd), C.byref(delta.struct),
                                          _stream_ptr(stream)))


class PushTarget:
    """Landing buffers of one receiver for dte_extract_delta_push (see dte_push_target in dte.h).
    On one GPU they are ordinary allocations; across GPUs the receiver allocates them and the sender
    reaches them through peer access."""

    def __init__(self, n_lists: int, capacity: int, n_ops: int, device):
        dev = torch.device(device)
        self.capacity, self.n_lists = int(capacity), int(n_lists)
        self.offsets = torch.empty(max(1, self.capacity), dtype=torch.int32, device=dev)
        self.values = torch.empty(max(1, self.capacity), dtype=torch.int16, device=dev)
        self.list_ptr = torch.zeros(self.n_lists + 1, dtype=torch.int64, device=dev)
        self.op_counts = torch.zeros(max(1, int(n_ops)), dtype=torch.int64, device=dev)
        self.n_ops = int(n_ops)
        self.status = torch.zeros(4, dtype=torch.int64, device=dev)
        self.counters = torch.zeros(4, dtype=torch.int64, device=dev)     # filled by dte_push_wait

    def struct(self) -> PushTargetStruct:
        return PushTargetStruct(self.offsets.data_ptr(), self.values.data_ptr(), self.capacity,
                                self.list_ptr.data_ptr(), self.op_counts.data_ptr(), self.status.data_ptr())

    def delta(self) -> Delta:
        """The receiver's share as a dte_delta (no copy); counters are those dte_push_wait fills."""
        d = Delta.__new__(Delta)
        d.capacity, d.n_lists = self.capacity, self.n_lists
        d.offsets, d.values, d.list_ptr, d.counters = self.offsets, self.values, self.list_ptr, self.counters
        d.struct = DeltaStruct(d.offsets.data_ptr(), d.values.data_ptr(), d.capacity, d.list_ptr.data_ptr(),
                               d.counters.data_ptr())
        return d


def dte_extract_delta_push(layout: Layout, tables, step, lr, beta1, beta2, eps, wd, delta: Delta,
                           targets: Sequence[Optional[PushTarget]], epoch: int, stream=None) -> None:
    """Extract into `delta` and deliver every receiver's share into targets[receiver] (None: skip)."""
    th, mm, vv = tables
    arr = (PushTargetStruct * max(1, len(targets)))()
    for r, t in enumerate(targets):
        if t is not None:
            arr[r] = t.struct()
    _check(lib().dte_extract_delta_push(layout._h, th, mm, vv, int(step), float(lr), float(beta1), float(beta2),
                                        float(eps), float(wd), C.byref(delta.struct), arr, len(targets),
                                        int(epoch), _stream_ptr(stream)))


def dte_push_wait(target: PushTarget, epoch: int, timeout_ms: int = 1000, stream=None) -> None:
    """Receiver side: wait (bounded) for `epoch` in the target's status block, then fill
    target.counters so that dte_apply(layout, target.delta(), ...) can follow on the same stream."""
    _check(lib().dte_push_wait(target.status.data_ptr(), int(epoch), int(timeout_ms), target.counters.data_ptr(),
                               target.status.device.index or 0, _stream_ptr(stream)))


def dte_op_counts(layout: Layout, delta: Delta, stream=None) -> torch.Tensor:
    """Entry count of every operation of the plan (plan order, zeros included), on the device."""
    n = int(lib().dte_layout_num_ops(layout._h))
    counts = torch.zeros(max(1, n), dtype=torch.int64, device=layout.device)
    _check(lib().dte_op_counts(layout._h, C.byref(delta.struct), counts.data_ptr(), _stream_ptr(stream)))
    return counts[:n]


def dte_apply(layout: Layout, delta: Delta, shard_table, stream=None) -> None:
    """Enqueue one apply.  `shard_table` = layout.shard_table(shards)."""
    _check(lib().dte_apply(layout._h, C.byref(delta.struct), shard_table, _stream_ptr(stream)))


# dte_chunk_ref as a numpy record: {byte_offset u64, list u32, first_entry u32}
CHUNK_REF_DTYPE = np.dtype([("byte_offset", np.uint64), ("list", np.uint32), ("first_entry", np.uint32)])


class ChunkStream:
    """Caller-owned device buffers of one serialised delta (see dte_pack_chunks in dte.h)."""

    def __init__(self, n_lists: int, entries: int, chunk_entries: int, fmt: int, device):
        L = lib()
        dev = torch.device(device)
        self.chunk_entries, self.format = int(chunk_entries), int(fmt)
        self.directory_capacity = int(L.dte_chunk_count_bound(n_lists, int(entries), self.chunk_entries))
        self.stream_capacity = int(L.dte_chunk_bytes_bound(n_lists, int(entries), self.chunk_entries, self.format))
        self.stream = torch.empty(max(16, self.stream_capacity), dtype=torch.uint8, device=dev)
        # 16 bytes per directory entry, one entry more than chunks
        self.directory = torch.zeros(2 * (self.directory_capacity + 1), dtype=torch.int64, device=dev)
        self.info = torch.zeros(4, dtype=torch.int64, device=dev)

    def to_host(self):
        """(stream uint8[bytes], directory records[n_chunks + 1], info) - synchronises."""
        info = self.info.cpu().numpy().astype(np.uint64)
        if int(info[2]) & DTE_DEV_OVERFLOW:
            return np.zeros(0, np.uint8), np.zeros(0, CHUNK_REF_DTYPE), info
        n_chunks, nbytes = int(info[0]), int(info[1])
        stream = self.stream[:nbytes].cpu().numpy()
        directory = self.directory[:2 * (n_chunks + 1)].cpu().numpy().view(CHUNK_REF_DTYPE)
        return stream, directory, info


def dte_pack_chunks(layout: Layout, delta: Delta, out: ChunkStream, stream=None) -> None:
    """Serialise a complete extract result into `out` (sizes are found on the device)."""
    _check(lib().dte_pack_chunks(layout._h, C.byref(delta.struct), out.chunk_entries, out.format,
                                 out.stream.data_ptr(), out.stream_capacity, out.directory.data_ptr(),
                                 out.directory_capacity, out.info.data_ptr(), _stream_ptr(stream)))


def dte_unpack_chunks(layout: Layout, stream_bytes: torch.Tensor, directory: torch.Tensor, n_chunks: int,
                      delta: Delta, stream=None, nbytes: Optional[int] = None) -> None:
    """Verify and decode a chunk stream into `delta` (delta.list_ptr must hold the manifest's list
    boundaries).  `stream_bytes`: uint8 device tensor; `directory`: device tensor holding
    n_chunks + 1 dte_chunk_ref records."""
    assert stream_bytes.dtype == torch.uint8 and stream_bytes.is_contiguous() and stream_bytes.device == layout.device
    assert directory.is_contiguous() and directory.device == layout.device
    assert directory.numel() * directory.element_size() >= 16 * (int(n_chunks) + 1)
    n = stream_bytes.numel() if nbytes is None else int(nbytes)
    _check(lib().dte_unpack_chunks(layout._h, stream_bytes.data_ptr(), n, directory.data_ptr(), int(n_chunks),
                                   C.byref(delta.struct), _stream_ptr(stream)))


def dte_apply_canonical(layout: Layout, canonical: Delta, shard_table, stream=None) -> None:
    """Map canonical entries (one list per SOURCE tensor) into the receiver's shards and store them:
    the destination side of the storage path.  Shards of other receivers may be None in the table."""
    _check(lib().dte_apply_canonical(layout._h, C.byref(canonical.struct), shard_table, _stream_ptr(stream)))


class HostResult:
    def __init__(self, n_lists, capacity, pin=True):
        self.offsets = torch.empty(max(1, capacity), dtype=torch.int32, pin_memory=pin)
        self.values = torch.empty(max(1, capacity), dtype=torch.int16, pin_memory=pin)
        self.list_ptr = torch.zeros(n_lists + 1, dtype=torch.int64, pin_memory=pin)
        self.counters = torch.zeros(4, dtype=torch.int64, pin_memory=pin)

    def arrays(self):
        lp = self.list_ptr.numpy().astype(np.uint64)
        n = int(lp[-1])
        return lp, self.offsets[:n].numpy().view(np.uint32), self.values[:n].numpy().view(np.uint16)


def dte_extract_delta_host(layout: Layout, theta_h, m_h, v_h, step, lr, beta1, beta2, eps, wd,
                           workspace: torch.Tensor, delta: Delta, result: HostResult,
                           stream=None) -> None:
    """Host-resident theta / m / v in, device delta + host copy of the lists out (synchronous)."""
    th = _ptr_table(theta_h, torch.float32)
    mm = _ptr_table(m_h, torch.float32)
    vv = _ptr_table(v_h, torch.float32)
    assert workspace.device == layout.device and workspace.is_contiguous()
    _check(lib().dte_extract_delta_host(
        layout._h, th, mm, vv, int(step), float(lr), float(beta1), float(beta2), float(eps), float(wd),
        workspace.data_ptr(), workspace.numel() * workspace.element_size(), C.byref(delta.struct),
        result.offsets.data_ptr(), result.values.data_ptr(), result.list_ptr.data_ptr(),
        result.counters.data_ptr(), _stream_ptr(stream)))
