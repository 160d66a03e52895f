"""ctypes binding of libdte_probes.so: measurement probes for the benchmark, not product code.

The probes time what the memory system does for an access pattern (a read-only stream; isolated
small stores and sector loads at ascending offsets) so that the path's kernels can be put next to
it.  Nothing in the delta-transfer path calls them.
"""
from __future__ import annotations

import ctypes as C

import torch

from . import build as _build

_lib = None

SPARSE_MODES = {0: "2-byte stores", 1: "4-byte stores", 2: "32-byte sector stores (no read)",
                3: "sector load + sector store", 4: "sector loads"}


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build_probes())
        vp, u64 = C.c_void_p, C.c_uint64
        L.dte_probe_read_bandwidth.argtypes = [vp, u64, vp, C.c_int, vp]
        L.dte_probe_read_bandwidth.restype = C.c_int
        L.dte_probe_make_offsets.argtypes = [vp, u64, C.c_uint32, C.c_uint32, vp]
        L.dte_probe_make_offsets.restype = C.c_int
        L.dte_probe_sparse_access.argtypes = [C.c_int, vp, u64, vp, vp, C.c_int, C.c_int, vp]
        L.dte_probe_sparse_access.restype = C.c_int
        _lib = L
    return _lib


def _check(err: int, what: str) -> None:
    if err != 0:
        raise RuntimeError(f"{what}: CUDA error {err}")


def _stream():
    return torch.cuda.current_stream().cuda_stream


def read_bandwidth(tensor: torch.Tensor, xor_out: torch.Tensor) -> None:
    """Enqueue one read-only pass over `tensor` on the current stream."""
    assert tensor.is_cuda and tensor.is_contiguous() and xor_out.is_cuda and xor_out.dtype == torch.int64
    _check(lib().dte_probe_read_bandwidth(tensor.data_ptr(), tensor.numel() * tensor.element_size(),
                                          xor_out.data_ptr(), tensor.device.index or 0, _stream()),
           "dte_probe_read_bandwidth")


def make_offsets(n: int, stride: int, jitter: int, device) -> torch.Tensor:
    """n ascending uint32 offsets (as int32 bits), one per `stride` elements."""
    off = torch.empty(n, dtype=torch.int32, device=device)
    _check(lib().dte_probe_make_offsets(off.data_ptr(), n, stride, jitter, _stream()), "dte_probe_make_offsets")
    return off


def sparse_access(mode: int, offsets: torch.Tensor, dst: torch.Tensor, sink: torch.Tensor,
                  ctas_per_sm: int = 6) -> None:
    """Enqueue one access per offset into `dst` (int16 elements); see SPARSE_MODES."""
    assert offsets.is_cuda and offsets.dtype == torch.int32 and dst.dtype == torch.int16 and sink.dtype == torch.int32
    _check(lib().dte_probe_sparse_access(mode, offsets.data_ptr(), offsets.numel(), dst.data_ptr(), sink.data_ptr(),
                                         ctas_per_sm, dst.device.index or 0, _stream()), "dte_probe_sparse_access")
