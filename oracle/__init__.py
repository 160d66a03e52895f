"""ctypes front end of the CPU oracle (test infrastructure, not product code).

Only tests, the smoke check and the benchmark's CPU-baseline leg import this
package.  It compiles ``dte_oracle.cpp`` and ``chunk_oracle.cpp`` with g++ on first use and exposes the
oracle's functions on numpy arrays.  Nothing here touches the CUDA library.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRCS = [os.path.join(_HERE, "dte_oracle.cpp"), os.path.join(_HERE, "chunk_oracle.cpp")]
_LIB = os.path.join(_HERE, "libdte_oracle.so")
_CXXFLAGS = ["-O2", "-std=c++17", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC"]
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle into ``libdte_oracle.so`` next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < max(map(os.path.getmtime, _SRCS)):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(["g++", *_CXXFLAGS, "-o", tmp, *_SRCS], check=True)
        os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    with _lock:
        if _lib is None:
            L = ctypes.CDLL(build())
            c = ctypes
            L.oracle_derive_constants.argtypes = [c.c_int64, c.c_double, c.c_double, c.c_double,
                                                  c.c_double, c.c_double, c.c_void_p]
            L.oracle_derive_constants.restype = None
            L.oracle_invert.argtypes = [c.c_void_p] * 3 + [c.c_uint64, c.c_void_p, c.c_void_p]
            L.oracle_invert.restype = None
            L.oracle_bf16_rne.argtypes = [c.c_void_p, c.c_uint64, c.c_void_p]
            L.oracle_bf16_rne.restype = None
            L.oracle_changed_mask.argtypes = [c.c_void_p] * 3 + [c.c_uint64] + [c.c_void_p] * 3
            L.oracle_changed_mask.restype = c.c_uint64
            L.oracle_extract.argtypes = [c.c_uint64, c.c_void_p, c.c_uint64, c.c_void_p, c.c_uint64,
                                         c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p]
            L.oracle_extract.restype = c.c_void_p
            L.oracle_result_error.argtypes = [c.c_void_p]
            L.oracle_result_error.restype = c.c_char_p
            L.oracle_result_total.argtypes = [c.c_void_p]
            L.oracle_result_total.restype = c.c_uint64
            L.oracle_result_copy.argtypes = [c.c_void_p] * 4
            L.oracle_result_copy.restype = None
            L.oracle_result_op_counts.argtypes = [c.c_void_p, c.c_void_p]
            L.oracle_result_op_counts.restype = None
            L.oracle_result_nonfinite.argtypes = [c.c_void_p]
            L.oracle_result_nonfinite.restype = c.c_uint64
            L.oracle_result_free.argtypes = [c.c_void_p]
            L.oracle_result_free.restype = None
            L.oracle_apply.argtypes = [c.c_uint64, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p,
                                       c.c_void_p]
            L.oracle_apply.restype = c.c_int
            L.oracle_apply_canonical.argtypes = [c.c_uint64, c.c_void_p, c.c_uint64, c.c_void_p, c.c_uint64,
                                                 c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p]
            L.oracle_apply_canonical.restype = c.c_int
            L.oracle_adler32.argtypes = [c.c_void_p, c.c_uint64]
            L.oracle_adler32.restype = c.c_uint32
            L.oracle_pack_chunks.argtypes = [c.c_uint64, c.c_void_p, c.c_void_p, c.c_void_p, c.c_uint32,
                                             c.c_uint32, c.c_void_p, c.c_void_p, c.c_void_p]
            L.oracle_pack_chunks.restype = c.c_uint64
            L.oracle_unpack_chunks.argtypes = [c.c_void_p, c.c_uint64, c.c_void_p, c.c_uint64, c.c_uint64,
                                               c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p]
            L.oracle_unpack_chunks.restype = c.c_uint64
            _lib = L
    return _lib


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32).reshape(-1)


def derive_constants(step, lr, beta1, beta2, eps, wd) -> np.ndarray:
    """{bc1, bc2, decay, lr, eps} as fp32 (Eq. 2's call-uniform scalars)."""
    out = np.zeros(5, np.float32)
    lib().oracle_derive_constants(int(step), float(lr), float(beta1), float(beta2), float(eps),
                                  float(wd), out.ctypes.data)
    return out


def invert(theta, m, v, consts) -> np.ndarray:
    """Reconstructed theta_{t-1} (Eq. 2), element-wise fp32."""
    theta, m, v = _f32(theta), _f32(m), _f32(v)
    c = _f32(consts)
    prev = np.empty_like(theta)
    lib().oracle_invert(theta.ctypes.data, m.ctypes.data, v.ctypes.data, theta.size,
                        c.ctypes.data, prev.ctypes.data)
    return prev


def bf16_rne(x) -> np.ndarray:
    """BF16 bit patterns (uint16) of fp32 inputs, round-to-nearest-even."""
    x = _f32(x)
    out = np.empty(x.size, np.uint16)
    lib().oracle_bf16_rne(x.ctypes.data, x.size, out.ctypes.data)
    return out


def changed_mask(theta, m, v, consts):
    """Eq. 4 on one tensor: (mask uint8[n], BF16(theta_t) uint16[n])."""
    theta, m, v = _f32(theta), _f32(m), _f32(v)
    c = _f32(consts)
    mask = np.empty(theta.size, np.uint8)
    val = np.empty(theta.size, np.uint16)
    lib().oracle_changed_mask(theta.ctypes.data, m.ctypes.data, v.ctypes.data, theta.size,
                              c.ctypes.data, mask.ctypes.data, val.ctypes.data)
    return mask, val


def _ptr_array(arrs):
    return (ctypes.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])


def extract(tensor_shapes, shard_numels, ops, theta, m, v, consts, with_op_counts=False, with_nonfinite=False):
    """Full extract (Eq. 2, 4, 5, 6) over a transfer plan.

    tensor_shapes: [(n0, n1)] per source tensor; shard_numels: [numel] per
    receiver-local tensor; ops: rows of 10 integers {src_tensor, dst_shard,
    a_s0, a_s1, e0, e1, dst_base, dst_ld, a_r0, a_r1}; theta/m/v: lists of
    fp32 arrays; consts: the 5 scalars of derive_constants, or one row of 5
    per source tensor (per-group learning rate / weight decay).  Returns (list_ptr uint64[n_shards+1], offsets uint32[M],
    values uint16[M]).
    """
    L = lib()
    shp = np.ascontiguousarray(tensor_shapes, dtype=np.int64).reshape(-1, 2)
    num = np.ascontiguousarray(shard_numels, dtype=np.int64).reshape(-1)
    op = np.ascontiguousarray(ops, dtype=np.int64).reshape(-1, 10)
    th = [_f32(a) for a in theta]
    mm = [_f32(a) for a in m]
    vv = [_f32(a) for a in v]
    for p in range(shp.shape[0]):
        n = int(shp[p, 0] * shp[p, 1])
        assert th[p].size == n and mm[p].size == n and vv[p].size == n, "tensor size mismatch"
    c = np.ascontiguousarray(consts, dtype=np.float32)
    if c.ndim == 1:                       # one parameter group: the same scalars for every tensor
        c = np.tile(c.reshape(1, 5), (shp.shape[0], 1))
    assert c.shape == (shp.shape[0], 5), "consts: 5 scalars, or 5 per source tensor"
    c = np.ascontiguousarray(c)
    h = L.oracle_extract(shp.shape[0], shp.ctypes.data, num.size, num.ctypes.data, op.shape[0],
                         op.ctypes.data, _ptr_array(th), _ptr_array(mm), _ptr_array(vv),
                         c.ctypes.data)
    try:
        err = L.oracle_result_error(h)
        if err:
            raise ValueError(err.decode())
        total = L.oracle_result_total(h)
        list_ptr = np.zeros(num.size + 1, np.uint64)
        offsets = np.zeros(total, np.uint32)
        values = np.zeros(total, np.uint16)
        L.oracle_result_copy(h, list_ptr.ctypes.data, offsets.ctypes.data, values.ctypes.data)
        op_counts = np.zeros(op.shape[0], np.uint64)
        L.oracle_result_op_counts(h, op_counts.ctypes.data)
        nonfinite = int(L.oracle_result_nonfinite(h))
    finally:
        L.oracle_result_free(h)
    out = (list_ptr, offsets, values)
    if with_op_counts:          # c_o per operation, plan order, zeros included (Section 4.3)
        out += (op_counts,)
    if with_nonfinite:          # receiver slots whose reconstruction is NaN, or Inf from a finite theta_t
        out += (nonfinite,)
    return out


def apply(shard_numels, list_ptr, offsets, values, shards) -> None:
    """Eq. 7 in place on ``shards`` (list of contiguous uint16 arrays)."""
    num = np.ascontiguousarray(shard_numels, dtype=np.int64).reshape(-1)
    lp = np.ascontiguousarray(list_ptr, dtype=np.uint64)
    off = np.ascontiguousarray(offsets, dtype=np.uint32)
    val = np.ascontiguousarray(values, dtype=np.uint16)
    for k, s in enumerate(shards):
        assert s.dtype == np.uint16 and s.flags.c_contiguous and s.size == num[k]
    rc = lib().oracle_apply(num.size, num.ctypes.data, lp.ctypes.data, off.ctypes.data,
                            val.ctypes.data, _ptr_array(shards))
    if rc != 0:
        raise ValueError("receiver index outside its shard")


def apply_canonical(tensor_shapes, shard_numels, ops, list_ptr, indices, values, shards) -> None:
    """Eq. 5-7 on canonical entries (destination-side mapping of the storage path), in place on
    ``shards``: a list of contiguous uint16 arrays, or None for shards other receivers hold."""
    shp = np.ascontiguousarray(tensor_shapes, dtype=np.int64).reshape(-1, 2)
    num = np.ascontiguousarray(shard_numels, dtype=np.int64).reshape(-1)
    op = np.ascontiguousarray(ops, dtype=np.int64).reshape(-1, 10)
    lp = np.ascontiguousarray(list_ptr, dtype=np.uint64)
    idx = np.ascontiguousarray(indices, dtype=np.uint32)
    val = np.ascontiguousarray(values, dtype=np.uint16)
    assert lp.size == shp.shape[0] + 1 and len(shards) == num.size
    ptrs = (ctypes.c_void_p * max(1, num.size))()
    for k, s in enumerate(shards):
        if s is not None:
            assert s.dtype == np.uint16 and s.flags.c_contiguous and s.size == num[k]
            ptrs[k] = s.ctypes.data
    rc = lib().oracle_apply_canonical(shp.shape[0], shp.ctypes.data, num.size, num.ctypes.data, op.shape[0],
                                      op.ctypes.data, lp.ctypes.data, idx.ctypes.data, val.ctypes.data, ptrs)
    if rc == 1:
        raise ValueError("receiver index outside its shard")
    if rc == 2:
        raise ValueError("canonical index outside its tensor")


def adler32(data) -> int:
    """Adler-32 (RFC 1950) of a byte string / uint8 array, by its definition."""
    b = np.ascontiguousarray(np.frombuffer(bytes(data), dtype=np.uint8))
    return int(lib().oracle_adler32(b.ctypes.data if b.size else None, b.size))


def pack_chunks(list_ptr, offsets, values, chunk_entries, fmt=0):
    """Serialise lists into the chunk stream of the storage path (Section 4.4).

    Returns (stream uint8[bytes], directory uint64[n_chunks + 1, 3] = {byte offset, list,
    first_entry}; the last row holds the total size)."""
    lp = np.ascontiguousarray(list_ptr, dtype=np.uint64)
    off = np.ascontiguousarray(offsets, dtype=np.uint32)
    val = np.ascontiguousarray(values, dtype=np.uint16)
    n_lists = lp.size - 1
    n_chunks = np.zeros(1, np.uint64)
    args = (n_lists, lp.ctypes.data, off.ctypes.data, val.ctypes.data, int(chunk_entries), int(fmt))
    size = lib().oracle_pack_chunks(*args, None, None, n_chunks.ctypes.data)
    if size == 2 ** 64 - 1:
        raise ValueError("chunk_entries must be a positive multiple of 8 and fmt 0, 1 or 2")
    stream = np.zeros(int(size), np.uint8)
    directory = np.zeros((int(n_chunks[0]) + 1, 3), np.uint64)
    lib().oracle_pack_chunks(*args, stream.ctypes.data, directory.ctypes.data, n_chunks.ctypes.data)
    return stream, directory


def unpack_chunks(stream, directory, list_ptr):
    """Inverse of pack_chunks: (offsets uint32[M], values uint16[M], rejected chunks, entries
    written); entries of rejected chunks stay zero."""
    st = np.ascontiguousarray(stream, dtype=np.uint8)
    d = np.ascontiguousarray(directory, dtype=np.uint64).reshape(-1, 3)
    lp = np.ascontiguousarray(list_ptr, dtype=np.uint64)
    total = int(lp[-1])
    off = np.zeros(total, np.uint32)
    val = np.zeros(total, np.uint16)
    written = np.zeros(1, np.uint64)
    rejected = lib().oracle_unpack_chunks(st.ctypes.data, st.size, d.ctypes.data, d.shape[0] - 1, lp.size - 1,
                                          lp.ctypes.data, off.ctypes.data, val.ctypes.data,
                                          written.ctypes.data)
    return off, val, int(rejected), int(written[0])
