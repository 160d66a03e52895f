"""B200 delta-transfer hot path: fused AdamW-inversion / BF16-compare / compaction /
remap extract kernel, sparse apply kernel and the storage path's chunk codec behind a C ABI
(include/dte.h)."""
from .binding import (CHUNK_REF_DTYPE, DTE_CHUNK_BYTE_PLANES, DTE_CHUNK_DELTA_PLANES, DTE_CHUNK_PLAIN, DTE_DEV_BOUNDS,
                      DTE_DEV_CORRUPT, DTE_DEV_OVERFLOW, DTE_DEV_TIMEOUT, SYMBOLS, ChunkStream, Delta,
                      DteError, HostResult, Layout, PushTarget, dte_extract_delta_push, dte_push_wait, dte_apply, dte_apply_canonical, dte_derive_constants, dte_extract_delta,
                      dte_extract_delta_groups, dte_extract_delta_host, dte_extract_delta_static,
                      dte_op_counts, dte_pack_chunks, dte_unpack_chunks, lib,
                      library_path)

__all__ = ["CHUNK_REF_DTYPE", "DTE_CHUNK_BYTE_PLANES", "DTE_CHUNK_DELTA_PLANES", "DTE_CHUNK_PLAIN", "DTE_DEV_BOUNDS",
           "DTE_DEV_CORRUPT", "DTE_DEV_OVERFLOW", "DTE_DEV_TIMEOUT", "SYMBOLS", "ChunkStream", "Delta",
           "DteError", "HostResult", "Layout", "PushTarget", "dte_extract_delta_push", "dte_push_wait", "dte_apply", "dte_apply_canonical", "dte_derive_constants", "dte_extract_delta",
           "dte_extract_delta_groups", "dte_extract_delta_host", "dte_extract_delta_static",
           "dte_op_counts", "dte_pack_chunks", "dte_unpack_chunks", "lib",
           "library_path"]
