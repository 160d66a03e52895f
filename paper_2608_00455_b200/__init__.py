"""B200 delta-transfer hot path: fused AdamW-inversion / BF16-compare / compaction /
remap extract kernel and sparse apply kernel behind a C ABI (include/dte.h)."""
from .binding import (Delta, DteError, HostResult, Layout, dte_apply, dte_derive_constants,
                      dte_extract_delta, dte_extract_delta_host, dte_extract_delta_static, dte_extract_delta_groups, dte_op_counts, lib, library_path, SYMBOLS,
                      DTE_DEV_BOUNDS, DTE_DEV_OVERFLOW, DTE_DEV_TIMEOUT)

__all__ = ["Delta", "DteError", "HostResult", "Layout", "dte_apply", "dte_derive_constants",
           "dte_extract_delta", "dte_extract_delta_host", "dte_extract_delta_static", "dte_extract_delta_groups", "dte_op_counts", "lib", "library_path", "SYMBOLS",
           "DTE_DEV_BOUNDS", "DTE_DEV_OVERFLOW", "DTE_DEV_TIMEOUT"]
