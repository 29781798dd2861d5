"""Thin ctypes binding of libmfet.so: same names as include/mfet.h, argument
marshalling only. Every step of the lookup path runs in the library's CUDA
kernels; if the library is missing this module raises at import instead of
falling back to anything else.

Pointers may be given as torch tensors (their data_ptr is taken), numpy arrays
(host arguments), or plain integers.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# MFET_LIBRARY selects another build of the same library (the bounds-checked one, libmfet_checked.so)
LIB_PATH = os.environ.get("MFET_LIBRARY") or os.path.join(_HERE, "libmfet.so")

F32, F16, BF16, INT4 = 0, 1, 2, 3
POOL_SUM, POOL_MEAN, POOL_WSUM = 0, 1, 2
LOC_DEVICE, LOC_HOST = 0, 1
VAL_NORMAL, VAL_GRID = 0, 1
OPT_GROUP_POLICY = 1
OPT_TILE = 2
OPT_PROFILE = 3
OPT_STAGE_IDS = 4
OPT_OVERLAP_LAUNCHES = 5
OK = 0
ERR_INVALID_ARG, ERR_NOT_REGISTERED, ERR_ALIGNMENT, ERR_UNSUPPORTED_DIM = -1, -2, -3, -4
ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = -5, -6, -7
DEV_ROW_RANGE, DEV_OFFSETS, DEV_CAPACITY, DEV_BOUNDS, DEV_STALLED = 1, 2, 4, 8, 16

EXPORTS = [
    "mfet_row_bytes", "mfet_tables_create", "mfet_tables_destroy", "mfet_host_tables_register",
    "mfet_hash_ids", "mfet_embedding_bag_forward", "mfet_dedup_rows", "mfet_cache_bytes",
    "mfet_cache_build", "mfet_workspace_bytes", "mfet_set_workspace", "mfet_host_io_bytes",
    "mfet_embedding_bag_forward_host", "mfet_table_fill", "mfet_query_status", "mfet_set_option",
    "mfet_launch_count", "mfet_status_string", "mfet_dedup_rows_static", "mfet_profile_read", "mfet_host_path_counts", "mfet_tables_set_version", "mfet_tables_version",
    "mfet_host_prefetch", "mfet_embedding_bag_backward", "mfet_embedding_bag_forward_host_async",
    "mfet_host_path_result", "mfet_host_fetch_rows",
]
BATCH_IDS_ARE_ROWS, BATCH_PREFETCHED = 1, 2
STATIC_DEDUP_MAX_IDS = 262144


class TableDesc(C.Structure):
    _fields_ = [("data", C.c_void_p), ("rows", C.c_uint64), ("dim", C.c_uint32), ("dtype", C.c_uint32),
                ("location", C.c_uint32), ("flags", C.c_uint32), ("hash_seed", C.c_uint64),
                ("row_stride_bytes", C.c_uint64)]


class BatchShape(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_features", C.c_int32), ("n_slots", C.c_int32),
                ("flags", C.c_int32), ("slot_feature", C.POINTER(C.c_int32)), ("out_ld", C.c_int64)]


if not os.path.exists(LIB_PATH):
    raise ImportError("libmfet.so is missing: build it with `python -m paper_2508_05700_b200.build` "
                      "(there is no fallback path)")
_lib = C.CDLL(LIB_PATH)

_P = C.c_void_p
_lib.mfet_row_bytes.restype = C.c_uint64
_lib.mfet_row_bytes.argtypes = [C.c_uint32, C.c_uint32]
_lib.mfet_status_string.restype = C.c_char_p
_lib.mfet_status_string.argtypes = [C.c_int]
_lib.mfet_tables_create.argtypes = [C.POINTER(TableDesc), C.c_int32, C.c_int32, C.POINTER(_P)]
_lib.mfet_tables_destroy.argtypes = [_P]
_lib.mfet_host_tables_register.argtypes = [_P, C.c_int32, _P, C.c_uint64, C.c_uint32]
_lib.mfet_hash_ids.argtypes = [_P, C.c_int32, _P, C.c_int64, _P, _P]
_lib.mfet_embedding_bag_forward.argtypes = [_P, C.POINTER(BatchShape), _P, _P, _P, _P, _P, _P, _P]
_lib.mfet_dedup_rows.argtypes = [_P, _P, C.c_int64, _P, _P, _P, C.c_int64, _P]
_lib.mfet_dedup_rows_static.argtypes = [C.c_int32, _P, C.c_int64, _P, _P, _P, C.c_int64, _P]
_lib.mfet_cache_bytes.argtypes = [_P, C.c_int32, C.c_int64, C.POINTER(C.c_uint64)]
_lib.mfet_cache_build.argtypes = [_P, C.c_int32, _P, C.c_int64, _P, C.c_uint64, _P]
_lib.mfet_workspace_bytes.argtypes = [_P, C.c_int64, C.POINTER(C.c_uint64)]
_lib.mfet_set_workspace.argtypes = [_P, _P, C.c_uint64, C.c_int64]
_lib.mfet_host_io_bytes.argtypes = [_P, C.POINTER(BatchShape), _P, C.c_int64, C.POINTER(C.c_uint64)]
_lib.mfet_embedding_bag_forward_host.argtypes = [_P, C.POINTER(BatchShape), _P, _P, _P, C.c_int64, _P, _P, _P,
                                                 _P, C.c_uint64, _P]
_lib.mfet_embedding_bag_forward_host_async.argtypes = _lib.mfet_embedding_bag_forward_host.argtypes
_lib.mfet_table_fill.argtypes = [_P, C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint64, C.c_uint64,
                                 C.c_uint32, _P]
_lib.mfet_query_status.argtypes = [_P, C.POINTER(C.c_uint32), C.c_int32]
_lib.mfet_set_option.argtypes = [_P, C.c_int32, C.c_int64]
_lib.mfet_profile_read.argtypes = [_P, C.POINTER(C.c_float)]
_lib.mfet_host_path_counts.argtypes = [_P, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
_lib.mfet_host_path_result.argtypes = [_P, _P, _P, _P, C.c_int64]
_lib.mfet_host_fetch_rows.argtypes = [_P, C.c_int32, _P, C.c_int64, _P, _P]
_lib.mfet_tables_set_version.argtypes = [_P, C.c_uint64]
_lib.mfet_tables_version.argtypes = [_P, C.POINTER(C.c_uint64)]
_lib.mfet_host_prefetch.argtypes = [_P, C.POINTER(BatchShape), _P, _P, _P, _P]
_lib.mfet_embedding_bag_backward.argtypes = [_P, C.POINTER(BatchShape), _P, _P, _P, _P, _P, _P, C.c_int32, _P, _P, _P, _P]
_lib.mfet_launch_count.argtypes = [_P, C.POINTER(C.c_uint64)]
for _n in EXPORTS:
    if _n not in ("mfet_row_bytes", "mfet_status_string"):
        getattr(_lib, _n).restype = C.c_int


class MfetError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (%d)" % (where, status_string(status), status))


def _ptr(x) -> Optional[int]:
    """Address of a torch tensor, numpy array, ctypes pointer or int; None stays NULL."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return int(x.data_ptr())
    if isinstance(x, np.ndarray):
        return int(x.ctypes.data)
    return C.cast(x, C.c_void_p).value


def _check(status: int, where: str) -> None:
    if status != OK:
        raise MfetError(status, where)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a), dtype=np.int32)


def status_string(status: int) -> str:
    return _lib.mfet_status_string(status).decode()


def row_bytes(dim: int, dtype: int) -> int:
    return int(_lib.mfet_row_bytes(dim, dtype))


def make_shape(batch: int, n_features: int, slot_feature, out_ld: int = 0, ids_are_rows: bool = False):
    """(BatchShape, keep-alive) for the forward calls."""
    sf = _i32(slot_feature)
    sh = BatchShape(batch, n_features, int(sf.size), 1 if ids_are_rows else 0,
                    sf.ctypes.data_as(C.POINTER(C.c_int32)), out_ld)
    return sh, sf


def mfet_tables_create(descs: Sequence[TableDesc], device: int = 0) -> int:
    arr = (TableDesc * len(descs))(*descs)
    h = _P()
    _check(_lib.mfet_tables_create(arr, len(descs), device, C.byref(h)), "mfet_tables_create")
    return h.value


def mfet_tables_destroy(h) -> None:
    _check(_lib.mfet_tables_destroy(h), "mfet_tables_destroy")


def mfet_host_tables_register(h, table_id: int, host_ptr, nbytes: int, flags: int = 0) -> None:
    _check(_lib.mfet_host_tables_register(h, table_id, _ptr(host_ptr), nbytes, flags), "mfet_host_tables_register")


def mfet_hash_ids(h, table_id: int, ids, n: int, rows_out, stream=None) -> None:
    _check(_lib.mfet_hash_ids(h, table_id, _ptr(ids), n, _ptr(rows_out), _ptr(stream)), "mfet_hash_ids")


def mfet_embedding_bag_forward(h, shape: BatchShape, ids, offsets, weights, table_ids, pooling, out,
                               stream=None) -> None:
    ti, po = _i32(table_ids), _i32(pooling)
    _check(_lib.mfet_embedding_bag_forward(h, C.byref(shape), _ptr(ids), _ptr(offsets), _ptr(weights),
                                           ti.ctypes.data, po.ctypes.data, _ptr(out), _ptr(stream)),
           "mfet_embedding_bag_forward")


def mfet_dedup_rows(h, rows, n: int, uniq, inverse, n_unique, max_row: int = 0, stream=None) -> None:
    _check(_lib.mfet_dedup_rows(h, _ptr(rows), n, _ptr(uniq), _ptr(inverse), _ptr(n_unique), max_row,
                                _ptr(stream)), "mfet_dedup_rows")


def mfet_dedup_rows_static(device: int, rows, n: int, uniq, inverse, n_unique, max_row: int = 0, stream=None) -> None:
    """Dedup on the library's built-in scratch array: no workspace, no allocation anywhere
    (n <= STATIC_DEDUP_MAX_IDS). Calls on one GPU share that array and must not overlap."""
    _check(_lib.mfet_dedup_rows_static(device, _ptr(rows), n, _ptr(uniq), _ptr(inverse), _ptr(n_unique), max_row,
                                       _ptr(stream)), "mfet_dedup_rows_static")


def mfet_cache_bytes(h, table_id: int, n: int) -> int:
    b = C.c_uint64()
    _check(_lib.mfet_cache_bytes(h, table_id, n, C.byref(b)), "mfet_cache_bytes")
    return int(b.value)


def mfet_cache_build(h, table_id: int, rows_sorted: np.ndarray, cache_mem, cache_bytes: int, stream=None) -> None:
    rs = np.ascontiguousarray(rows_sorted, dtype=np.int64)
    _check(_lib.mfet_cache_build(h, table_id, rs.ctypes.data, rs.size, _ptr(cache_mem), cache_bytes, _ptr(stream)),
           "mfet_cache_build")


def mfet_workspace_bytes(h, max_ids: int) -> int:
    b = C.c_uint64()
    _check(_lib.mfet_workspace_bytes(h, max_ids, C.byref(b)), "mfet_workspace_bytes")
    return int(b.value)


def mfet_set_workspace(h, dev_ptr, nbytes: int, max_ids: int) -> None:
    _check(_lib.mfet_set_workspace(h, _ptr(dev_ptr), nbytes, max_ids), "mfet_set_workspace")


def mfet_host_io_bytes(h, shape: BatchShape, table_ids, nnz: int) -> int:
    ti = _i32(table_ids)
    b = C.c_uint64()
    _check(_lib.mfet_host_io_bytes(h, C.byref(shape), ti.ctypes.data, nnz, C.byref(b)), "mfet_host_io_bytes")
    return int(b.value)


def mfet_embedding_bag_forward_host(h, shape: BatchShape, ids_host, offsets_host, weights_host, nnz: int,
                                    table_ids, pooling, out_host, dev_io, dev_io_bytes: int, stream=None) -> None:
    ti, po = _i32(table_ids), _i32(pooling)
    _check(_lib.mfet_embedding_bag_forward_host(h, C.byref(shape), _ptr(ids_host), _ptr(offsets_host),
                                                _ptr(weights_host), nnz, ti.ctypes.data, po.ctypes.data,
                                                _ptr(out_host), _ptr(dev_io), dev_io_bytes, _ptr(stream)),
           "mfet_embedding_bag_forward_host")


def mfet_embedding_bag_forward_host_async(h, shape: BatchShape, ids_host, offsets_host, weights_host, nnz: int,
                                          table_ids, pooling, out_host, dev_io, dev_io_bytes: int, stream=None) -> None:
    ti, po = _i32(table_ids), _i32(pooling)
    _check(_lib.mfet_embedding_bag_forward_host_async(h, C.byref(shape), _ptr(ids_host), _ptr(offsets_host),
                                                      _ptr(weights_host), nnz, ti.ctypes.data, po.ctypes.data,
                                                      _ptr(out_host), _ptr(dev_io), dev_io_bytes, _ptr(stream)),
           "mfet_embedding_bag_forward_host_async")


def mfet_table_fill(data, row0: int, n_rows: int, dim: int, dtype: int, row_stride_bytes: int, value_key: int,
                    value_mode: int = VAL_NORMAL, stream=None) -> None:
    _check(_lib.mfet_table_fill(_ptr(data), row0, n_rows, dim, dtype, row_stride_bytes,
                                value_key & (2**64 - 1), value_mode, _ptr(stream)), "mfet_table_fill")


def mfet_query_status(h, clear: bool = False) -> int:
    bits = C.c_uint32()
    _check(_lib.mfet_query_status(h, C.byref(bits), 1 if clear else 0), "mfet_query_status")
    return int(bits.value)


def mfet_set_option(h, option: int, value: int) -> None:
    _check(_lib.mfet_set_option(h, option, value), "mfet_set_option")


def mfet_profile_read(h):
    """(dedup_ms, fetch_ms, pool_ms) of the last forward call's host-table path."""
    ms = (C.c_float * 3)()
    _check(_lib.mfet_profile_read(h, ms), "mfet_profile_read")
    return tuple(float(x) for x in ms)


def mfet_host_path_counts(h):
    """(distinct rows, distinct rows missing from the cache) of the last host-table slot."""
    a, b = C.c_int64(), C.c_int64()
    _check(_lib.mfet_host_path_counts(h, C.byref(a), C.byref(b)), "mfet_host_path_counts")
    return int(a.value), int(b.value)


def mfet_host_path_result(h, uniq, src, miss_rows, capacity: int) -> None:
    _check(_lib.mfet_host_path_result(h, _ptr(uniq), _ptr(src), _ptr(miss_rows), capacity), "mfet_host_path_result")


def mfet_host_fetch_rows(h, table_id: int, rows, n: int, dst, stream=None) -> None:
    _check(_lib.mfet_host_fetch_rows(h, table_id, _ptr(rows), n, _ptr(dst), _ptr(stream)), "mfet_host_fetch_rows")


def mfet_tables_set_version(h, version: int) -> None:
    _check(_lib.mfet_tables_set_version(h, version & (2**64 - 1)), "mfet_tables_set_version")


def mfet_tables_version(h) -> int:
    v = C.c_uint64()
    _check(_lib.mfet_tables_version(h, C.byref(v)), "mfet_tables_version")
    return int(v.value)


def mfet_host_prefetch(h, shape: BatchShape, ids, offsets, table_ids, stream=None) -> None:
    ti = _i32(table_ids)
    _check(_lib.mfet_host_prefetch(h, C.byref(shape), _ptr(ids), _ptr(offsets), ti.ctypes.data, _ptr(stream)),
           "mfet_host_prefetch")


def mfet_embedding_bag_backward(h, shape: BatchShape, ids, offsets, weights, table_ids, pooling, grad_out, slot: int,
                                grad_rows, grad_vals, n_rows, stream=None) -> None:
    ti, po = _i32(table_ids), _i32(pooling)
    _check(_lib.mfet_embedding_bag_backward(h, C.byref(shape), _ptr(ids), _ptr(offsets), _ptr(weights), ti.ctypes.data,
                                            po.ctypes.data, _ptr(grad_out), slot, _ptr(grad_rows), _ptr(grad_vals),
                                            _ptr(n_rows), _ptr(stream)), "mfet_embedding_bag_backward")


def mfet_launch_count(h) -> int:
    n = C.c_uint64()
    _check(_lib.mfet_launch_count(h, C.byref(n)), "mfet_launch_count")
    return int(n.value)
