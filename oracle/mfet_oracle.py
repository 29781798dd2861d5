"""ctypes veneer over oracle.cpp (test infrastructure only; no arithmetic here).

Every function marshals numpy arrays to the C entry points of `liboracle.so`,
which is built from `oracle.cpp` with the host compiler on first use.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")

F32, F16, BF16, INT4 = 0, 1, 2, 3
POOL_SUM, POOL_MEAN, POOL_WSUM = 0, 1, 2
VAL_NORMAL, VAL_GRID = 0, 1


def build(force: bool = False) -> str:
    """Compile oracle.cpp into liboracle.so (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
             "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


class _TableC(C.Structure):
    _fields_ = [("data", C.c_void_p), ("rows", C.c_uint64), ("dim", C.c_uint32),
                ("dtype", C.c_uint32), ("hash_seed", C.c_uint64), ("row_stride", C.c_uint64),
                ("value_key", C.c_uint64), ("value_mode", C.c_uint32), ("reserved", C.c_uint32)]


@dataclass
class Table:
    """One embedding table as the oracle sees it.

    `data` is a C-contiguous numpy array holding the stored rows (any dtype; only
    its bytes are read) or None for a procedural table whose entries are the
    pure function (value_key, value_mode, row, column) defined in oracle.cpp.
    """
    rows: int
    dim: int
    dtype: int
    hash_seed: int = 0
    value_key: int = 0
    value_mode: int = VAL_NORMAL
    data: Optional[np.ndarray] = None
    row_stride: int = 0

    def c(self) -> _TableC:
        ptr = None
        if self.data is not None:
            assert self.data.flags["C_CONTIGUOUS"]
            ptr = self.data.ctypes.data
        return _TableC(ptr, self.rows, self.dim, self.dtype, self.hash_seed & (2**64 - 1),
                       self.row_stride, self.value_key & (2**64 - 1), self.value_mode, 0)


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.orc_splitmix64.restype = C.c_uint64
        L.orc_splitmix64.argtypes = [C.c_uint64]
        L.orc_hash_row.restype = C.c_int64
        L.orc_hash_row.argtypes = [C.c_uint64, C.c_uint64, C.c_uint64]
        L.orc_hash_ids.restype = None
        L.orc_hash_ids.argtypes = [C.c_void_p, C.c_int64, C.c_uint64, C.c_uint64, C.c_void_p]
        for name, res, arg in (("orc_f16_bits_to_f32_bits", C.c_uint32, C.c_uint16),
                               ("orc_bf16_bits_to_f32_bits", C.c_uint32, C.c_uint16),
                               ("orc_f32_bits_to_bf16_bits", C.c_uint16, C.c_uint32),
                               ("orc_f32_bits_to_f16_bits", C.c_uint16, C.c_uint32)):
            getattr(L, name).restype = res
            getattr(L, name).argtypes = [arg]
        L.orc_row_bytes.restype = C.c_uint64
        L.orc_row_bytes.argtypes = [C.c_uint32, C.c_uint32]
        L.orc_table_value_f32.restype = C.c_float
        L.orc_table_value_f32.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint64, C.c_uint32]
        L.orc_table_value_bits.restype = C.c_uint32
        L.orc_table_value_bits.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32,
                                           C.c_uint64, C.c_uint32]
        L.orc_int4_quantize_row.restype = None
        L.orc_int4_quantize_row.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p]
        L.orc_table_fill.restype = None
        L.orc_table_fill.argtypes = [C.POINTER(_TableC), C.c_uint64, C.c_uint64, C.c_void_p]
        L.orc_decode_row_f32.restype = None
        L.orc_decode_row_f32.argtypes = [C.POINTER(_TableC), C.c_uint64, C.c_void_p]
        L.orc_embedding_bag.restype = C.c_int
        L.orc_embedding_bag.argtypes = [C.POINTER(_TableC), C.c_int32, C.c_int32, C.c_int32,
                                        C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64,
                                        C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                        C.c_int32, C.c_void_p]
        L.orc_embedding_bag_backward_slot.restype = C.c_int
        L.orc_embedding_bag_backward_slot.argtypes = [C.POINTER(_TableC), C.c_int32, C.c_void_p,
                                                      C.c_void_p, C.c_void_p, C.c_int32, C.c_int64,
                                                      C.c_int64, C.c_int32, C.c_void_p, C.c_void_p,
                                                      C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_dedup.restype = C.c_int64
        L.orc_dedup.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]
        _lib = L
    return _lib


def _arr(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a), dtype=dtype)


def splitmix64(x: int) -> int:
    return int(lib().orc_splitmix64(x & (2**64 - 1)))


def hash_row(id_: int, seed: int, rows: int) -> int:
    return int(lib().orc_hash_row(id_ & (2**64 - 1), seed & (2**64 - 1), rows))


def hash_ids(ids, seed: int, rows: int) -> np.ndarray:
    ids = _arr(ids, np.uint64)
    out = np.empty(ids.shape, np.int64)
    lib().orc_hash_ids(ids.ctypes.data, ids.size, seed & (2**64 - 1), rows, out.ctypes.data)
    return out


def f16_bits_to_f32_bits(h: int) -> int:
    return int(lib().orc_f16_bits_to_f32_bits(h))


def bf16_bits_to_f32_bits(h: int) -> int:
    return int(lib().orc_bf16_bits_to_f32_bits(h))


def f32_bits_to_f16_bits(f: int) -> int:
    return int(lib().orc_f32_bits_to_f16_bits(f))


def f32_bits_to_bf16_bits(f: int) -> int:
    return int(lib().orc_f32_bits_to_bf16_bits(f))


def row_bytes(dim: int, dtype: int) -> int:
    return int(lib().orc_row_bytes(dim, dtype))


def table_value_f32(key: int, mode: int, dim: int, r: int, d: int) -> float:
    return float(lib().orc_table_value_f32(key & (2**64 - 1), mode, dim, r, d))


def table_value_bits(key: int, mode: int, dim: int, dtype: int, r: int, d: int) -> int:
    return int(lib().orc_table_value_bits(key & (2**64 - 1), mode, dim, dtype, r, d))


def int4_quantize_row(x) -> np.ndarray:
    x = _arr(x, np.float32)
    out = np.zeros(row_bytes(x.size, INT4), np.uint8)
    lib().orc_int4_quantize_row(x.ctypes.data, x.size, out.ctypes.data)
    return out


def table_fill(t: Table, r0: int = 0, r1: Optional[int] = None) -> np.ndarray:
    """Rows [r0, r1) of a procedural table as stored bytes, uint8 [r1-r0, row_bytes]."""
    r1 = t.rows if r1 is None else r1
    out = np.zeros((r1 - r0, row_bytes(t.dim, t.dtype)), np.uint8)
    tc = t.c()
    lib().orc_table_fill(C.byref(tc), r0, r1, out.ctypes.data)
    return out


def decode_row(t: Table, r: int) -> np.ndarray:
    out = np.empty(t.dim, np.float32)
    tc = t.c()
    lib().orc_decode_row_f32(C.byref(tc), r, out.ctypes.data)
    return out


def embedding_bag(tables: Sequence[Table], batch: int, n_features: int, slot_feature, table_ids,
                  pooling, ids, offsets, weights=None, out_ld: int = 0, ids_are_rows: bool = False,
                  samples: Optional[Sequence[int]] = None) -> np.ndarray:
    """Pooled output. All samples -> fp32 [batch, out_ld]; with `samples`, only
    those samples are computed and returned as fp32 [len(samples), out_ld]."""
    slot_feature = _arr(slot_feature, np.int32)
    table_ids = _arr(table_ids, np.int32)
    pooling = _arr(pooling, np.int32)
    ids = _arr(ids, np.uint64)
    offsets = _arr(offsets, np.int64)
    w = None if weights is None else _arr(weights, np.float32)
    n_slots = int(slot_feature.size)
    if out_ld == 0:
        out_ld = int(sum(tables[int(t)].dim for t in table_ids))
    tarr = (_TableC * len(tables))(*[t.c() for t in tables])
    wptr = None if w is None else w.ctypes.data

    def call(b0, b1, out_ptr):
        rc = lib().orc_embedding_bag(tarr, len(tables), batch, n_features, n_slots,
                                     slot_feature.ctypes.data, table_ids.ctypes.data,
                                     pooling.ctypes.data, out_ld, int(ids_are_rows),
                                     ids.ctypes.data, offsets.ctypes.data, wptr, b0, b1, out_ptr)
        if rc != 0:
            raise ValueError("oracle: invalid argument")

    if samples is None:
        out = np.zeros((batch, out_ld), np.float32)
        call(0, batch, out.ctypes.data)
        return out
    out = np.zeros((len(samples), out_ld), np.float32)
    for k, b in enumerate(samples):
        # the C routine writes sample b at out + b*out_ld: shift the base so it lands on row k
        call(int(b), int(b) + 1, out.ctypes.data + (k - int(b)) * out_ld * 4)
    return out


def embedding_bag_backward_slot(tables: Sequence[Table], batch: int, slot_feature, table_ids,
                                pooling, s: int, out_ld: int, col_off: int, ids, offsets, weights,
                                grad_out, ids_are_rows: bool = False) -> np.ndarray:
    """Dense double [rows, dim] gradient of slot `s`'s table."""
    slot_feature = _arr(slot_feature, np.int32)
    table_ids = _arr(table_ids, np.int32)
    pooling = _arr(pooling, np.int32)
    ids = _arr(ids, np.uint64)
    offsets = _arr(offsets, np.int64)
    w = None if weights is None else _arr(weights, np.float32)
    g = _arr(grad_out, np.float32)
    t = tables[int(table_ids[s])]
    out = np.zeros((t.rows, t.dim), np.float64)
    tarr = (_TableC * len(tables))(*[x.c() for x in tables])
    rc = lib().orc_embedding_bag_backward_slot(
        tarr, batch, slot_feature.ctypes.data, table_ids.ctypes.data, pooling.ctypes.data, s, out_ld,
        col_off, int(ids_are_rows), ids.ctypes.data, offsets.ctypes.data,
        None if w is None else w.ctypes.data, g.ctypes.data, out.ctypes.data)
    if rc != 0:
        raise ValueError("oracle: invalid argument")
    return out


def dedup(rows):
    rows = _arr(rows, np.int64)
    uniq = np.empty(rows.size, np.int64)
    inv = np.empty(rows.size, np.int32)
    n = int(lib().orc_dedup(rows.ctypes.data, rows.size, uniq.ctypes.data, inv.ctypes.data))
    return uniq[:n].copy(), inv
