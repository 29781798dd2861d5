"""Shared plumbing of the GPU parity tests: device tables, calls through the
C-ABI binding, the oracle's view of the same tables, and the comparison rule."""
from __future__ import annotations

import numpy as np
import torch

import oracle as orc
from paper_2508_05700_b200 import inputs as gi

ATOL, RTOL = 1e-6, 1e-5  # pooled fp32 output: |gpu - ref| <= ATOL + RTOL*|ref|


def mfet():
    from paper_2508_05700_b200 import mfet as m
    return m


def assert_close(gpu: np.ndarray, ref: np.ndarray, what=""):
    gpu = np.asarray(gpu, np.float64)
    ref = np.asarray(ref, np.float64)
    assert gpu.shape == ref.shape, (gpu.shape, ref.shape)
    assert np.isfinite(gpu).all(), what + ": non-finite output"
    err = np.abs(gpu - ref)
    bad = err > ATOL + RTOL * np.abs(ref)
    assert not bad.any(), "%s: %d mismatches, max abs err %.3e at %s" % (
        what, int(bad.sum()), float(err.max()), np.unravel_index(err.argmax(), err.shape))


class DeviceTables:
    """Tables of a workload in HBM (or pinned host memory), filled by the library's
    own generator, plus the oracle's procedural view of the same contents."""

    def __init__(self, specs, value_mode=0, device=0, host_pinned=True):
        m = mfet()
        self.m = m
        self.specs = specs
        self.mem = []
        descs = []
        self.oracle_tables = []
        for s in specs:
            rb = m.row_bytes(s.dim, s.dtype)
            if s.location == gi.LOC_DEVICE:
                buf = torch.empty(s.rows * rb, dtype=torch.uint8, device="cuda:%d" % device)
                m.mfet_table_fill(buf, 0, s.rows, s.dim, s.dtype, 0, s.value_key, value_mode,
                                  torch.cuda.current_stream().cuda_stream)
                descs.append(m.TableDesc(buf.data_ptr(), s.rows, s.dim, s.dtype, m.LOC_DEVICE, 0, s.hash_seed, 0))
            else:
                buf = torch.empty(s.rows * rb, dtype=torch.uint8, pin_memory=host_pinned)
                descs.append(m.TableDesc(None, s.rows, s.dim, s.dtype, m.LOC_HOST, 0, s.hash_seed, 0))
            self.mem.append(buf)
            self.oracle_tables.append(orc.Table(rows=s.rows, dim=s.dim, dtype=s.dtype, hash_seed=s.hash_seed,
                                                value_key=s.value_key, value_mode=value_mode))
        self.h = m.mfet_tables_create(descs, device)
        self.value_mode = value_mode
        self.ws = None
        self.cache = {}
        for i, s in enumerate(specs):
            if s.location == gi.LOC_HOST:
                buf = self.mem[i]
                m.mfet_host_tables_register(self.h, i, buf.data_ptr(), buf.numel(), 1 if host_pinned else 0)
                # fill the pinned rows from the GPU through the unified address space
                m.mfet_table_fill(buf.data_ptr(), 0, s.rows, s.dim, s.dtype, 0, s.value_key, value_mode,
                                  torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()

    def set_workspace(self, max_ids):
        m = self.m
        nbytes = m.mfet_workspace_bytes(self.h, max_ids)
        self.ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
        m.mfet_set_workspace(self.h, self.ws, self.ws.numel(), max_ids)

    def build_cache(self, table_id, rows_sorted):
        m = self.m
        nbytes = m.mfet_cache_bytes(self.h, table_id, len(rows_sorted))
        mem = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
        m.mfet_cache_build(self.h, table_id, np.asarray(rows_sorted, np.int64), mem, mem.numel(),
                           torch.cuda.current_stream().cuda_stream)
        self.cache[table_id] = mem

    def close(self):
        if self.h is not None:
            torch.cuda.synchronize()
            self.m.mfet_tables_destroy(self.h)
            self.h = None

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()


def forward(dt: DeviceTables, batch, n_features, slot_feature, table_ids, pooling, ids, offsets, weights,
            out_ld=0, ids_are_rows=False, out=None):
    """One call of mfet_embedding_bag_forward on numpy inputs; returns the output as numpy."""
    m = dt.m
    total = sum(dt.specs[int(t)].dim for t in table_ids)
    ld = out_ld or total
    d_ids = torch.from_numpy(np.ascontiguousarray(ids, np.uint64).view(np.int64)).cuda()
    if d_ids.numel() == 0:
        d_ids = torch.zeros(1, dtype=torch.int64, device="cuda")  # the ABI wants a non-NULL pointer
    d_off = torch.from_numpy(np.ascontiguousarray(offsets, np.int64)).cuda()
    d_w = None if weights is None else torch.from_numpy(np.ascontiguousarray(weights, np.float32)).cuda()
    if d_w is not None and d_w.numel() == 0:
        d_w = torch.zeros(1, dtype=torch.float32, device="cuda")
    if out is None:
        out = torch.full((batch, ld), float("nan"), dtype=torch.float32, device="cuda")
    shape, keep = m.make_shape(batch, n_features, slot_feature, out_ld, ids_are_rows)
    m.mfet_embedding_bag_forward(dt.h, shape, d_ids, d_off, d_w, table_ids, pooling, out,
                                 torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert m.mfet_query_status(dt.h) == 0
    return out.cpu().numpy()


def workload_forward(dt: DeviceTables, w: gi.Workload, b: gi.Batch, **kw):
    return forward(dt, w.batch, w.n_features, w.slot_feature, w.table_ids, w.pooling, b.ids, b.offsets,
                   b.weights, **kw)


def workload_oracle(dt: DeviceTables, w: gi.Workload, b: gi.Batch, samples=None):
    return orc.embedding_bag(dt.oracle_tables, w.batch, w.n_features, w.slot_feature, w.table_ids, w.pooling,
                             b.ids, b.offsets, b.weights, samples=samples)
