"""LookupEngine: owns the memory around one mfet table set (PyTorch is used for
device/pinned memory and streams only) and exposes the forward call on device
tensors or host buffers. All arithmetic happens inside libmfet.so.
"""
from __future__ import annotations

import ctypes
import mmap
from typing import List, Optional

import numpy as np
import torch

from . import inputs as gi
from . import mfet as m


class LookupEngine:
    """Tables of a workload placed in HBM / host memory and filled with the
    library's synthetic generator, plus workspace and hot-row cache set-up."""

    def __init__(self, w: gi.Workload, device: int = 0, value_mode: int = m.VAL_NORMAL, fill: bool = True):
        self.w = w
        self.device = device
        torch.cuda.set_device(device)
        self.stream = torch.cuda.current_stream().cuda_stream
        self.mem: List[object] = []
        self._host_maps = []
        descs = []
        for s in w.tables:
            rb = m.row_bytes(s.dim, s.dtype)
            if s.location == gi.LOC_DEVICE:
                buf = torch.empty(s.rows * rb, dtype=torch.uint8, device="cuda:%d" % device)
                descs.append(m.TableDesc(buf.data_ptr(), s.rows, s.dim, s.dtype, m.LOC_DEVICE, 0, s.hash_seed, 0))
                self.mem.append(buf)
            else:
                # anonymous pages; the library pins and maps them when the table is registered
                mm = mmap.mmap(-1, s.rows * rb, flags=mmap.MAP_PRIVATE | mmap.MAP_ANONYMOUS)
                self._host_maps.append(mm)
                descs.append(m.TableDesc(None, s.rows, s.dim, s.dtype, m.LOC_HOST, 0, s.hash_seed, 0))
                self.mem.append(mm)
        self.h = m.mfet_tables_create(descs, device)
        self.ws = None
        self.cache_mem = {}
        for i, s in enumerate(w.tables):
            rb = m.row_bytes(s.dim, s.dtype)
            if s.location == gi.LOC_HOST:
                addr = ctypes.addressof(ctypes.c_char.from_buffer(self.mem[i]))
                m.mfet_host_tables_register(self.h, i, addr, s.rows * rb, 0)
                ptr = addr
            else:
                ptr = self.mem[i].data_ptr()
            if fill:
                m.mfet_table_fill(ptr, 0, s.rows, s.dim, s.dtype, 0, s.value_key, value_mode, self.stream)
        torch.cuda.synchronize()
        self.shape, self._keep = m.make_shape(w.batch, w.n_features, w.slot_feature)

    # ---- set-up -----------------------------------------------------------

    def host_table_ids(self):
        return [i for i, s in enumerate(self.w.tables) if s.location == gi.LOC_HOST]

    def set_workspace(self, max_ids: int) -> None:
        n = m.mfet_workspace_bytes(self.h, max_ids)
        self.ws = torch.empty(max(n, 256), dtype=torch.uint8, device="cuda:%d" % self.device)
        m.mfet_set_workspace(self.h, self.ws, self.ws.numel(), max_ids)

    def build_hot_cache(self, table_id: int, feature: int, n_rows: int) -> int:
        """Cache the rows of the most frequent IDs of `feature`: IDs are taken in
        popularity order and hashed by the library until `n_rows` distinct rows
        are found. Returns the number of cached rows."""
        want = int(n_rows)
        if want <= 0:
            return 0
        count = int(want * 1.05) + 1024
        ids = gi.hot_ids(self.w, feature, count)
        d = torch.from_numpy(ids.view(np.int64)).cuda(self.device)
        m.mfet_hash_ids(self.h, table_id, d, d.numel(), d, self.stream)
        rows = d.cpu().numpy()
        del d
        # the first `want` distinct rows in popularity order, ascending (host-side set-up, numpy)
        uniq, first = np.unique(rows, return_index=True)
        if uniq.size > want:
            bound = np.partition(first, want - 1)[want - 1]
            uniq = uniq[first <= bound]
        rows_sorted = np.ascontiguousarray(uniq, dtype=np.int64)
        nbytes = m.mfet_cache_bytes(self.h, table_id, rows_sorted.size)
        mem = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda:%d" % self.device)
        m.mfet_cache_build(self.h, table_id, rows_sorted, mem, mem.numel(), self.stream)
        self.cache_mem[table_id] = mem
        return int(rows_sorted.size)

    # ---- the call ----------------------------------------------------------

    def forward(self, ids: torch.Tensor, offsets: torch.Tensor, weights: Optional[torch.Tensor],
                out: torch.Tensor, table_ids=None, pooling=None, shape=None) -> None:
        """Asynchronous on the current stream; all tensors live on the engine's GPU."""
        m.mfet_embedding_bag_forward(self.h, shape or self.shape, ids, offsets, weights,
                                     self.w.table_ids if table_ids is None else table_ids,
                                     self.w.pooling if pooling is None else pooling, out, self.stream)

    def close(self) -> None:
        if self.h is not None:
            torch.cuda.synchronize()
            m.mfet_tables_destroy(self.h)
            self.h = None
        self.mem = []
        for mm in self._host_maps:
            try:
                mm.close()
            except BufferError:
                pass
        self._host_maps = []

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()
