"""Sparse table gradients on the GPU against the oracle's dense scatter-add (paper, Section 4.3:
the tables are fine-tuned, so gradients flow to the looked-up rows)."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_2508_05700_b200 import inputs as gi
from tests.helpers import DeviceTables, mfet

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("config,rows_scale,batch_scale", [(3, 2e-5, 1 / 16), (2, 1e-4, 1 / 8), (4, 5e-5, 1 / 64)])
def test_backward_matches_oracle(config, rows_scale, batch_scale):
    m = mfet()
    w = gi.make_workload(config, rows_scale=rows_scale, batch_scale=batch_scale)
    b = gi.make_batch(w, 0)
    rng = np.random.default_rng(config)
    gout = (0.01 * rng.standard_normal((w.batch, w.out_dim))).astype(np.float32)
    cap = int(np.diff(b.offsets.reshape(-1)[::w.batch]).max()) + 64
    with DeviceTables(w.tables) as dt:
        dt.set_workspace(cap)
        d_ids = torch.from_numpy(b.ids.view(np.int64)).cuda()
        d_off = torch.from_numpy(b.offsets).cuda()
        d_w = None if b.weights is None else torch.from_numpy(b.weights).cuda()
        d_g = torch.from_numpy(gout).cuda()
        shape, keep = m.make_shape(w.batch, w.n_features, w.slot_feature)
        col = 0
        for s in range(w.n_slots):
            t = w.tables[int(w.table_ids[s])]
            if s in (0, w.n_slots - 1, w.n_slots // 2):
                rows = torch.full((cap,), -1, dtype=torch.int64, device="cuda")
                vals = torch.full((cap, t.dim), float("nan"), dtype=torch.float32, device="cuda")
                nr = torch.zeros(1, dtype=torch.int64, device="cuda")
                m.mfet_embedding_bag_backward(dt.h, shape, d_ids, d_off, d_w, w.table_ids, w.pooling, d_g, s, rows,
                                              vals, nr, torch.cuda.current_stream().cuda_stream)
                torch.cuda.synchronize()
                assert m.mfet_query_status(dt.h) == 0
                k = int(nr.item())
                got_rows = rows[:k].cpu().numpy()
                got = vals[:k].cpu().numpy().astype(np.float64)
                ref = orc.embedding_bag_backward_slot(dt.oracle_tables, w.batch, w.slot_feature, w.table_ids, w.pooling,
                                                      s, w.out_dim, col, b.ids, b.offsets, b.weights, gout)
                f = int(w.slot_feature[s])
                want_rows = np.unique(orc.hash_ids(b.ids[b.offsets[f * w.batch]:b.offsets[(f + 1) * w.batch]],
                                                   t.hash_seed, t.rows))
                assert np.array_equal(got_rows, want_rows)          # bit-exact index work
                touched = np.zeros(t.rows, bool)
                touched[got_rows] = True
                assert not ref[~touched].any()                      # rows outside the list have zero gradient
                # a hot row sums thousands of signed terms: the fp32 error scales with the sum of their
                # magnitudes, which the oracle gives when fed |grad_out| and |weights|
                mass = orc.embedding_bag_backward_slot(dt.oracle_tables, w.batch, w.slot_feature, w.table_ids,
                                                       w.pooling, s, w.out_dim, col, b.ids, b.offsets,
                                                       None if b.weights is None else np.abs(b.weights), np.abs(gout))
                err = np.abs(got - ref[got_rows])
                assert np.isfinite(got).all()
                assert (err <= 1e-6 + 1e-5 * mass[got_rows]).all(), float((err / (1e-6 + 1e-5 * mass[got_rows])).max())
            col += t.dim


@pytest.mark.parametrize("B,max_len,rows,dim,pool", [(300, 40, 7, 136, 2), (300, 40, 1, 8, 1), (3, 4, 5, 264, 0),
                                                    (64, 300, 3, 32, 0), (5000, 6, 2, 136, 1), (1025, 30, 3, 72, 2),
                                                    (2048, 12, 40, 128, 0)])
def test_backward_hot_rows_and_tiny_workspaces(B, max_len, rows, dim, pool):
    """A few rows that receive hundreds or thousands of lookups each (their runs are summed in pieces
    by many warps and combined; runs of more than 32 pieces by a whole block), more than 128 columns,
    column counts that are no multiple of 32, batches of more than 1024 samples (the bag search then
    starts in an excerpt of the offsets) and a workspace too small to hold partial sums (then one warp
    sums everything): the sparse gradient against the oracle's dense scatter-add."""
    m = mfet()
    rng = np.random.default_rng(B * 1000 + dim)
    spec = gi.TableSpec(rows, dim, gi.F32, 0x5EED, 0x1234)
    lens = rng.integers(0, max_len + 1, size=B)
    off = np.zeros(B + 1, np.int64)
    np.cumsum(lens, out=off[1:])
    n = int(off[-1])
    ids = rng.integers(0, 2**40, size=n, dtype=np.uint64)
    wts = rng.random(n).astype(np.float32)
    gout = (0.01 * rng.standard_normal((B, dim))).astype(np.float32)
    with DeviceTables([spec]) as dt:
        dt.set_workspace(max(n, 1))
        shape, keep = m.make_shape(B, 1, [0])
        g_rows = torch.full((max(n, 1),), -1, dtype=torch.int64, device="cuda")
        g_vals = torch.full((max(n, 1), dim), float("nan"), dtype=torch.float32, device="cuda")
        nr = torch.zeros(1, dtype=torch.int64, device="cuda")
        d_ids = torch.from_numpy(ids.view(np.int64)).cuda() if n else torch.zeros(1, dtype=torch.int64, device="cuda")
        m.mfet_embedding_bag_backward(dt.h, shape, d_ids, torch.from_numpy(off).cuda(), torch.from_numpy(wts).cuda()
                                      if n else torch.zeros(1, device="cuda"), [0], [pool], torch.from_numpy(gout).cuda(),
                                      0, g_rows, g_vals, nr, torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert m.mfet_query_status(dt.h) == 0
        k = int(nr.item())
        got_rows, got = g_rows[:k].cpu().numpy(), g_vals[:k].cpu().numpy().astype(np.float64)
        ref = orc.embedding_bag_backward_slot(dt.oracle_tables, B, [0], [0], [pool], 0, dim, 0, ids, off, wts, gout)
        mass = orc.embedding_bag_backward_slot(dt.oracle_tables, B, [0], [0], [pool], 0, dim, 0, ids, off, wts,
                                               np.abs(gout))
        assert np.array_equal(got_rows, np.unique(orc.hash_ids(ids, spec.hash_seed, rows)))
        err = np.abs(got - ref[got_rows])
        assert np.isfinite(got).all()
        assert (err <= 1e-6 + 1e-5 * mass[got_rows]).all(), float((err / (1e-6 + 1e-5 * mass[got_rows])).max())
        again = torch.full_like(g_vals, float("nan"))
        m.mfet_embedding_bag_backward(dt.h, shape, d_ids, torch.from_numpy(off).cuda(), torch.from_numpy(wts).cuda()
                                      if n else torch.zeros(1, device="cuda"), [0], [pool], torch.from_numpy(gout).cuda(),
                                      0, g_rows, again, nr, torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert torch.equal(again[:k], g_vals[:k])  # the order of the additions is fixed
