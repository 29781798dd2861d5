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
