"""The host-buffer entry points: the asynchronous variant on two streams gives the same bits as
the waiting one and as the device-buffer call."""
import numpy as np
import pytest
import torch

from paper_2508_05700_b200 import inputs as gi
from tests.helpers import DeviceTables, mfet, workload_forward

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("config,rs,bs", [(3, 0.001, 1 / 16), (5, 0.001, 1 / 16)])
def test_async_host_forward_on_two_streams(config, rs, bs):
    m = mfet()
    w = gi.make_workload(config, rows_scale=rs, batch_scale=bs)
    batches = [gi.make_batch(w, j) for j in range(4)]
    with DeviceTables(w.tables) as dt:
        if config == 5:
            dt.set_workspace(max(int(b.offsets[w.batch] - b.offsets[0]) for b in batches) + 1024)
        want = [workload_forward(dt, w, b) for b in batches]
        shape, keep = m.make_shape(w.batch, w.n_features, w.slot_feature)
        nnz = [int(b.offsets[-1]) for b in batches]
        nbytes = max(m.mfet_host_io_bytes(dt.h, shape, w.table_ids, n) for n in nnz)
        lanes = [torch.cuda.Stream(), torch.cuda.Stream()]
        io = [torch.empty(nbytes, dtype=torch.uint8, device="cuda") for _ in lanes]
        outs = [torch.empty(w.batch, w.out_dim, dtype=torch.float32).pin_memory() for _ in batches]
        pin = [(torch.from_numpy(b.ids.view(np.int64)).pin_memory(), torch.from_numpy(b.offsets).pin_memory(),
                None if b.weights is None else torch.from_numpy(b.weights).pin_memory()) for b in batches]
        for j in range(4):
            a = j % 2
            lanes[a].synchronize()
            m.mfet_embedding_bag_forward_host_async(dt.h, shape, pin[j][0], pin[j][1], pin[j][2], nnz[j], w.table_ids,
                                                    w.pooling, outs[j], io[a], nbytes, lanes[a].cuda_stream)
        torch.cuda.synchronize()
        assert m.mfet_query_status(dt.h) == 0
        for j in range(4):
            assert np.array_equal(outs[j].numpy(), want[j]), j
        sync_out = torch.empty(w.batch, w.out_dim, dtype=torch.float32).pin_memory()
        m.mfet_embedding_bag_forward_host(dt.h, shape, pin[0][0], pin[0][1], pin[0][2], nnz[0], w.table_ids, w.pooling,
                                          sync_out, io[0], nbytes, torch.cuda.current_stream().cuda_stream)
        assert np.array_equal(sync_out.numpy(), want[0])
