"""Nothing is written outside the arrays that the caller hands over: guard bands with a known bit
pattern sit right before and after the output, the workspace (which holds the staging of fetched
rows), the cache memory and the gradient arrays, the output's padding columns carry the pattern
too, and all of them, and the inputs, must come back unchanged. These tests run on the normal
library and again, from test_gpu_checked_build.py, on the bounds-checked build."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_2508_05700_b200 import inputs as gi
from tests.helpers import DeviceTables, assert_close, mfet, workload_oracle

pytestmark = pytest.mark.gpu

GUARD = 4096          # bytes on either side
PATTERN = 0xA5


def _guarded(nbytes, align=256):
    """(whole buffer, usable view of nbytes starting at a multiple of `align`)."""
    whole = torch.full((GUARD + nbytes + GUARD + align,), PATTERN, dtype=torch.uint8, device="cuda")
    start = GUARD + (-(whole.data_ptr() + GUARD)) % align
    return whole, whole[start:start + nbytes], start


def _intact(whole, start, nbytes):
    h = whole.cpu().numpy()
    return bool((h[:start] == PATTERN).all() and (h[start + nbytes:] == PATTERN).all())


def _stream():
    return torch.cuda.current_stream().cuda_stream


@pytest.mark.parametrize("config,rows_scale,batch_scale,pad", [(3, 1e-3, 1 / 16, 0), (3, 1e-3, 1 / 16, 5), (4, 2e-4, 1 / 64, 3),
                                                              (2, 1e-3, 1 / 8, 1), (1, 1.0, 1.0, 0)])
def test_output_guards_and_padding_columns_stay_untouched(config, rows_scale, batch_scale, pad):
    m = mfet()
    w = gi.make_workload(config, rows_scale=rows_scale, batch_scale=batch_scale)
    b = gi.make_batch(w, 0)
    ld = w.out_dim + pad
    with DeviceTables(w.tables) as dt:
        whole, view, start = _guarded(w.batch * ld * 4, align=4 if pad else 256)
        out = view.view(torch.float32).view(w.batch, ld)
        d_ids = torch.from_numpy(b.ids.view(np.int64)).cuda()
        d_off = torch.from_numpy(b.offsets).cuda()
        d_w = None if b.weights is None else torch.from_numpy(b.weights).cuda()
        shape, keep = m.make_shape(w.batch, w.n_features, w.slot_feature, out_ld=ld)
        for overlap in (0, 1):
            m.mfet_set_option(dt.h, m.OPT_OVERLAP_LAUNCHES, overlap)
            m.mfet_embedding_bag_forward(dt.h, shape, d_ids, d_off, d_w, w.table_ids, w.pooling, out, _stream())
            m.mfet_embedding_bag_forward(dt.h, shape, d_ids, d_off, d_w, w.table_ids, w.pooling, out, _stream())
        torch.cuda.synchronize()
        assert m.mfet_query_status(dt.h) == 0
        assert _intact(whole, start, w.batch * ld * 4)
        got = out.cpu().numpy()
        if pad:
            assert (got[:, w.out_dim:].view(np.uint8) == PATTERN).all()
        assert_close(got[:, :w.out_dim], workload_oracle(dt, w, b))
        assert np.array_equal(d_ids.cpu().numpy(), b.ids.view(np.int64)) and np.array_equal(d_off.cpu().numpy(), b.offsets)


def test_workspace_cache_and_gradient_guards_stay_untouched():
    m = mfet()
    w = gi.make_workload(5, rows_scale=0.001, batch_scale=0.125)
    bs = [gi.make_batch(w, j) for j in range(3)]
    n_host = max(int(b.offsets[w.batch] - b.offsets[0]) for b in bs)
    cap = n_host + 17
    with DeviceTables(w.tables) as dt:
        ws_bytes = m.mfet_workspace_bytes(dt.h, cap)
        ws_whole, ws, ws_start = _guarded(ws_bytes)
        m.mfet_set_workspace(dt.h, ws, ws_bytes, cap)
        # hot-row cache in guarded memory
        hot = gi.hot_ids(w, 0, int(w.tables[0].rows * 0.02))
        rows = np.unique(orc.hash_ids(hot, w.tables[0].hash_seed, w.tables[0].rows))
        c_bytes = m.mfet_cache_bytes(dt.h, 0, rows.size)
        c_whole, cache, c_start = _guarded(c_bytes)
        m.mfet_cache_build(dt.h, 0, rows, cache, c_bytes, _stream())
        shape, keep = m.make_shape(w.batch, w.n_features, w.slot_feature)
        pre, keep2 = m.make_shape(w.batch, w.n_features, w.slot_feature)
        pre.flags |= m.BATCH_PREFETCHED
        out = torch.empty(w.batch, w.out_dim, dtype=torch.float32, device="cuda")
        dev = [(torch.from_numpy(b.ids.view(np.int64)).cuda(), torch.from_numpy(b.offsets).cuda()) for b in bs]
        # serial path, then the pipelined one (second result set of the workspace)
        m.mfet_embedding_bag_forward(dt.h, shape, dev[0][0], dev[0][1], None, w.table_ids, w.pooling, out, _stream())
        torch.cuda.synchronize()
        assert_close(out.cpu().numpy(), workload_oracle(dt, w, bs[0]))
        m.mfet_host_prefetch(dt.h, shape, dev[1][0], dev[1][1], w.table_ids, _stream())
        m.mfet_host_prefetch(dt.h, shape, dev[2][0], dev[2][1], w.table_ids, _stream())
        for j in (1, 2):
            m.mfet_embedding_bag_forward(dt.h, pre, dev[j][0], dev[j][1], None, w.table_ids, w.pooling, out, _stream())
            torch.cuda.synchronize()
            assert_close(out.cpu().numpy(), workload_oracle(dt, w, bs[j]))
        # dedup and backward through the same workspace, results in guarded arrays
        r = torch.from_numpy(orc.hash_ids(bs[0].ids[:n_host // 2], 0, 10**6)).cuda()
        u_whole, uniq, u_start = _guarded(r.numel() * 8)
        i_whole, inv, i_start = _guarded(r.numel() * 4)
        nu = torch.zeros(1, dtype=torch.int64, device="cuda")
        m.mfet_dedup_rows(dt.h, r, r.numel(), uniq, inv, nu, 10**6, _stream())
        n_f = int(bs[0].offsets[w.batch] - bs[0].offsets[0])
        gr_whole, g_rows, gr_start = _guarded(n_f * 8)
        gv_whole, g_vals, gv_start = _guarded(n_f * 64 * 4)
        g = torch.randn(w.batch, w.out_dim, device="cuda")
        m.mfet_embedding_bag_backward(dt.h, shape, dev[0][0], dev[0][1], None, w.table_ids, w.pooling, g, 0, g_rows, g_vals,
                                      nu, _stream())
        torch.cuda.synchronize()
        assert m.mfet_query_status(dt.h) == 0
        assert _intact(ws_whole, ws_start, ws_bytes), "workspace guard"
        assert _intact(c_whole, c_start, c_bytes), "cache guard"
        assert _intact(u_whole, u_start, r.numel() * 8) and _intact(i_whole, i_start, r.numel() * 4), "dedup outputs"
        assert _intact(gr_whole, gr_start, n_f * 8) and _intact(gv_whole, gv_start, n_f * 64 * 4), "gradient outputs"


def test_checked_build_reports_a_row_outside_the_table_and_skips_it():
    """Only on the bounds-checked build: a row list for mfet_host_fetch_rows with an index beyond the
    table sets MFET_DEV_BOUNDS, the entry is skipped (zeros) and the other rows arrive."""
    m = mfet()
    if "checked" not in m.LIB_PATH:
        pytest.skip("needs the bounds-checked build of the library (MFET_LIBRARY)")
    spec = gi.TableSpec(64, 8, gi.F16, 0, 0x99, gi.LOC_HOST)
    with DeviceTables([spec]) as dt:
        rows = torch.tensor([3, 64 + 5, 63], dtype=torch.int64, device="cuda")
        dst = torch.full((3 * 16,), 0xEE, dtype=torch.uint8, device="cuda")
        m.mfet_host_fetch_rows(dt.h, 0, rows, 3, dst, _stream())
        torch.cuda.synchronize()
        assert m.mfet_query_status(dt.h, clear=True) == m.DEV_BOUNDS
        got = dst.cpu().numpy().reshape(3, 16)
        host = dt.mem[0].numpy().reshape(64, 16)
        assert np.array_equal(got[0], host[3]) and np.array_equal(got[2], host[63]) and not got[1].any()
