"""Layout corner cases of the forward call: padded row strides, one table shared by several
features, features read by no slot, a batch of one sample, repeated slots."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_2508_05700_b200 import inputs as gi
from tests.helpers import assert_close, mfet

pytestmark = pytest.mark.gpu


def _ragged(rng, n):
    lens = rng.integers(0, 15, size=n)
    lens[rng.random(n) < 0.2] = 0
    off = np.zeros(n + 1, np.int64)
    np.cumsum(lens, out=off[1:])
    return off


@pytest.mark.parametrize("dtype,dim,pad", [(gi.F32, 32, 16), (gi.BF16, 64, 128), (gi.F16, 24, 16), (gi.INT4, 64, 16)])
def test_padded_row_stride(dtype, dim, pad):
    m = mfet()
    rows, key, seed = 3001, 0xFEEDFACE12345, 0x77
    rb = m.row_bytes(dim, dtype)
    stride = rb + pad
    buf = torch.full((rows * stride,), 0x5A, dtype=torch.uint8, device="cuda")  # padding holds junk
    s = torch.cuda.current_stream().cuda_stream
    m.mfet_table_fill(buf, 0, rows, dim, dtype, stride, key, m.VAL_NORMAL, s)
    h = m.mfet_tables_create([m.TableDesc(buf.data_ptr(), rows, dim, dtype, m.LOC_DEVICE, 0, seed, stride)])
    try:
        rng = np.random.default_rng(dim)
        B = 70
        off = _ragged(rng, B)
        ids = rng.integers(0, 2**40, size=max(int(off[-1]), 1), dtype=np.uint64)
        w = rng.random(ids.size).astype(np.float32)
        out = torch.full((B, dim), float("nan"), device="cuda")
        sh, keep = m.make_shape(B, 1, [0])
        m.mfet_embedding_bag_forward(h, sh, torch.from_numpy(ids.view(np.int64)).cuda(), torch.from_numpy(off).cuda(),
                                     torch.from_numpy(w).cuda(), [0], [m.POOL_WSUM], out, s)
        torch.cuda.synchronize()
        assert m.mfet_query_status(h) == 0
    finally:
        m.mfet_tables_destroy(h)
    ot = orc.Table(rows=rows, dim=dim, dtype=dtype, hash_seed=seed, value_key=key)
    ref = orc.embedding_bag([ot], B, 1, [0], [0], [orc.POOL_WSUM], ids, off, w)
    assert_close(out.cpu().numpy(), ref, "stride %d" % stride)


def test_shared_tables_unused_features_and_single_sample():
    m = mfet()
    specs = [gi.TableSpec(4099, 32, gi.BF16, 11, 101), gi.TableSpec(257, 8, gi.F32, 0, 202)]
    from tests.helpers import DeviceTables, forward
    rng = np.random.default_rng(3)
    with DeviceTables(specs) as dt:
        for B in (1, 2, 65):
            F = 4
            off = _ragged(rng, F * B)
            ids = rng.integers(0, 2**40, size=max(int(off[-1]), 1), dtype=np.uint64)
            w = rng.random(ids.size).astype(np.float32)
            # feature 1 is read by no slot; table 0 serves features 0, 2 and (twice) 3
            sf, ti, po = [0, 2, 2, 3, 3], [0, 0, 1, 0, 0], [0, 1, 2, 2, 0]
            got = forward(dt, B, F, sf, ti, po, ids, off, w)
            ref = orc.embedding_bag(dt.oracle_tables, B, F, sf, ti, po, ids, off, w)
            assert got.shape == (B, 32 + 32 + 8 + 32 + 32)
            assert_close(got, ref, "B=%d" % B)


def test_batch_zero_is_a_no_op():
    m = mfet()
    dummy = torch.zeros(64, dtype=torch.uint8, device="cuda")
    h = m.mfet_tables_create([m.TableDesc(dummy.data_ptr(), 4, 4, m.F32, m.LOC_DEVICE, 0, 0, 0)])
    try:
        n0 = m.mfet_launch_count(h)
        sh, keep = m.make_shape(0, 1, [0])
        m.mfet_embedding_bag_forward(h, sh, None, None, None, [0], [0], None)
        assert m.mfet_launch_count(h) == n0
    finally:
        m.mfet_tables_destroy(h)
