"""GPU parity: every result of the CUDA library is compared with the CPU oracle on
the same seeded inputs, through the C-ABI binding. Indices and dedup output are
bit-exact; pooled fp32 outputs are within |gpu - ref| <= 1e-6 + 1e-5*|ref|."""
import os

import numpy as np
import pytest
import torch

import oracle as orc
from paper_2508_05700_b200 import inputs as gi
from tests.helpers import (DeviceTables, assert_close, forward, mfet, workload_forward, workload_oracle)

pytestmark = pytest.mark.gpu
GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _stream():
    return torch.cuda.current_stream().cuda_stream


# ------------------------------------------------------------------ hash ----

@pytest.mark.parametrize("rows", [1, 7, 100_000, 10_000_000, 50_000_000, 10**9, 2**32 - 1, 2**32, 2**32 + 1,
                                  2**40 + 12345, 2**63 - 1])
def test_hash_ids_bit_exact(rows):
    m = mfet()
    rng = np.random.default_rng(rows % 1000)
    n = 300_001
    ids = rng.integers(0, 2**64 - 1, size=n, dtype=np.uint64)
    ids[:6] = [0, 1, 2, 2**40 - 1, 2**63, 2**64 - 1]
    seed = 0 if rows in (1, 100_000) else 0x5DEECE66D1234567
    dummy = torch.zeros(16, dtype=torch.uint8, device="cuda")
    h = m.mfet_tables_create([m.TableDesc(dummy.data_ptr(), rows, 4, m.F32, m.LOC_DEVICE, 0, seed, 0)])
    try:
        d_ids = torch.from_numpy(ids.view(np.int64)).cuda()
        d_rows = torch.empty(n, dtype=torch.int64, device="cuda")
        m.mfet_hash_ids(h, 0, d_ids, n, d_rows, _stream())
        got = d_rows.cpu().numpy()
        assert np.array_equal(got, orc.hash_ids(ids, seed, rows))
        # in place
        m.mfet_hash_ids(h, 0, d_ids, n, d_ids, _stream())
        assert np.array_equal(d_ids.cpu().numpy(), got)
        m.mfet_hash_ids(h, 0, None, 0, None, _stream())  # n = 0 is a no-op
    finally:
        m.mfet_tables_destroy(h)


def _ids_that_hash_to(values, seed):
    """Raw IDs whose splitmix64(id ^ seed) is exactly `values`: the generator's output function is a
    bijection of 64-bit words (xor-shifts and odd multipliers), inverted here step by step in python
    integers. Test-side only: it lets the test choose the number that goes INTO the modulo."""
    M = (1 << 64) - 1

    def unshift(y, s):
        x = y
        for _ in range(64 // s + 1):
            x = y ^ (x >> s)
        return x
    inv1, inv2 = pow(0xBF58476D1CE4E5B9, -1, 1 << 64), pow(0x94D049BB133111EB, -1, 1 << 64)
    out = []
    for v in values:
        z = unshift(int(v), 31)
        z = (z * inv2) & M
        z = unshift(z, 27)
        z = (z * inv1) & M
        z = unshift(z, 30)
        out.append(((z - 0x9E3779B97F4A7C15) & M) ^ seed)
    return np.array(out, dtype=np.uint64)


@pytest.mark.parametrize("rows", [1, 2, 3, 10, 100_000, 50_000_000, 10**9, 2**31, 2**32 - 1, 2**32, 2**32 + 1, 3 * 2**40 + 7,
                                  2**62, 2**62 + 1, 2**63 - 1])
def test_hash_modulo_at_chosen_hash_values(rows):
    """The exact modulo on the values where a reciprocal-based remainder can go wrong: hash values at
    and around multiples of `rows`, at the top of the 64-bit range, and around 2^32 and 2^63. The IDs
    are constructed so that their hash IS the chosen value (checked through the oracle's own hash)."""
    m = mfet()
    seed = 0x243F6A8885A308D3
    M64 = 1 << 64
    want_h = {0, 1, rows - 1, rows, rows + 1, 2 * rows - 1, 2 * rows, M64 - 1, M64 - 2, M64 - rows, (M64 - 1) // rows * rows,
              (M64 - 1) // rows * rows - 1, (M64 - 1) // rows * rows + rows - 1, 2**32 - 1, 2**32, 2**63 - 1, 2**63, 2**63 + 1}
    rng = np.random.default_rng(rows % 977)
    for _ in range(3000):  # multiples of rows, plus and minus one, all over the range
        q = int(rng.integers(0, M64 // rows, dtype=np.uint64)) if rows < M64 // 2 else int(rng.integers(0, 2))
        want_h.update({q * rows - 1, q * rows, q * rows + 1, q * rows + rows - 1})
    hs = sorted(v for v in want_h if 0 <= v < M64)
    ids = _ids_that_hash_to(hs, seed)
    assert [orc.splitmix64(int(i) ^ seed) for i in ids[:50]] == hs[:50]  # the construction, against the oracle's hash
    dummy = torch.zeros(16, dtype=torch.uint8, device="cuda")
    h = m.mfet_tables_create([m.TableDesc(dummy.data_ptr(), rows, 4, m.F32, m.LOC_DEVICE, 0, seed, 0)])
    try:
        d_ids = torch.from_numpy(ids.view(np.int64)).cuda()
        d_rows = torch.empty(ids.size, dtype=torch.int64, device="cuda")
        m.mfet_hash_ids(h, 0, d_ids, ids.size, d_rows, _stream())
        got = d_rows.cpu().numpy()
        assert np.array_equal(got, orc.hash_ids(ids, seed, rows))
        assert np.array_equal(got, np.array([v % rows for v in hs], dtype=np.int64))  # and against the plain definition
    finally:
        m.mfet_tables_destroy(h)


@pytest.mark.parametrize("n", [1, 2, 3, 511, 513, 100_000, 100_001])
@pytest.mark.parametrize("shift_in,shift_out", [(0, 0), (1, 0), (0, 1), (1, 1)])
def test_hash_ids_any_length_and_alignment(n, shift_in, shift_out):
    """The hash kernel pairs IDs up when both arrays are 16-byte aligned and falls back to single
    IDs otherwise; odd lengths and 8-byte-aligned arrays give the same rows."""
    m = mfet()
    rng = np.random.default_rng(n + 10 * shift_in + 100 * shift_out)
    rows, seed = 50_000_000, 0xC0FFEE
    ids = rng.integers(0, 2**64 - 1, size=n, dtype=np.uint64)
    dummy = torch.zeros(16, dtype=torch.uint8, device="cuda")
    h = m.mfet_tables_create([m.TableDesc(dummy.data_ptr(), rows, 4, m.F32, m.LOC_DEVICE, 0, seed, 0)])
    try:
        buf_in = torch.zeros(n + 2, dtype=torch.int64, device="cuda")
        buf_out = torch.full((n + 2,), -7, dtype=torch.int64, device="cuda")
        d_ids = buf_in[shift_in:shift_in + n]
        d_ids.copy_(torch.from_numpy(ids.view(np.int64)))
        d_rows = buf_out[shift_out:shift_out + n]
        m.mfet_hash_ids(h, 0, d_ids, n, d_rows, _stream())
        assert np.array_equal(d_rows.cpu().numpy(), orc.hash_ids(ids, seed, rows))
        out = buf_out.cpu().numpy()
        assert (out[:shift_out] == -7).all() and (out[shift_out + n:] == -7).all()  # nothing written outside
    finally:
        m.mfet_tables_destroy(h)


# ------------------------------------------------------------------ fill ----

@pytest.mark.parametrize("dtype", [gi.F32, gi.F16, gi.BF16])
@pytest.mark.parametrize("mode", [0, 1])
def test_table_fill_bit_exact(dtype, mode):
    m = mfet()
    rows, dim, key = 5003, 40, 0x1234ABCD9876FEDB
    rb = m.row_bytes(dim, dtype)
    buf = torch.zeros(rows * rb, dtype=torch.uint8, device="cuda")
    m.mfet_table_fill(buf, 0, rows, dim, dtype, 0, key, mode, _stream())
    got = buf.cpu().numpy().reshape(rows, rb)
    want = orc.table_fill(orc.Table(rows=rows, dim=dim, dtype=dtype, value_key=key, value_mode=mode))
    assert np.array_equal(got, want)
    # a sub-range (rows 4000..4099 land at data + r*stride) with a padded stride
    stride = rb + 32
    buf2 = torch.zeros(100 * stride, dtype=torch.uint8, device="cuda")
    m.mfet_table_fill(buf2.data_ptr() - 4000 * stride, 4000, 100, dim, dtype, stride, key, mode, _stream())
    got2 = buf2.cpu().numpy().reshape(100, stride)
    assert np.array_equal(got2[:, :rb], want[4000:4100])
    assert not got2[:, rb:].any()


def test_table_fill_frozen_literals():
    m = mfet()
    with open(os.path.join(GOLD, "table_values.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            key, mode, dim, dtype, r, d, bits = (int(x, 0) for x in line.split())
            rb = m.row_bytes(dim, dtype)
            buf = torch.zeros(rb, dtype=torch.uint8, device="cuda")
            m.mfet_table_fill(buf.data_ptr() - r * rb, r, 1, dim, dtype, 0, key, mode, _stream())
            raw = buf.cpu().numpy()
            got = int(raw.view(np.uint32)[d]) if dtype == gi.F32 else int(raw.view(np.uint16)[d])
            assert got == bits, line


# ----------------------------------------------------------- dtype decode ---

@pytest.mark.parametrize("dtype", [gi.F16, gi.BF16])
def test_decode_all_16bit_patterns(dtype):
    """Every finite 16-bit pattern decodes on the GPU to the oracle's fp32 bits
    (single-ID bags, pre-hashed row indices, so the output is the row itself)."""
    m = mfet()
    pat = np.arange(65536, dtype=np.uint16).reshape(8192, 8)
    tab = torch.from_numpy(pat.view(np.int16).copy()).cuda()
    h = m.mfet_tables_create([m.TableDesc(tab.data_ptr(), 8192, 8, dtype, m.LOC_DEVICE, 0, 0, 0)])
    try:
        ids = torch.arange(8192, dtype=torch.int64, device="cuda")
        off = torch.arange(8193, dtype=torch.int64, device="cuda")
        out = torch.empty(8192, 8, dtype=torch.float32, device="cuda")
        shape, keep = m.make_shape(8192, 1, [0], ids_are_rows=True)
        m.mfet_embedding_bag_forward(h, shape, ids, off, None, [0], [m.POOL_SUM], out, _stream())
        got = out.cpu().numpy().view(np.uint32).reshape(-1)
    finally:
        m.mfet_tables_destroy(h)
    conv = orc.f16_bits_to_f32_bits if dtype == gi.F16 else orc.bf16_bits_to_f32_bits
    want = np.array([conv(int(x)) for x in range(65536)], np.uint32)
    finite = np.isfinite(want.view(np.float32)) & (want != 0x80000000)  # 0 + (-0) = +0 on both sides
    assert np.array_equal(got[finite], want[finite])
    assert (got[want == 0x80000000] == 0).all()


# ------------------------------------------------------------ tiny cases ----

def _mat_tables(tabs, dtypes, seeds=None):
    """Materialised tables (numpy fp32 [rows, dim]) -> (device handle pieces, oracle tables)."""
    m = mfet()
    dev, descs, otabs = [], [], []
    for i, (x, dt) in enumerate(zip(tabs, dtypes)):
        x = np.ascontiguousarray(x, np.float32)
        if dt == gi.F32:
            raw = x
        elif dt == gi.F16:
            raw = x.astype(np.float16)
        else:
            raw = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy()
        raw = np.ascontiguousarray(raw)
        d = torch.from_numpy(raw.view(np.uint8).reshape(-1).copy()).cuda()
        seed = seeds[i] if seeds else 0
        dev.append(d)
        descs.append(m.TableDesc(d.data_ptr(), x.shape[0], x.shape[1], dt, m.LOC_DEVICE, 0, seed, 0))
        otabs.append(orc.Table(rows=x.shape[0], dim=x.shape[1], dtype=dt, hash_seed=seed, data=raw))
    return dev, descs, otabs


class _Mat:
    def __init__(self, tabs, dtypes, seeds=None):
        self.m = mfet()
        self.dev, descs, self.oracle_tables = _mat_tables(tabs, dtypes, seeds)
        self.specs = [gi.TableSpec(t.shape[0], t.shape[1], dt, 0, 0) for t, dt in zip(tabs, dtypes)]
        self.h = self.m.mfet_tables_create(descs)

    def close(self):
        torch.cuda.synchronize()
        self.m.mfet_tables_destroy(self.h)


@pytest.mark.parametrize("dtype", [gi.F32, gi.F16, gi.BF16])
def test_hand_computed_tiny_bags(dtype):
    g = {}
    with open(os.path.join(GOLD, "tiny_bags.txt")) as fh:
        for line in fh:
            if not line.startswith("#") and line.strip():
                k, *v = line.split()
                g[k] = np.array([float(x) for x in v])
    D = 8  # rows must be a multiple of 16 bytes: the 2 real columns are padded with zeros
    tab = np.zeros((4, D), np.float32)
    tab[:, :2] = g["table"].reshape(4, 2)
    mt = _Mat([tab], [dtype])
    try:
        for pool, key in ((0, "sum"), (1, "mean"), (2, "wsum")):
            out = forward(mt, 3, 1, [0], [0], [pool], g["ids"].astype(np.uint64), g["offsets"].astype(np.int64),
                          g["weights"].astype(np.float32), ids_are_rows=True)
            assert np.array_equal(out[:, :2], g[key].reshape(3, 2).astype(np.float32)), key
            assert not out[:, 2:].any()
    finally:
        mt.close()


def _ragged(rng, n_bags, pattern):
    if pattern == "mixed":
        lens = rng.integers(0, 12, size=n_bags)
        lens[rng.random(n_bags) < 0.25] = 0
        lens[rng.integers(0, n_bags, 5)] = rng.integers(33, 300, 5)
    elif pattern == "ones":
        lens = np.ones(n_bags, np.int64)
    elif pattern == "empty_edges":
        lens = rng.integers(1, 9, size=n_bags)
        lens[0] = lens[-1] = lens[n_bags // 2] = 0
    elif pattern == "all_empty":
        lens = np.zeros(n_bags, np.int64)
    elif pattern == "long":
        lens = rng.integers(30, 700, size=n_bags)
    else:
        raise ValueError(pattern)
    off = np.zeros(n_bags + 1, np.int64)
    np.cumsum(lens, out=off[1:])
    return off


@pytest.mark.parametrize("dtype,dim", [(gi.F32, 4), (gi.F32, 32), (gi.F32, 20), (gi.F16, 8), (gi.F16, 64),
                                       (gi.BF16, 32), (gi.BF16, 64), (gi.BF16, 128), (gi.BF16, 24),
                                       (gi.F16, 256), (gi.F32, 128), (gi.BF16, 520), (gi.F32, 260)])
@pytest.mark.parametrize("pattern", ["mixed", "ones", "empty_edges", "all_empty", "long"])
@pytest.mark.parametrize("policy", [0, 1, 2])
def test_unit_parity(dtype, dim, pattern, policy):
    rng = np.random.default_rng(dim * 7 + dtype)
    rows = 16 if pattern != "long" else 977
    B = 77 if pattern != "long" else 19
    tab = (0.01 * rng.standard_normal((rows, dim))).astype(np.float32)  # the workloads' value scale
    mt = _Mat([tab], [dtype], seeds=[0xABCDEF])
    try:
        mt.m.mfet_set_option(mt.h, mt.m.OPT_GROUP_POLICY, policy)
        off = _ragged(rng, B, pattern)
        ids = rng.integers(0, 2**40, size=int(off[-1]), dtype=np.uint64)
        if ids.size > 4:
            ids[1] = ids[0]  # duplicate inside a bag
        w = rng.random(ids.size).astype(np.float32)
        for pool in (0, 1, 2):
            got = forward(mt, B, 1, [0], [0], [pool], ids, off, w)
            ref = orc.embedding_bag(mt.oracle_tables, B, 1, [0], [0], [pool], ids, off, w)
            assert_close(got, ref, "pool %d" % pool)
            lens = np.diff(off)
            assert not got[lens == 0].any()
    finally:
        mt.close()


@pytest.mark.parametrize("stage", [32, 100, 2048])
@pytest.mark.parametrize("tile", [8, 32, 128])
@pytest.mark.parametrize("dtype,dim", [(gi.BF16, 64), (gi.F16, 32), (gi.F32, 128), (gi.BF16, 24)])
def test_staging_windows_cut_bags_anywhere(stage, tile, dtype, dim):
    """A tile with more IDs than the staging capacity is pooled in several passes: bags cut by a
    pass boundary (once or many times), empty bags on a boundary and tiles that end on one give
    the oracle's result for every pooling, whatever the capacity and the tile size."""
    rng = np.random.default_rng(stage * 131 + tile * 7 + dim)
    B = 150
    lens = rng.integers(0, 40, size=B)
    lens[rng.random(B) < 0.2] = 0
    # bags that fill whole passes (at most 700 IDs: the fp32 tolerance is derived for bags of that size)
    lens[[3, 77, 149]] = [min(stage, 600), min(3 * stage + 5, 700), min(2 * stage, 650)]
    lens[[4, 5]] = 0  # empty bags right behind one
    off = np.zeros(B + 1, np.int64)
    np.cumsum(lens, out=off[1:])
    tab = (0.01 * rng.standard_normal((211, dim))).astype(np.float32)
    mt = _Mat([tab], [dtype], seeds=[0x5EED])
    try:
        mt.m.mfet_set_option(mt.h, mt.m.OPT_TILE, tile)
        mt.m.mfet_set_option(mt.h, mt.m.OPT_STAGE_IDS, stage)
        ids = rng.integers(0, 2**40, size=int(off[-1]), dtype=np.uint64)
        w = rng.random(ids.size).astype(np.float32)
        for pool in (0, 1, 2):
            got = forward(mt, B, 1, [0], [0], [pool], ids, off, w)
            ref = orc.embedding_bag(mt.oracle_tables, B, 1, [0], [0], [pool], ids, off, w)
            assert_close(got, ref, "pool %d" % pool)
            assert not got[lens == 0].any()
        assert mt.m.mfet_query_status(mt.h, clear=True) == 0
    finally:
        mt.close()


def test_stage_option_range():
    mt = _Mat([np.zeros((4, 8), np.float32)], [gi.F32])
    try:
        m = mt.m
        for bad in (1, 31, 8193, -5):
            with pytest.raises(m.MfetError):
                m.mfet_set_option(mt.h, m.OPT_STAGE_IDS, bad)
        for good in (0, 32, 8192):
            m.mfet_set_option(mt.h, m.OPT_STAGE_IDS, good)
    finally:
        mt.close()


@pytest.mark.parametrize("stage", [4095, 5755, 6000, 6144, 8192])
def test_large_staging_capacities_launch(stage):
    """Staging capacities whose shared memory per block lies just under, around and above 48 KB
    (static and dynamic together; a weighted slot stages 8 bytes per ID): the launch is accepted
    and matches the oracle."""
    rng = np.random.default_rng(stage)
    B = 300
    lens = rng.integers(0, 60, size=B)
    off = np.zeros(B + 1, np.int64)
    np.cumsum(lens, out=off[1:])
    tab = (0.01 * rng.standard_normal((509, 64))).astype(np.float32)
    mt = _Mat([tab], [gi.BF16], seeds=[77])
    try:
        mt.m.mfet_set_option(mt.h, mt.m.OPT_STAGE_IDS, stage)
        ids = rng.integers(0, 2**40, size=int(off[-1]), dtype=np.uint64)
        w = rng.random(ids.size).astype(np.float32)
        for pool in (0, 2):
            got = forward(mt, B, 1, [0], [0], [pool], ids, off, w)
            ref = orc.embedding_bag(mt.oracle_tables, B, 1, [0], [0], [pool], ids, off, w)
            assert_close(got, ref, "stage %d pool %d" % (stage, pool))
    finally:
        mt.close()


@pytest.mark.parametrize("tile", [8, 16, 0])
def test_many_tiles_per_slot_at_full_batch(tile):
    """Workload 3 at its full batch over small tables, cut into many more tiles than the GPU
    keeps resident: whole output against the oracle for two batches in a row, and the bits of
    the first batch repeat."""
    w = gi.make_workload(3, rows_scale=2e-4, batch_scale=1.0)
    b0, b1 = gi.make_batch(w, 0), gi.make_batch(w, 1)
    with DeviceTables(w.tables) as dt:
        if tile:
            dt.m.mfet_set_option(dt.h, dt.m.OPT_TILE, tile)
        first = workload_forward(dt, w, b0)
        assert_close(first, workload_oracle(dt, w, b0), "first call")
        second = workload_forward(dt, w, b1)
        assert_close(second, workload_oracle(dt, w, b1), "second call")
        again = workload_forward(dt, w, b0)
        assert np.array_equal(first.view(np.uint32), again.view(np.uint32))


def test_overlapping_launches_give_the_same_bits():
    """MFET_OPT_OVERLAP_LAUNCHES: back-to-back forward calls on one stream, into the same output buffer
    and into different ones, with a consumer kernel between them; every result has the bits of the
    serialised launches and matches the oracle."""
    w = gi.make_workload(3, rows_scale=1e-3, batch_scale=1 / 8)
    bs = [gi.make_batch(w, j) for j in range(4)]
    with DeviceTables(w.tables) as dt:
        m = dt.m
        serial = [workload_forward(dt, w, b) for b in bs]
        assert_close(serial[0], workload_oracle(dt, w, bs[0]))
        m.mfet_set_option(dt.h, m.OPT_OVERLAP_LAUNCHES, 1)
        d = [(torch.from_numpy(b.ids.view(np.int64)).cuda(), torch.from_numpy(b.offsets).cuda(),
              torch.from_numpy(b.weights).cuda()) for b in bs]
        shape, keep = m.make_shape(w.batch, w.n_features, w.slot_feature)
        torch.cuda.synchronize()
        s = _stream()
        out = torch.empty(w.batch, w.out_dim, dtype=torch.float32, device="cuda")
        copies = []
        for rep in range(3):
            for j in range(4):
                m.mfet_embedding_bag_forward(dt.h, shape, d[j][0], d[j][1], d[j][2], w.table_ids, w.pooling, out, s)
                copies.append((j, out.clone()))  # a kernel that reads the result, between two forward calls
        outs = [torch.empty_like(out) for _ in range(4)]
        for j in range(4):  # and directly back to back into different buffers
            m.mfet_embedding_bag_forward(dt.h, shape, d[j][0], d[j][1], d[j][2], w.table_ids, w.pooling, outs[j], s)
        torch.cuda.synchronize()
        assert m.mfet_query_status(dt.h) == 0
        for j, c in copies:
            assert np.array_equal(c.cpu().numpy(), serial[j]), j
        for j in range(4):
            assert np.array_equal(outs[j].cpu().numpy(), serial[j]), j
        with pytest.raises(m.MfetError):
            m.mfet_set_option(dt.h, m.OPT_OVERLAP_LAUNCHES, 2)


def test_single_row_table_and_prehashed_rows():
    rng = np.random.default_rng(3)
    tab = rng.standard_normal((1, 32)).astype(np.float32)
    mt = _Mat([tab], [gi.F32], seeds=[77])
    try:
        off = np.array([0, 3, 3, 10], np.int64)
        ids = rng.integers(0, 2**40, size=10, dtype=np.uint64)
        got = forward(mt, 3, 1, [0], [0], [0], ids, off, None)
        assert_close(got, np.stack([3 * tab[0], 0 * tab[0], 7 * tab[0]]))
    finally:
        mt.close()


def test_grid_tables_are_bit_exact_in_any_order():
    """Grid-valued tables make every unweighted sum exact in fp32, so GPU and oracle agree bit for bit."""
    w = gi.make_workload(2, rows_scale=1e-3, batch_scale=1 / 16)
    with DeviceTables(w.tables, value_mode=1) as dt:
        b = gi.make_batch(w, 0)
        sums = np.array([gi.POOL_SUM] * w.n_slots, np.int32)
        for policy in (0, 1, 2):
            dt.m.mfet_set_option(dt.h, dt.m.OPT_GROUP_POLICY, policy)
            got = forward(dt, w.batch, w.n_features, w.slot_feature, w.table_ids, sums, b.ids, b.offsets, None)
            ref = orc.embedding_bag(dt.oracle_tables, w.batch, w.n_features, w.slot_feature, w.table_ids, sums,
                                    b.ids, b.offsets, None)
            assert np.array_equal(got, ref)


# --------------------------------------------------------------- workloads --

SCALED = {1: (1.0, 1.0), 2: (0.01, 0.25), 3: (0.004, 0.125), 4: (0.005, 1 / 32), 5: (0.002, 0.125)}


@pytest.mark.parametrize("config", [1, 2, 3, 4])
def test_workload_parity_scaled(config):
    rs, bs = SCALED[config]
    w = gi.make_workload(config, rows_scale=rs, batch_scale=bs)
    with DeviceTables(w.tables) as dt:
        for j in (0, 1):
            b = gi.make_batch(w, j)
            got = workload_forward(dt, w, b)
            ref = workload_oracle(dt, w, b)
            assert_close(got, ref, "config %d batch %d" % (config, j))
        # bit-identical on a second run (fixed summation order)
        again = workload_forward(dt, w, b)
        assert np.array_equal(got, again)


def test_facets_concat_equals_single_slot_calls():
    w = gi.make_workload(3, rows_scale=0.002, batch_scale=1 / 16)
    with DeviceTables(w.tables) as dt:
        b = gi.make_batch(w, 0)
        full = workload_forward(dt, w, b)
        col = 0
        for s in range(w.n_slots):
            D = w.tables[int(w.table_ids[s])].dim
            one = forward(dt, w.batch, w.n_features, [int(w.slot_feature[s])], [int(w.table_ids[s])],
                          [int(w.pooling[s])], b.ids, b.offsets, b.weights)
            assert np.array_equal(full[:, col:col + D], one)
            col += D
        assert col == 896


def test_output_leading_dimension_and_unaligned_out():
    w = gi.make_workload(3, rows_scale=0.001, batch_scale=1 / 64)
    with DeviceTables(w.tables) as dt:
        b = gi.make_batch(w, 0)
        ref = workload_oracle(dt, w, b)
        wide = workload_forward(dt, w, b, out_ld=900)
        assert_close(wide[:, :896], ref)
        assert np.isnan(wide[:, 896:]).all()  # columns beyond the slots are left alone
        odd = workload_forward(dt, w, b, out_ld=899)  # rows not 16-byte aligned: scalar stores
        assert_close(odd[:, :896], ref)
        # an output base that is only 4-byte aligned
        big = torch.full((w.batch * 896 + 1,), float("nan"), dtype=torch.float32, device="cuda")
        view = big[1:].view(w.batch, 896)
        got = workload_forward(dt, w, b, out=view)
        assert_close(got, ref)


def test_many_slots_need_several_launches():
    rng = np.random.default_rng(5)
    tabs = [(0.01 * rng.standard_normal((50, 8))).astype(np.float32) for _ in range(4)]
    mt = _Mat(tabs, [gi.F32, gi.F16, gi.BF16, gi.F32], seeds=[1, 2, 3, 4])
    try:
        B, F, L = 33, 3, 130
        off = _ragged(rng, F * B, "mixed")
        ids = rng.integers(0, 2**40, size=int(off[-1]), dtype=np.uint64)
        w = rng.random(ids.size).astype(np.float32)
        sf = np.sort(rng.integers(0, F, L)).astype(np.int32)
        ti = rng.integers(0, 4, L).astype(np.int32)
        po = rng.integers(0, 3, L).astype(np.int32)
        got = forward(mt, B, F, sf, ti, po, ids, off, w)
        ref = orc.embedding_bag(mt.oracle_tables, B, F, sf, ti, po, ids, off, w)
        assert_close(got, ref)
    finally:
        mt.close()


def test_forward_host_equals_forward():
    m = mfet()
    w = gi.make_workload(2, rows_scale=0.001, batch_scale=1 / 16)
    with DeviceTables(w.tables) as dt:
        b = gi.make_batch(w, 0)
        ref = workload_forward(dt, w, b)
        shape, keep = m.make_shape(w.batch, w.n_features, w.slot_feature)
        nnz = int(b.offsets[-1])
        nbytes = m.mfet_host_io_bytes(dt.h, shape, w.table_ids, nnz)
        io = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        ids_h = torch.from_numpy(b.ids.view(np.int64)).pin_memory()
        off_h = torch.from_numpy(b.offsets).pin_memory()
        out_h = torch.empty(w.batch, w.out_dim, dtype=torch.float32).pin_memory()
        m.mfet_embedding_bag_forward_host(dt.h, shape, ids_h, off_h, None, nnz, w.table_ids, w.pooling, out_h, io,
                                          nbytes, _stream())
        assert np.array_equal(out_h.numpy(), ref)


# ------------------------------------------------------------------ dedup ---

@pytest.mark.parametrize("n,hi", [(0, 10), (1, 10), (2, 2), (255, 10**9), (256, 10**9), (257, 50), (2047, 10**9),
                                  (2048, 3), (2049, 10**6), (4096, 1), (65537, 10**9), (300_000, 10**9),
                                  (300_000, 2**62), (100_000, 70_000), (8191, 2**33), (8192, 2**22), (8193, 2**11),
                                  (16 * 512 * 3 + 5, 2047), (1_040_384, 10**9), (1_040_385, 10**9), (1_300_000, 2**40),
                                  (524_289, 2**34 + 3)])
def test_dedup_bit_exact(n, hi):
    """Sizes around the sort's tile boundaries and up to 1.3 million IDs, keys of 1 to 62 bits; a
    third of the values repeat a few hot rows the way Zipf-distributed IDs do."""
    m = mfet()
    rng = np.random.default_rng(n + hi % 97)
    rows = rng.integers(0, hi, size=n, dtype=np.int64)
    if n > 16:
        hot = rng.integers(0, hi, size=5, dtype=np.int64)
        pick = rng.random(n) < 0.33
        rows[pick] = hot[rng.integers(0, 5, size=int(pick.sum()))]
    dummy = torch.zeros(16, dtype=torch.uint8, device="cuda")
    h = m.mfet_tables_create([m.TableDesc(dummy.data_ptr(), 8, 4, m.F32, m.LOC_DEVICE, 0, 0, 0)])
    try:
        cap = max(n, 1) + 100
        ws = torch.empty(m.mfet_workspace_bytes(h, cap), dtype=torch.uint8, device="cuda")
        m.mfet_set_workspace(h, ws, ws.numel(), cap)
        d_rows = torch.from_numpy(rows).cuda()
        uniq = torch.full((max(n, 1),), -7, dtype=torch.int64, device="cuda")
        inv = torch.full((max(n, 1),), -7, dtype=torch.int32, device="cuda")
        nu = torch.full((1,), -7, dtype=torch.int64, device="cuda")
        for max_row in (0, hi):
            m.mfet_dedup_rows(h, d_rows, n, uniq, inv, nu, max_row, _stream())
            torch.cuda.synchronize()
            wu, wi = orc.dedup(rows)
            k = int(nu.item())
            assert k == wu.size
            assert np.array_equal(uniq.cpu().numpy()[:k], wu)
            assert np.array_equal(inv.cpu().numpy()[:n], wi)
            assert np.array_equal(d_rows.cpu().numpy(), rows)  # input untouched
        assert m.mfet_query_status(h) == 0
    finally:
        m.mfet_tables_destroy(h)


def test_dedup_on_two_streams_next_to_a_busy_pooling_stream():
    """The sort's tiles wait for the counts of earlier tiles of the same launch. Two handles sort on two
    streams while a third stream keeps the GPU's multiprocessors busy with pooling launches, so that tiles are
    dispatched late and out of step: every result must still be exact and no wait may run out
    (MFET_DEV_STALLED)."""
    m = mfet()
    rng = np.random.default_rng(5)
    w = gi.make_workload(2, rows_scale=0.002, batch_scale=1.0)
    b = gi.make_batch(w, 0)
    streams = [torch.cuda.Stream() for _ in range(3)]
    dummy = torch.zeros(16, dtype=torch.uint8, device="cuda")
    hs = [m.mfet_tables_create([m.TableDesc(dummy.data_ptr(), 8, 4, m.F32, m.LOC_DEVICE, 0, 0, 0)]) for _ in range(2)]
    try:
        with DeviceTables(w.tables) as dt:
            d_ids = torch.from_numpy(b.ids.view(np.int64)).cuda()
            d_off = torch.from_numpy(b.offsets).cuda()
            d_w = None if b.weights is None else torch.from_numpy(b.weights).cuda()
            out = torch.empty(w.batch, w.out_dim, dtype=torch.float32, device="cuda")
            shape, keep = m.make_shape(w.batch, w.n_features, w.slot_feature)
            sizes = [(300_000, 10**9), (90_000, 5 * 10**7)]
            work = []
            for h, (n, hi) in zip(hs, sizes):
                ws = torch.empty(m.mfet_workspace_bytes(h, n), dtype=torch.uint8, device="cuda")
                m.mfet_set_workspace(h, ws, ws.numel(), n)
                rows = rng.integers(0, hi, size=n, dtype=np.int64)
                rows[rng.random(n) < 0.3] = rows[1]
                work.append((ws, rows, torch.from_numpy(rows).cuda(), torch.empty(n, dtype=torch.int64, device="cuda"),
                             torch.empty(n, dtype=torch.int32, device="cuda"), torch.zeros(1, dtype=torch.int64, device="cuda")))
            torch.cuda.synchronize()
            for it in range(150):
                for _ in range(2):
                    m.mfet_embedding_bag_forward(dt.h, shape, d_ids, d_off, d_w, w.table_ids, w.pooling, out,
                                                 streams[2].cuda_stream)
                for k, (h, (n, hi)) in enumerate(zip(hs, sizes)):
                    ws, rows, d_rows, uniq, inv, nu = work[k]
                    m.mfet_dedup_rows(h, d_rows, n, uniq, inv, nu, hi, streams[k].cuda_stream)
            torch.cuda.synchronize()
            for k, (h, (n, hi)) in enumerate(zip(hs, sizes)):
                ws, rows, d_rows, uniq, inv, nu = work[k]
                assert m.mfet_query_status(h) == 0
                wu, wi = orc.dedup(rows)
                kk = int(nu.item())
                assert kk == wu.size
                assert np.array_equal(uniq.cpu().numpy()[:kk], wu)
                assert np.array_equal(inv.cpu().numpy(), wi)
            assert m.mfet_query_status(dt.h) == 0
    finally:
        for h in hs:
            m.mfet_tables_destroy(h)


def test_workspace_capacity_limit():
    """The dedup hands counts from tile to tile in 30 bits: a workspace for 2^30 - 1 IDs or more is refused
    by name, before anything is launched."""
    m = mfet()
    dummy = torch.zeros(16, dtype=torch.uint8, device="cuda")
    h = m.mfet_tables_create([m.TableDesc(dummy.data_ptr(), 8, 4, m.F32, m.LOC_DEVICE, 0, 0, 0)])
    try:
        assert m.mfet_workspace_bytes(h, (1 << 30) - 2) > 0
        for bad in ((1 << 30) - 1, 1 << 30, 1 << 40):
            with pytest.raises(m.MfetError) as e:
                m.mfet_workspace_bytes(h, bad)
            assert e.value.status == m.ERR_INVALID_ARG
    finally:
        m.mfet_tables_destroy(h)


def test_dedup_calls_of_changing_size_queued_on_one_workspace():
    """Calls of very different sizes and key widths, queued back to back on one stream and one workspace
    with no synchronisation in between: every call's kernels must find the tile counters, the digit
    totals and the ping-pong buffers as the call before left them, wherever that call's tiles ended."""
    m = mfet()
    rng = np.random.default_rng(77)
    dummy = torch.zeros(16, dtype=torch.uint8, device="cuda")
    h = m.mfet_tables_create([m.TableDesc(dummy.data_ptr(), 8, 4, m.F32, m.LOC_DEVICE, 0, 0, 0)])
    try:
        cap = 700_000
        ws = torch.empty(m.mfet_workspace_bytes(h, cap), dtype=torch.uint8, device="cuda")
        m.mfet_set_workspace(h, ws, ws.numel(), cap)
        calls = [(600_000, 10**9), (3, 5), (70_000, 2**40), (2048 * 16, 300), (2048 * 16 + 1, 10**6), (1, 1),
                 (2048 * 17, 2**20), (650_000, 2**62), (4097, 256), (600_000, 10**9)]
        held = []
        for n, hi in calls:
            rows = rng.integers(0, hi, size=n, dtype=np.int64)
            if n > 100:
                rows[rng.random(n) < 0.4] = rows[0]          # one very hot row
            d_rows = torch.from_numpy(rows).cuda()
            uniq = torch.full((n,), -7, dtype=torch.int64, device="cuda")
            inv = torch.full((n,), -7, dtype=torch.int32, device="cuda")
            nu = torch.full((1,), -7, dtype=torch.int64, device="cuda")
            held.append((rows, d_rows, uniq, inv, nu))
        for _ in range(2):
            for (n, hi), (rows, d_rows, uniq, inv, nu) in zip(calls, held):
                m.mfet_dedup_rows(h, d_rows, n, uniq, inv, nu, hi, _stream())
        torch.cuda.synchronize()
        assert m.mfet_query_status(h) == 0
        for (n, hi), (rows, d_rows, uniq, inv, nu) in zip(calls, held):
            wu, wi = orc.dedup(rows)
            k = int(nu.item())
            assert k == wu.size, (n, hi)
            assert np.array_equal(uniq.cpu().numpy()[:k], wu), (n, hi)
            assert np.array_equal(inv.cpu().numpy(), wi), (n, hi)
    finally:
        m.mfet_tables_destroy(h)


# -------------------------------------------------------------- host path ---

def _hot_rows(dt, w, table_id, feature, count, rows_total):
    """Hashed rows of the `count` hottest IDs of a feature (hashing done by the library), first
    distinct rows in popularity order, returned sorted."""
    m = dt.m
    ids = gi.hot_ids(w, feature, count)
    d = torch.from_numpy(ids.view(np.int64)).cuda()
    r = torch.empty_like(d)
    m.mfet_hash_ids(dt.h, table_id, d, d.numel(), r, _stream())
    rows = r.cpu().numpy()
    _, first = np.unique(rows, return_index=True)
    keep = rows[np.sort(first)]
    return np.sort(keep)


@pytest.mark.parametrize("pinned_by_caller", [True, False])
def test_host_table_path_matches_oracle_and_hbm_placement(pinned_by_caller):
    w = gi.make_workload(5, rows_scale=0.002, batch_scale=0.125)  # host table: 2M rows x 64 fp16 = 256 MB
    b = gi.make_batch(w, 0)
    n_host = int(b.offsets[w.batch] - b.offsets[0])
    with DeviceTables(w.tables, host_pinned=pinned_by_caller) as dt:
        dt.set_workspace(int(n_host * 1.25) + 1024)
        ref = workload_oracle(dt, w, b)
        cold = workload_forward(dt, w, b)           # no cache: every distinct row crosses PCIe
        assert_close(cold, ref, "host path, no cache")
        hot = _hot_rows(dt, w, 0, 0, int(w.tables[0].rows * w.cache_fraction), w.tables[0].rows)
        dt.build_cache(0, hot)
        warm = workload_forward(dt, w, b)           # cache on
        assert np.array_equal(warm, cold)
        b1 = gi.make_batch(w, 1)
        assert_close(workload_forward(dt, w, b1), workload_oracle(dt, w, b1), "host path, cache on")
        dt.build_cache(0, np.arange(0, w.tables[0].rows, dtype=np.int64))  # everything cached
        assert np.array_equal(workload_forward(dt, w, b), cold)
        dt.m.mfet_set_option(dt.h, dt.m.OPT_STAGE_IDS, 96)  # many staging passes per tile, bags cut between them
        assert_close(workload_forward(dt, w, b), ref, "host path, small staging buffer")
        dt.m.mfet_set_option(dt.h, dt.m.OPT_STAGE_IDS, 0)
        launches = dt.m.mfet_launch_count(dt.h)
        assert launches > 0
    # the same table placed in HBM gives the same bits
    specs = [gi.TableSpec(t.rows, t.dim, t.dtype, t.hash_seed, t.value_key, gi.LOC_DEVICE) for t in w.tables]
    with DeviceTables(specs) as dt2:
        hbm = workload_forward(dt2, w, b)
    assert_close(hbm, ref)
    assert np.array_equal(hbm[:, 64:], cold[:, 64:])
    assert_close(hbm[:, :64], cold[:, :64])


def test_host_table_feature_without_a_single_id():
    """A batch in which the host-table feature has only empty bags: the sort runs over zero keys (the count
    is read on the device), the slot's columns are zeros, nothing is fetched, no error bit is set, and the
    batch after it finds the workspace's counters as a normal batch leaves them."""
    w = gi.make_workload(5, rows_scale=0.001, batch_scale=0.0625)
    b = gi.make_batch(w, 0)
    B = w.batch
    cut = int(b.offsets[B])                                   # the IDs of feature 0 (the host table's)
    off = b.offsets.copy()
    off[:B + 1] = 0
    off[B + 1:] -= cut
    hollow = gi.Batch(b.ids[cut:].copy(), off, None if b.weights is None else b.weights[cut:].copy())
    with DeviceTables(w.tables) as dt:
        dt.set_workspace(cut + 1024)
        full_before = workload_forward(dt, w, b)
        got = workload_forward(dt, w, hollow)
        assert dt.m.mfet_query_status(dt.h) == 0
        assert dt.m.mfet_host_path_counts(dt.h) == (0, 0)
        assert not got[:, :w.tables[0].dim].any()
        assert_close(got, workload_oracle(dt, w, hollow), "host-table feature with no IDs")
        assert np.array_equal(workload_forward(dt, w, b), full_before)
        assert dt.m.mfet_query_status(dt.h) == 0


@pytest.mark.parametrize("cache_share", [0.0, 0.02, 1.0])
def test_cache_probe_and_miss_list_against_a_host_computation(cache_share):
    """The host-table slot's intermediate results, read back: distinct rows = numpy's sorted unique
    of the hashed rows; a distinct row has a cache slot exactly when it is in the cache list, and
    that slot holds it; the miss list is the ascending complement; the fetched rows and the cached
    rows are the table's rows, bit for bit."""
    w = gi.make_workload(5, rows_scale=0.001, batch_scale=0.25)
    b = gi.make_batch(w, 3)
    n_host = int(b.offsets[w.batch] - b.offsets[0])
    with DeviceTables(w.tables) as dt:
        m = dt.m
        cap = n_host + 64
        dt.set_workspace(cap)
        rows_total = w.tables[0].rows
        cached = np.zeros(0, np.int64)
        if cache_share >= 1.0:
            cached = np.arange(rows_total, dtype=np.int64)
        elif cache_share > 0:
            cached = _hot_rows(dt, w, 0, 0, int(rows_total * cache_share), rows_total)
        if cached.size:
            dt.build_cache(0, cached)
        got = workload_forward(dt, w, b)
        assert_close(got, workload_oracle(dt, w, b))
        n_unique, n_miss = m.mfet_host_path_counts(dt.h)
        uniq = torch.full((cap,), -1, dtype=torch.int64, device="cuda")
        src = torch.full((cap,), 0x7FFFFFFF, dtype=torch.int32, device="cuda")
        miss = torch.full((cap,), -1, dtype=torch.int64, device="cuda")
        m.mfet_host_path_result(dt.h, uniq, src, miss, cap)
        want_rows = orc.hash_ids(b.ids[:n_host], w.tables[0].hash_seed, rows_total)
        want_uniq = np.unique(want_rows)
        assert n_unique == want_uniq.size
        uniq, src, miss = uniq.cpu().numpy(), src.cpu().numpy(), miss.cpu().numpy()
        assert np.array_equal(uniq[:n_unique], want_uniq)
        assert (uniq[n_unique:] == -1).all() and (src[n_unique:] == 0x7FFFFFFF).all()
        in_cache = np.isin(want_uniq, cached)
        assert np.array_equal(src[:n_unique] >= 0, in_cache)
        assert np.array_equal(cached[src[:n_unique][in_cache]], want_uniq[in_cache])
        want_miss = want_uniq[~in_cache]
        assert n_miss == want_miss.size
        assert np.array_equal(miss[:n_miss], want_miss) and (miss[n_miss:] == -1).all()
        assert np.array_equal(-1 - src[:n_unique][~in_cache], np.arange(n_miss))
        # the fetch of listed rows, by itself: the rows of the host table, bit for bit
        if n_miss:
            rb = m.row_bytes(w.tables[0].dim, w.tables[0].dtype)
            dst = torch.zeros(n_miss * rb + 16, dtype=torch.uint8, device="cuda")
            m.mfet_host_fetch_rows(dt.h, 0, torch.from_numpy(want_miss).cuda(), n_miss, dst, _stream())
            torch.cuda.synchronize()
            host = dt.mem[0].numpy().reshape(rows_total, rb)
            assert np.array_equal(dst.cpu().numpy()[:n_miss * rb].reshape(n_miss, rb), host[want_miss])
            assert not dst.cpu().numpy()[n_miss * rb:].any()
        with pytest.raises(m.MfetError):
            m.mfet_host_path_result(dt.h, None, None, None, max(0, n_unique - 1))
        with pytest.raises(m.MfetError):
            m.mfet_host_fetch_rows(dt.h, 1, miss, 1, miss)  # table 1 is not a host table


def test_bad_prehashed_row_on_the_host_table_path_counts_as_the_last_row():
    """A caller-given row index beyond the table, on a slot whose table is in host memory: the error
    bit is set and the lookup reads the table's last row (documented; a device-memory table skips it)."""
    rows, dim = 64, 8
    spec = gi.TableSpec(rows, dim, gi.F16, 0, 0x77, gi.LOC_HOST)
    with DeviceTables([spec]) as dt:
        m = dt.m
        dt.set_workspace(64)
        ids = np.array([3, 999, 5, 63], np.uint64)
        off = np.array([0, 3, 4], np.int64)
        shape, keep = m.make_shape(2, 1, [0], ids_are_rows=True)
        out = torch.full((2, dim), float("nan"), dtype=torch.float32, device="cuda")
        m.mfet_embedding_bag_forward(dt.h, shape, torch.from_numpy(ids.view(np.int64)).cuda(),
                                     torch.from_numpy(off).cuda(), None, [0], [0], out, _stream())
        torch.cuda.synchronize()
        assert m.mfet_query_status(dt.h, clear=True) == m.DEV_ROW_RANGE
        ok_ids = np.array([3, 63, 5, 63], np.uint64)
        ref = orc.embedding_bag(dt.oracle_tables, 2, 1, [0], [0], [0], ok_ids, off, None, ids_are_rows=True)
        assert_close(out.cpu().numpy(), ref)


@pytest.mark.parametrize("dtype,dim", [(gi.BF16, 64), (gi.F32, 8)])
def test_tables_of_more_than_2_to_32_rows(dtype, dim):
    """Row indices that need more than 32 bits: a table declared with 2^32 + 1000 rows whose data
    pointer is placed so that rows 2^32 - 500 ... 2^32 + 999 fall into a small buffer; the batch
    gives row indices directly. SUM and WSUM (the staging then also holds weights and the upper
    index halves) against the oracle."""
    m = mfet()
    rows = 2**32 + 1000
    r0, n_real = 2**32 - 500, 1500
    key = 0xC0FFEE
    rb = m.row_bytes(dim, dtype)
    buf = torch.zeros(n_real * rb, dtype=torch.uint8, device="cuda")
    base = buf.data_ptr() - r0 * rb
    m.mfet_table_fill(base, r0, n_real, dim, dtype, 0, key, m.VAL_NORMAL, _stream())
    h = m.mfet_tables_create([m.TableDesc(base, rows, dim, dtype, m.LOC_DEVICE, 0, 0, 0)])
    try:
        rng = np.random.default_rng(dim)
        B = 200
        lens = rng.integers(0, 30, size=B)
        lens[7] = 150  # a whole-warp bag
        off = np.zeros(B + 1, np.int64)
        np.cumsum(lens, out=off[1:])
        ids = (r0 + rng.integers(0, n_real, size=int(off[-1]))).astype(np.uint64)
        wts = rng.random(ids.size).astype(np.float32)
        otab = [orc.Table(rows=rows, dim=dim, dtype=dtype, hash_seed=0, value_key=key)]
        shape, keep = m.make_shape(B, 1, [0], ids_are_rows=True)
        d_ids, d_off, d_w = torch.from_numpy(ids.view(np.int64)).cuda(), torch.from_numpy(off).cuda(), torch.from_numpy(wts).cuda()
        for pool in (0, 2):
            out = torch.full((B, dim), float("nan"), dtype=torch.float32, device="cuda")
            m.mfet_embedding_bag_forward(h, shape, d_ids, d_off, d_w, [0], [pool], out, _stream())
            torch.cuda.synchronize()
            assert m.mfet_query_status(h) == 0
            ref = orc.embedding_bag(otab, B, 1, [0], [0], [pool], ids, off, wts, ids_are_rows=True)
            assert_close(out.cpu().numpy(), ref, "pool %d" % pool)
        bad = ids.copy()
        bad[5] = rows + 3  # beyond the table: skipped, error bit
        m.mfet_embedding_bag_forward(h, shape, torch.from_numpy(bad.view(np.int64)).cuda(), d_off, d_w, [0], [0], out, _stream())
        torch.cuda.synchronize()
        assert m.mfet_query_status(h, clear=True) == m.DEV_ROW_RANGE
    finally:
        m.mfet_tables_destroy(h)


def test_host_slot_over_workspace_capacity_sets_error_bit():
    w = gi.make_workload(5, rows_scale=0.0005, batch_scale=1 / 64)
    b = gi.make_batch(w, 0)
    with DeviceTables(w.tables) as dt:
        dt.set_workspace(16)  # far too small for the host feature
        m = dt.m
        out = torch.full((w.batch, w.out_dim), float("nan"), dtype=torch.float32, device="cuda")
        shape, keep = m.make_shape(w.batch, w.n_features, w.slot_feature)
        m.mfet_embedding_bag_forward(dt.h, shape, torch.from_numpy(b.ids.view(np.int64)).cuda(),
                                     torch.from_numpy(b.offsets).cuda(), None, w.table_ids, w.pooling, out, _stream())
        torch.cuda.synchronize()
        assert m.mfet_query_status(dt.h, clear=True) & m.DEV_CAPACITY
        assert m.mfet_query_status(dt.h) == 0
        got = out.cpu().numpy()
        assert not got[:, :64].any()  # the over-capacity slot is written as zeros
        assert_close(got[:, 64:], workload_oracle(dt, w, b)[:, 64:])


# ----------------------------------------------------------- host-side errors

def test_argument_errors_are_reported_before_any_launch():
    m = mfet()
    dummy = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    good = m.TableDesc(dummy.data_ptr(), 8, 4, m.F32, m.LOC_DEVICE, 0, 0, 0)

    def status(fn, *a, **k):
        try:
            fn(*a, **k)
        except m.MfetError as e:
            return e.status
        return 0

    assert status(m.mfet_tables_create, [m.TableDesc(dummy.data_ptr(), 0, 4, m.F32, 0, 0, 0, 0)]) == m.ERR_INVALID_ARG
    assert status(m.mfet_tables_create, [m.TableDesc(None, 8, 4, m.F32, 0, 0, 0, 0)]) == m.ERR_INVALID_ARG
    assert status(m.mfet_tables_create, [m.TableDesc(dummy.data_ptr(), 8, 3, m.F32, 0, 0, 0, 0)]) == m.ERR_UNSUPPORTED_DIM
    assert status(m.mfet_tables_create, [m.TableDesc(dummy.data_ptr() + 4, 8, 4, m.F32, 0, 0, 0, 0)]) == m.ERR_ALIGNMENT
    assert status(m.mfet_tables_create, [m.TableDesc(dummy.data_ptr(), 8, 4, m.F32, 0, 0, 0, 24)]) == m.ERR_ALIGNMENT
    assert status(m.mfet_tables_create, [m.TableDesc(dummy.data_ptr(), 8, 4, 9, 0, 0, 0, 0)]) == m.ERR_INVALID_ARG
    assert status(m.mfet_tables_create, [good], 9999) == m.ERR_INVALID_ARG
    host = m.TableDesc(None, 64, 8, m.F16, m.LOC_HOST, 0, 0, 0)
    h = m.mfet_tables_create([good, host])
    try:
        launches = m.mfet_launch_count(h)
        ids = torch.zeros(4, dtype=torch.int64, device="cuda")
        off = torch.tensor([0, 2, 4], dtype=torch.int64, device="cuda")
        out = torch.zeros(2, 4, device="cuda")
        sh, k = m.make_shape(2, 1, [0])
        assert status(m.mfet_embedding_bag_forward, h, sh, ids, off, None, [5], [0], out) == m.ERR_INVALID_ARG
        assert status(m.mfet_embedding_bag_forward, h, sh, ids, off, None, [0], [3], out) == m.ERR_INVALID_ARG
        assert status(m.mfet_embedding_bag_forward, h, sh, ids, off, None, [0], [m.POOL_WSUM], out) == m.ERR_INVALID_ARG
        assert status(m.mfet_embedding_bag_forward, h, sh, None, off, None, [0], [0], out) == m.ERR_INVALID_ARG
        assert status(m.mfet_embedding_bag_forward, h, sh, ids, off, None, [1], [0], out) == m.ERR_NOT_REGISTERED
        sh2, k2 = m.make_shape(2, 1, [0], out_ld=2)
        assert status(m.mfet_embedding_bag_forward, h, sh2, ids, off, None, [0], [0], out) == m.ERR_INVALID_ARG
        sh3, k3 = m.make_shape(2, 1, [1])
        assert status(m.mfet_embedding_bag_forward, h, sh3, ids, off, None, [0], [0], out) == m.ERR_INVALID_ARG
        assert status(m.mfet_hash_ids, h, 7, ids, 4, ids) == m.ERR_INVALID_ARG
        assert status(m.mfet_host_tables_register, h, 0, dummy.data_ptr(), 4096) == m.ERR_INVALID_ARG
        pinned = torch.zeros(64 * 16, dtype=torch.uint8).pin_memory()
        assert status(m.mfet_host_tables_register, h, 1, pinned.data_ptr(), 100, 1) == m.ERR_INVALID_ARG
        assert status(m.mfet_host_tables_register, h, 1, pinned.data_ptr() + 8, 1016, 1) == m.ERR_ALIGNMENT
        assert status(m.mfet_cache_build, h, 1, np.array([1, 2], np.int64), dummy, 4096) == m.ERR_NOT_REGISTERED
        m.mfet_host_tables_register(h, 1, pinned.data_ptr(), pinned.numel(), 1)
        assert status(m.mfet_host_tables_register, h, 1, pinned.data_ptr(), pinned.numel(), 1) == m.ERR_INVALID_ARG
        assert status(m.mfet_embedding_bag_forward, h, sh, ids, off, None, [1], [0],
                      torch.zeros(2, 8, device="cuda")) == m.ERR_WORKSPACE
        assert status(m.mfet_cache_build, h, 1, np.array([2, 1], np.int64), dummy, 4096) == m.ERR_INVALID_ARG
        assert status(m.mfet_cache_build, h, 1, np.array([1, 64], np.int64), dummy, 4096) == m.ERR_INVALID_ARG
        assert status(m.mfet_cache_build, h, 1, np.array([1, 2], np.int64), dummy, 16) == m.ERR_WORKSPACE
        assert status(m.mfet_set_workspace, h, dummy.data_ptr() + 16, 4000, 4) == m.ERR_ALIGNMENT
        assert status(m.mfet_set_workspace, h, dummy, 256, 1000) == m.ERR_WORKSPACE
        assert status(m.mfet_dedup_rows, h, ids, 4, ids, ids, ids, 0) == m.ERR_WORKSPACE
        assert status(m.mfet_set_option, h, 99, 0) == m.ERR_INVALID_ARG
        assert m.mfet_launch_count(h) == launches  # nothing was launched by any rejected call
        assert m.mfet_query_status(h) == 0
    finally:
        m.mfet_tables_destroy(h)
    assert "workspace" in m.status_string(m.ERR_WORKSPACE)


def test_device_error_bits_for_bad_prehashed_rows_and_offsets():
    rng = np.random.default_rng(1)
    tab = rng.standard_normal((16, 8)).astype(np.float32)
    mt = _Mat([tab], [gi.F32])
    try:
        m = mt.m
        ids = torch.tensor([1, 99, 2], dtype=torch.int64, device="cuda")  # 99 >= rows
        off = torch.tensor([0, 3], dtype=torch.int64, device="cuda")
        out = torch.empty(1, 8, device="cuda")
        sh, k = m.make_shape(1, 1, [0], ids_are_rows=True)
        m.mfet_embedding_bag_forward(mt.h, sh, ids, off, None, [0], [0], out)
        torch.cuda.synchronize()
        assert m.mfet_query_status(mt.h, clear=True) == m.DEV_ROW_RANGE
        assert_close(out.cpu().numpy()[0], tab[1] + tab[2])  # the bad index is skipped
        off_bad = torch.tensor([0, 3, 1], dtype=torch.int64, device="cuda")
        out2 = torch.empty(2, 8, device="cuda")
        sh2, k2 = m.make_shape(2, 1, [0], ids_are_rows=True)
        ids2 = torch.tensor([1, 3, 2], dtype=torch.int64, device="cuda")
        m.mfet_embedding_bag_forward(mt.h, sh2, ids2, off_bad, None, [0], [0], out2)
        torch.cuda.synchronize()
        assert m.mfet_query_status(mt.h, clear=True) == m.DEV_OFFSETS
        assert not out2.cpu().numpy()[1].any()
    finally:
        mt.close()


# ------------------------------------------------------------------- INT4 ---

@pytest.mark.parametrize("dim", [8, 24, 32, 64, 128, 264])
@pytest.mark.parametrize("mode", [0, 1])
def test_int4_table_fill_bit_exact(dim, mode):
    """Paper, Section 4.1.2 (INT4 post-training quantisation; the row format is this library's)."""
    m = mfet()
    rows, key = 1237, 0x0F1E2D3C4B5A6978
    rb = m.row_bytes(dim, m.INT4)
    assert rb % 16 == 0 and rb >= dim // 2 + 4
    buf = torch.full((rows * rb,), 0xAB, dtype=torch.uint8, device="cuda")
    m.mfet_table_fill(buf, 0, rows, dim, m.INT4, 0, key, mode, _stream())
    got = buf.cpu().numpy().reshape(rows, rb)
    want = orc.table_fill(orc.Table(rows=rows, dim=dim, dtype=orc.INT4, value_key=key, value_mode=mode))
    assert np.array_equal(got, want)


@pytest.mark.parametrize("dim", [8, 24, 32, 64, 128, 264])
@pytest.mark.parametrize("policy", [0, 1, 2])
def test_int4_pooling_parity(dim, policy):
    specs = [gi.TableSpec(5003, dim, gi.INT4, 0x1234567, 0xABCDEF0123), gi.TableSpec(977, dim, gi.INT4, 99, 777)]
    rng = np.random.default_rng(dim + policy)
    with DeviceTables(specs) as dt:
        dt.m.mfet_set_option(dt.h, dt.m.OPT_GROUP_POLICY, policy)
        B, F = 61, 2
        off = _ragged(rng, F * B, "mixed")
        ids = rng.integers(0, 2**40, size=int(off[-1]), dtype=np.uint64)
        w = rng.random(ids.size).astype(np.float32)
        sf, ti, po = [0, 0, 1, 1], [0, 1, 1, 0], [0, 2, 1, 2]
        got = forward(dt, B, F, sf, ti, po, ids, off, w)
        ref = orc.embedding_bag(dt.oracle_tables, B, F, sf, ti, po, ids, off, w)
        assert_close(got, ref, "int4 dim %d" % dim)
        # single-ID bags return the decoded row itself, bit for bit
        one = forward(dt, 8, 1, [0], [0], [0], np.arange(8, dtype=np.uint64), np.arange(9, dtype=np.int64), None,
                      ids_are_rows=True)
        want = np.stack([orc.decode_row(dt.oracle_tables[0], r) for r in range(8)])
        assert np.array_equal(one, want)


def test_int4_host_table_behind_the_cache():
    """The quantised table in host memory (the paper's serving set-up: INT4 tables on the CPU side)."""
    w = gi.make_workload(5, rows_scale=0.001, batch_scale=0.125)
    w.tables[0].dtype = gi.INT4
    b = gi.make_batch(w, 0)
    n_host = int(b.offsets[w.batch] - b.offsets[0])
    with DeviceTables(w.tables) as dt:
        dt.set_workspace(n_host + 1024)
        ref = workload_oracle(dt, w, b)
        cold = workload_forward(dt, w, b)
        assert_close(cold, ref, "int4 host table, no cache")
        dt.build_cache(0, _hot_rows(dt, w, 0, 0, int(w.tables[0].rows * 0.05), w.tables[0].rows))
        assert np.array_equal(workload_forward(dt, w, b), cold)


# ------------------------------------------------- early fetch, version tag --

def test_prefetched_batches_give_the_same_bits_as_the_serial_path():
    """Paper, Section 3.4: the embedding fetch starts early and overlaps other work; the result
    must not depend on it."""
    m = mfet()
    w = gi.make_workload(5, rows_scale=0.001, batch_scale=0.125)
    bs = [gi.make_batch(w, j) for j in range(3)]
    cap = max(int(b.offsets[w.batch] - b.offsets[0]) for b in bs) + 1024
    with DeviceTables(w.tables) as dt:
        dt.set_workspace(cap)
        dt.build_cache(0, _hot_rows(dt, w, 0, 0, int(w.tables[0].rows * 0.02), w.tables[0].rows))
        serial = [workload_forward(dt, w, b) for b in bs]
        d_ids = [torch.from_numpy(b.ids.view(np.int64)).cuda() for b in bs]
        d_off = [torch.from_numpy(b.offsets).cuda() for b in bs]
        outs = [torch.full((w.batch, w.out_dim), float("nan"), device="cuda") for _ in bs]
        plain, keep = m.make_shape(w.batch, w.n_features, w.slot_feature)
        pre, keep2 = m.make_shape(w.batch, w.n_features, w.slot_feature)
        pre.flags |= m.BATCH_PREFETCHED
        s = _stream()

        def status(fn, *a):
            try:
                fn(*a)
            except m.MfetError as e:
                return e.status
            return 0

        # a flagged forward without a prefetch is refused
        assert status(m.mfet_embedding_bag_forward, dt.h, pre, d_ids[0], d_off[0], None, w.table_ids, w.pooling,
                      outs[0], s) == m.ERR_INVALID_ARG
        m.mfet_host_prefetch(dt.h, plain, d_ids[0], d_off[0], w.table_ids, s)
        m.mfet_host_prefetch(dt.h, plain, d_ids[1], d_off[1], w.table_ids, s)
        # both result sets are taken; and an unflagged forward may not cut in
        assert status(m.mfet_host_prefetch, dt.h, plain, d_ids[2], d_off[2], w.table_ids, s) == m.ERR_INVALID_ARG
        assert status(m.mfet_embedding_bag_forward, dt.h, plain, d_ids[0], d_off[0], None, w.table_ids, w.pooling,
                      outs[0], s) == m.ERR_INVALID_ARG
        m.mfet_embedding_bag_forward(dt.h, pre, d_ids[0], d_off[0], None, w.table_ids, w.pooling, outs[0], s)
        m.mfet_host_prefetch(dt.h, plain, d_ids[2], d_off[2], w.table_ids, s)
        m.mfet_embedding_bag_forward(dt.h, pre, d_ids[1], d_off[1], None, w.table_ids, w.pooling, outs[1], s)
        m.mfet_embedding_bag_forward(dt.h, pre, d_ids[2], d_off[2], None, w.table_ids, w.pooling, outs[2], s)
        torch.cuda.synchronize()
        assert m.mfet_query_status(dt.h) == 0
        for j in range(3):
            assert np.array_equal(outs[j].cpu().numpy(), serial[j]), j
        # afterwards the serial path works again
        assert np.array_equal(workload_forward(dt, w, bs[0]), serial[0])
    # a batch without exactly one host-table slot cannot be prefetched
    w2 = gi.make_workload(2, rows_scale=0.001, batch_scale=1 / 16)
    with DeviceTables(w2.tables) as dt2:
        b = gi.make_batch(w2, 0)
        sh, k = m.make_shape(w2.batch, w2.n_features, w2.slot_feature)
        try:
            m.mfet_host_prefetch(dt2.h, sh, torch.from_numpy(b.ids.view(np.int64)).cuda(),
                                 torch.from_numpy(b.offsets).cuda(), w2.table_ids)
            raise AssertionError("expected INVALID_ARG")
        except m.MfetError as e:
            assert e.status == m.ERR_INVALID_ARG


def test_early_fetch_pipeline_in_steady_state():
    """Every step announces its successor (prefetch of batch j+1, then the pooling of batch j), for many
    steps over rotating batches and without a synchronisation in between: the dedup of one batch runs
    while the rows of another are fetched and a third is pooled, and every result has the serial path's bits."""
    m = mfet()
    w = gi.make_workload(5, rows_scale=0.001, batch_scale=0.125)
    bs = [gi.make_batch(w, j) for j in range(3)]
    cap = max(int(b.offsets[w.batch] - b.offsets[0]) for b in bs) + 1024
    with DeviceTables(w.tables) as dt:
        dt.set_workspace(cap)
        dt.build_cache(0, _hot_rows(dt, w, 0, 0, int(w.tables[0].rows * 0.02), w.tables[0].rows))
        serial = [workload_forward(dt, w, b) for b in bs]
        d_ids = [torch.from_numpy(b.ids.view(np.int64)).cuda() for b in bs]
        d_off = [torch.from_numpy(b.offsets).cuda() for b in bs]
        steps = 10
        outs = [torch.full((w.batch, w.out_dim), float("nan"), device="cuda") for _ in range(steps)]
        plain, keep = m.make_shape(w.batch, w.n_features, w.slot_feature)
        pre, keep2 = m.make_shape(w.batch, w.n_features, w.slot_feature)
        pre.flags |= m.BATCH_PREFETCHED
        s = _stream()
        m.mfet_host_prefetch(dt.h, plain, d_ids[0], d_off[0], w.table_ids, s)
        for j in range(steps):
            k, kn = j % 3, (j + 1) % 3
            if j + 1 < steps:
                m.mfet_host_prefetch(dt.h, plain, d_ids[kn], d_off[kn], w.table_ids, s)
            m.mfet_embedding_bag_forward(dt.h, pre, d_ids[k], d_off[k], None, w.table_ids, w.pooling, outs[j], s)
        torch.cuda.synchronize()
        assert m.mfet_query_status(dt.h) == 0
        for j in range(steps):
            assert np.array_equal(outs[j].cpu().numpy(), serial[j % 3]), j
        n_unique, n_miss = m.mfet_host_path_counts(dt.h)
        assert 0 < n_miss <= n_unique <= cap
        assert np.array_equal(workload_forward(dt, w, bs[1]), serial[1])  # and the serial path afterwards


def test_version_tag_is_echoed_unchanged():
    """Paper, Algorithm 2: embeddings are returned together with the version of the tables."""
    m = mfet()
    dummy = torch.zeros(64, dtype=torch.uint8, device="cuda")
    a = m.mfet_tables_create([m.TableDesc(dummy.data_ptr(), 4, 4, m.F32, m.LOC_DEVICE, 0, 0, 0)])
    b = m.mfet_tables_create([m.TableDesc(dummy.data_ptr(), 4, 4, m.F32, m.LOC_DEVICE, 0, 0, 0)])
    try:
        assert m.mfet_tables_version(a) == 0
        m.mfet_tables_set_version(a, 20250807)
        m.mfet_tables_set_version(b, 2**64 - 1)
        assert m.mfet_tables_version(a) == 20250807 and m.mfet_tables_version(b) == 2**64 - 1
    finally:
        m.mfet_tables_destroy(a)
        m.mfet_tables_destroy(b)
