"""Pins of the CPU oracle against things other than itself.

The paper prints no numerical example of the lookup path (Section 2.2 describes
hashed tables in words), so every pin here is a published test vector of the
public hash, a closed form, an invariant, a brute-force restatement with a
different structure, or a library routine on a special case.
"""
import os

import numpy as np
import pytest
import torch

import oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")
M64 = (1 << 64) - 1
GOLDEN_INC = 0x9E3779B97F4A7C15


def py_splitmix64(x):
    """Big-integer restatement used as an independent cross-check."""
    z = (x + GOLDEN_INC) & M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M64
    return z ^ (z >> 31)


# ------------------------------------------------------------------ hash ----

def test_splitmix64_published_vectors():
    n = 0
    with open(os.path.join(GOLD, "splitmix64_vectors.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            seed, k, val = line.split()
            got = orc.splitmix64((int(seed) + (int(k) - 1) * GOLDEN_INC) & M64)
            assert got == int(val, 0), line
            n += 1
    assert n == 8


def test_splitmix64_is_a_bijection_on_a_sample():
    xs = np.random.default_rng(1).integers(0, 2**63, size=20000, dtype=np.uint64)
    hs = {orc.splitmix64(int(x)) for x in np.unique(xs)}
    assert len(hs) == len(np.unique(xs))


def test_hash_mod_rows_against_big_integers():
    rng = np.random.default_rng(2)
    ids = rng.integers(0, 2**64 - 1, size=10000, dtype=np.uint64)
    ids[:4] = [0, 1, 2**40 - 1, 2**64 - 1]
    for rows in (1, 2, 7, 100_000, 10_000_000, 50_000_000, 10**9, 2**32 - 1, 2**32, 2**32 + 1,
                 2**40 + 12345, 2**62 + 3, 2**63 - 1):
        for seed in (0, 0x1234_5678_9ABC_DEF1):
            got = orc.hash_ids(ids, seed, rows)
            want = [py_splitmix64(int(i) ^ seed) % rows for i in ids]
            assert got.tolist() == want
            assert got.min() >= 0 and got.max() < rows


def test_hash_mod_special_cases():
    ids = np.arange(0, 5000, dtype=np.uint64)
    assert not orc.hash_ids(ids, 0, 1).any()
    for k in (1, 10, 33, 63):
        got = orc.hash_ids(ids, 0, 1 << k)
        want = [py_splitmix64(int(i)) & ((1 << k) - 1) for i in ids]
        assert got.tolist() == want


def test_collisions_fall_as_the_table_grows():
    # Section 2.2: collisions appear when distinct IDs outnumber rows; a larger vocabulary reduces them.
    ids = np.arange(1, 200001, dtype=np.uint64) * np.uint64(2654435761)
    last = None
    for rows in (10_000, 100_000, 1_000_000, 100_000_000):
        coll = ids.size - np.unique(orc.hash_ids(ids, 0, rows)).size
        # birthday estimate: n - rows*(1 - exp(-n/rows))
        est = ids.size - rows * (1 - np.exp(-ids.size / rows))
        assert abs(coll - est) <= 0.02 * ids.size + 50
        assert last is None or coll < last
        last = coll


# ---------------------------------------------------------- number formats --

def test_fp16_decode_exhaustive_vs_numpy():
    h = np.arange(65536, dtype=np.uint16)
    want = h.view(np.float16).astype(np.float32).view(np.uint32)
    got = np.array([orc.f16_bits_to_f32_bits(int(x)) for x in h], np.uint32)
    nan = np.isnan(h.view(np.float16))
    assert np.array_equal(got[~nan], want[~nan])
    assert np.isnan(got[nan].view(np.float32)).all()


def test_bf16_decode_exhaustive_vs_torch():
    h = np.arange(65536, dtype=np.uint16)
    t = torch.from_numpy(h.view(np.int16).copy()).view(torch.bfloat16).to(torch.float32)
    want = t.numpy().view(np.uint32)
    got = np.array([orc.bf16_bits_to_f32_bits(int(x)) for x in h], np.uint32)
    nan = np.isnan(want.view(np.float32))
    assert np.array_equal(got[~nan], want[~nan])


def _float_probe_bits():
    rng = np.random.default_rng(3)
    bits = rng.integers(0, 2**32, size=60000, dtype=np.uint64).astype(np.uint32)
    # values near fp16 range edges, ties, subnormals
    special = np.array([0.0, -0.0, 1.0, 65504.0, 65519.99, 65520.0, 1e-8, 5.96e-8, 2.98e-8, 2.9802322e-8,
                        6.1e-5, 6.097e-5, 1.0009765625, 1.00048828125, 1.000732421875, 0.01, -0.0123,
                        3.0e38, 1.0e-40], np.float32).view(np.uint32)
    grid = (np.float32(1.0) + np.arange(0, 4096, dtype=np.float32) * np.float32(2.0 ** -13)).view(np.uint32)
    return np.concatenate([bits, special, grid])


def test_f32_to_f16_rne_vs_numpy():
    bits = _float_probe_bits()
    f = bits.view(np.float32)
    ok = ~np.isnan(f)
    with np.errstate(over="ignore"):
        want = f.astype(np.float16).view(np.uint16)
    got = np.array([orc.f32_bits_to_f16_bits(int(b)) for b in bits], np.uint16)
    assert np.array_equal(got[ok], want[ok])


def test_f32_to_bf16_rne_vs_torch():
    bits = _float_probe_bits()
    f = torch.from_numpy(bits.view(np.float32).copy())
    want = f.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([orc.f32_bits_to_bf16_bits(int(b)) for b in bits], np.uint16)
    ok = ~np.isnan(bits.view(np.float32))
    assert np.array_equal(got[ok], want[ok])


# ------------------------------------------------------------ table values --

def test_table_values_frozen_literals():
    n = 0
    with open(os.path.join(GOLD, "table_values.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            key, mode, dim, dtype, r, d, bits = (int(x, 0) for x in line.split())
            assert orc.table_value_bits(key, mode, dim, dtype, r, d) == bits, line
            n += 1
    assert n >= 8


def test_table_value_definition_against_big_integers():
    # the generator's definition, restated with python integers and numpy rounding
    c = np.float32(0.01 / np.sqrt(4 * (65536.0 ** 2 - 1) / 12))
    rng = np.random.default_rng(4)
    for _ in range(300):
        key = int(rng.integers(0, 2**63)) * 2 + 1
        dim = int(rng.choice([4, 32, 64, 128]))
        r = int(rng.integers(0, 10**9))
        d = int(rng.integers(0, dim))
        u = py_splitmix64((key + r * dim + d) & M64)
        s = (u & 0xFFFF) + ((u >> 16) & 0xFFFF) + ((u >> 32) & 0xFFFF) + (u >> 48)
        v = np.float32(s - 131070) * c
        assert orc.table_value_f32(key, orc.VAL_NORMAL, dim, r, d) == float(v)
        g = np.float32(((u & 0xFF) - 128) * 2.0 ** -13)
        assert orc.table_value_f32(key, orc.VAL_GRID, dim, r, d) == float(g)
        assert orc.table_value_bits(key, orc.VAL_NORMAL, dim, orc.F16, r, d) == int(v.astype(np.float16).view(np.uint16))
        bf = torch.tensor([float(v)], dtype=torch.float32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)[0]
        assert orc.table_value_bits(key, orc.VAL_NORMAL, dim, orc.BF16, r, d) == int(bf)


def test_table_values_look_normal():
    t = orc.Table(rows=4096, dim=64, dtype=orc.F32, value_key=0xABCDEF12345)
    x = orc.table_fill(t).view(np.float32)
    assert abs(x.mean()) < 1e-4
    assert abs(x.std() - 0.01) < 1e-4
    assert np.abs(x).max() <= 0.0347  # Irwin-Hall of four uniforms ends at 3.46 sigma
    # each row is a different draw
    assert np.unique(x[:, 0]).size > 4000


def test_grid_values_are_exact_in_every_dtype():
    for dt in (orc.F32, orc.F16, orc.BF16):
        t = orc.Table(rows=512, dim=32, dtype=dt, value_key=77, value_mode=orc.VAL_GRID)
        vals = np.stack([orc.decode_row(t, r) for r in range(512)])
        k = vals * 2.0 ** 13
        assert np.array_equal(k, np.rint(k)) and k.min() >= -128 and k.max() <= 127
        ref = orc.Table(rows=512, dim=32, dtype=orc.F32, value_key=77, value_mode=orc.VAL_GRID)
        assert np.array_equal(vals, orc.table_fill(ref).view(np.float32))


def test_fill_matches_decode_and_materialised_equals_procedural():
    rng = np.random.default_rng(5)
    for dt in (orc.F32, orc.F16, orc.BF16):
        proc = orc.Table(rows=300, dim=16, dtype=dt, hash_seed=9, value_key=1234567)
        raw = orc.table_fill(proc)
        mat = orc.Table(rows=300, dim=16, dtype=dt, hash_seed=9, data=raw)
        for r in rng.integers(0, 300, 20):
            assert np.array_equal(orc.decode_row(proc, int(r)), orc.decode_row(mat, int(r)))


# ----------------------------------------------------------------- pooling --

def _read_tiny():
    d = {}
    with open(os.path.join(GOLD, "tiny_bags.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            k, *v = line.split()
            d[k] = np.array([float(x) for x in v])
    return d


@pytest.mark.parametrize("dtype", [orc.F32, orc.F16, orc.BF16])
def test_hand_computed_tiny_bags(dtype):
    g = _read_tiny()
    tab32 = g["table"].astype(np.float32).reshape(4, 2)
    if dtype == orc.F32:
        data = tab32
    elif dtype == orc.F16:
        data = tab32.astype(np.float16)
    else:
        data = torch.from_numpy(tab32).to(torch.bfloat16).view(torch.int16).numpy()
    t = orc.Table(rows=4, dim=2, dtype=dtype, data=np.ascontiguousarray(data))
    ids = g["ids"].astype(np.uint64)
    off = g["offsets"].astype(np.int64)
    w = g["weights"].astype(np.float32)
    for pool, key in ((orc.POOL_SUM, "sum"), (orc.POOL_MEAN, "mean"), (orc.POOL_WSUM, "wsum")):
        out = orc.embedding_bag([t], 3, 1, [0], [0], [pool], ids, off, w, ids_are_rows=True)
        assert np.array_equal(out, g[key].reshape(3, 2).astype(np.float32)), key


def _random_case(rng, rows, dims, B, F, max_len, dtypes=None, empty_frac=0.2):
    """Random materialised tables + ragged bags; one slot per (feature, facet)."""
    tables = []
    for i, D in enumerate(dims):
        dt = (dtypes[i] if dtypes else orc.F32)
        x = rng.standard_normal((rows, D)).astype(np.float32)
        if dt == orc.F16:
            data = x.astype(np.float16)
        elif dt == orc.BF16:
            data = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy()
        else:
            data = x
        tables.append(orc.Table(rows=rows, dim=D, dtype=dt, hash_seed=int(rng.integers(0, 2**63)),
                                data=np.ascontiguousarray(data)))
    lens = rng.integers(0, max_len + 1, size=F * B)
    lens[rng.random(F * B) < empty_frac] = 0
    off = np.zeros(F * B + 1, np.int64)
    np.cumsum(lens, out=off[1:])
    ids = rng.integers(0, 2**40, size=int(off[-1]), dtype=np.uint64)
    w = rng.random(int(off[-1])).astype(np.float32)
    return tables, ids, off, w


def _dense(t: orc.Table) -> np.ndarray:
    return np.stack([orc.decode_row(t, r) for r in range(t.rows)]).astype(np.float64)


def test_pooling_brute_force_count_matrix():
    """Second, differently structured implementation: scatter each bag into a dense
    count (or weight) matrix C[bag, row] and multiply by the table."""
    rng = np.random.default_rng(6)
    B, F = 37, 2
    tables, ids, off, w = _random_case(rng, rows=53, dims=[8, 4], B=B, F=F, max_len=9,
                                       dtypes=[orc.F16, orc.BF16])
    slot_feature, table_ids = [0, 1, 1], [0, 1, 0]
    for pool in (orc.POOL_SUM, orc.POOL_MEAN, orc.POOL_WSUM):
        out = orc.embedding_bag(tables, B, F, slot_feature, table_ids, [pool] * 3, ids, off, w)
        col = 0
        for s in range(3):
            t = tables[table_ids[s]]
            f = slot_feature[s]
            Cm = np.zeros((B, t.rows))
            for b in range(B):
                for i in range(off[f * B + b], off[f * B + b + 1]):
                    r = py_splitmix64(int(ids[i]) ^ t.hash_seed) % t.rows
                    Cm[b, r] += float(w[i]) if pool == orc.POOL_WSUM else 1.0
                n = off[f * B + b + 1] - off[f * B + b]
                if pool == orc.POOL_MEAN and n > 0:
                    Cm[b] /= n
            want = Cm @ _dense(t)
            np.testing.assert_allclose(out[:, col:col + t.dim], want, rtol=1e-6, atol=1e-7)
            col += t.dim


@pytest.mark.parametrize("pool,mode", [(orc.POOL_SUM, "sum"), (orc.POOL_MEAN, "mean"), (orc.POOL_WSUM, "sum")])
def test_pooling_vs_torch_embedding_bag(pool, mode):
    """Special case that reduces to a library routine: pre-hashed indices, one table."""
    rng = np.random.default_rng(7)
    B = 64
    tables, ids, off, w = _random_case(rng, rows=101, dims=[16], B=B, F=1, max_len=40)
    rows = rng.integers(0, 101, size=ids.size).astype(np.uint64)
    out = orc.embedding_bag(tables, B, 1, [0], [0], [pool], rows, off, w, ids_are_rows=True)
    weight = torch.from_numpy(_dense(tables[0]))
    psw = torch.from_numpy(w.astype(np.float64)) if pool == orc.POOL_WSUM else None
    want = torch.nn.functional.embedding_bag(torch.from_numpy(rows.astype(np.int64)), weight,
                                             torch.from_numpy(off[:-1]), mode=mode,
                                             per_sample_weights=psw, include_last_offset=False)
    np.testing.assert_allclose(out, want.numpy(), rtol=1e-6, atol=1e-7)


def test_pooling_invariants():
    rng = np.random.default_rng(8)
    B, F = 50, 3
    tables, ids, off, w = _random_case(rng, rows=200, dims=[8, 8, 8], B=B, F=F, max_len=12)
    sf, ti = [0, 1, 2], [0, 1, 2]
    s = orc.embedding_bag(tables, B, F, sf, ti, [orc.POOL_SUM] * 3, ids, off, w)
    m = orc.embedding_bag(tables, B, F, sf, ti, [orc.POOL_MEAN] * 3, ids, off, w)
    ws = orc.embedding_bag(tables, B, F, sf, ti, [orc.POOL_WSUM] * 3, ids, off, w)
    lens = np.diff(off).reshape(F, B)
    # empty bag -> exact zeros for all poolings
    for f in range(F):
        e = lens[f] == 0
        assert e.any()
        for o in (s, m, ws):
            assert not o[e, 8 * f:8 * f + 8].any()
        # mean * len == sum
        np.testing.assert_allclose(m[~e, 8 * f:8 * f + 8] * lens[f][~e, None], s[~e, 8 * f:8 * f + 8],
                                   rtol=1e-6, atol=1e-7)
    # WSUM with unit weights == SUM (bit-exact: same double accumulation)
    ones = np.ones_like(w)
    assert np.array_equal(orc.embedding_bag(tables, B, F, sf, ti, [orc.POOL_WSUM] * 3, ids, off, ones), s)
    # WSUM is linear in the weights
    w2 = rng.random(w.size).astype(np.float32)
    a = orc.embedding_bag(tables, B, F, sf, ti, [orc.POOL_WSUM] * 3, ids, off, w2)
    both = orc.embedding_bag(tables, B, F, sf, ti, [orc.POOL_WSUM] * 3, ids, off, (w.astype(np.float64) + w2).astype(np.float32))
    np.testing.assert_allclose(both, ws.astype(np.float64) + a, rtol=1e-5, atol=1e-6)
    # permuting IDs (with their weights) inside every bag changes nothing beyond rounding
    ids_p, w_p = ids.copy(), w.copy()
    for k in range(F * B):
        p = rng.permutation(off[k + 1] - off[k]) + off[k]
        ids_p[off[k]:off[k + 1]] = ids[p]
        w_p[off[k]:off[k + 1]] = w[p]
    np.testing.assert_allclose(orc.embedding_bag(tables, B, F, sf, ti, [orc.POOL_WSUM] * 3, ids_p, off, w_p),
                               ws, rtol=1e-6, atol=1e-7)
    # MEAN ignores weights
    assert np.array_equal(orc.embedding_bag(tables, B, F, sf, ti, [orc.POOL_MEAN] * 3, ids, off, None), m)


def test_duplicates_count_with_multiplicity():
    t = orc.Table(rows=8, dim=4, dtype=orc.F32, data=np.arange(32, dtype=np.float32).reshape(8, 4))
    out = orc.embedding_bag([t], 1, 1, [0], [0], [orc.POOL_SUM], np.array([5, 5, 5], np.uint64),
                            np.array([0, 3], np.int64), ids_are_rows=True)
    assert np.array_equal(out[0], 3 * np.arange(20, 24, dtype=np.float32))


def test_concat_of_facets_equals_single_slot_calls():
    """Section 4.1.1: every facet table of an ID feature contributes separately."""
    rng = np.random.default_rng(9)
    B, F = 40, 2
    tables, ids, off, w = _random_case(rng, rows=97, dims=[4, 8, 16, 8], B=B, F=F, max_len=7,
                                       dtypes=[orc.BF16, orc.F16, orc.F32, orc.BF16])
    sf, ti = [0, 0, 0, 1, 1], [0, 1, 2, 3, 1]
    pool = [orc.POOL_SUM, orc.POOL_WSUM, orc.POOL_MEAN, orc.POOL_WSUM, orc.POOL_SUM]
    full = orc.embedding_bag(tables, B, F, sf, ti, pool, ids, off, w)
    assert full.shape == (B, 4 + 8 + 16 + 8 + 8)
    col = 0
    for s in range(5):
        one = orc.embedding_bag(tables, B, F, [sf[s]], [ti[s]], [pool[s]], ids, off, w)
        D = tables[ti[s]].dim
        assert np.array_equal(full[:, col:col + D], one)
        col += D
    # sampled evaluation returns the same rows
    pick = [3, 0, 39, 17]
    assert np.array_equal(orc.embedding_bag(tables, B, F, sf, ti, pool, ids, off, w, samples=pick), full[pick])
    # a wider leading dimension leaves the extra columns untouched (zero)
    wide = orc.embedding_bag(tables, B, F, sf, ti, pool, ids, off, w, out_ld=60)
    assert np.array_equal(wide[:, :44], full) and not wide[:, 44:].any()


def test_exact_sums_on_grid_tables_any_order():
    """With grid-valued tables every unweighted sum is exact, so fp32 and fp64, in any order, agree bit for bit."""
    rng = np.random.default_rng(10)
    t = orc.Table(rows=1000, dim=8, dtype=orc.BF16, hash_seed=5, value_key=99, value_mode=orc.VAL_GRID)
    B = 30
    lens = rng.integers(0, 300, size=B)
    off = np.zeros(B + 1, np.int64)
    np.cumsum(lens, out=off[1:])
    ids = rng.integers(0, 2**40, size=int(off[-1]), dtype=np.uint64)
    out = orc.embedding_bag([t], B, 1, [0], [0], [orc.POOL_SUM], ids, off)
    rows = orc.hash_ids(ids, 5, 1000)
    dense = _dense(t).astype(np.float32)
    for b in range(B):
        acc = np.zeros(8, np.float32)
        for r in rows[off[b]:off[b + 1]][::-1]:  # reversed order, fp32
            acc += dense[r]
        assert np.array_equal(out[b], acc)


def test_invalid_arguments_are_rejected():
    t = orc.Table(rows=4, dim=2, dtype=orc.F32, data=np.zeros((4, 2), np.float32))
    ids = np.array([9], np.uint64)
    off = np.array([0, 1], np.int64)
    with pytest.raises(ValueError):
        orc.embedding_bag([t], 1, 1, [0], [0], [orc.POOL_SUM], ids, off, ids_are_rows=True)
    with pytest.raises(ValueError):
        orc.embedding_bag([t], 1, 1, [0], [0], [7], ids, off)
    with pytest.raises(ValueError):
        orc.embedding_bag([t], 1, 1, [0], [0], [orc.POOL_WSUM], ids, off, None)


# ------------------------------------------------------------------ dedup ---

@pytest.mark.parametrize("n,hi", [(0, 10), (1, 10), (1000, 1), (1000, 50), (5000, 10**12), (4097, 3000)])
def test_dedup_vs_numpy_unique(n, hi):
    rng = np.random.default_rng(11)
    rows = rng.integers(0, hi, size=n, dtype=np.int64)
    uniq, inv = orc.dedup(rows)
    wu, wi = np.unique(rows, return_inverse=True)
    assert np.array_equal(uniq, wu) and np.array_equal(inv, wi.astype(np.int32))
    assert (np.diff(uniq) > 0).all()
    assert np.array_equal(uniq[inv], rows)
    assert uniq.size == len(set(rows.tolist()))


# ------------------------------------------------------------------- INT4 ---

def test_int4_round_trip_error_bound():
    """Section 4.1.2 gives no INT4 format; this build's format is pinned by its own
    error bound: |x - decode| <= scale/2 + the fp16 rounding of bias and scale."""
    rng = np.random.default_rng(12)
    for dim in (8, 32, 64, 128):
        for _ in range(50):
            x = (rng.standard_normal(dim) * 0.01).astype(np.float32)
            q = orc.int4_quantize_row(x)
            assert q.size == orc.row_bytes(dim, orc.INT4) and q.size % 16 == 0
            t = orc.Table(rows=1, dim=dim, dtype=orc.INT4, data=q)
            y = orc.decode_row(t, 0)
            scale = float(q[dim // 2:dim // 2 + 2].view(np.float16)[0])
            bias = float(q[dim // 2 + 2:dim // 2 + 4].view(np.float16)[0])
            lo, hi = float(x.min()), float(x.max())
            slack = abs(bias - lo) + 15 * abs(scale - (hi - lo) / 15) + 1e-9
            assert np.abs(x - y).max() <= scale / 2 + slack
            # codes decode to bias + code*scale exactly (fp32 fma)
            codes = np.array([(q[d // 2] >> (4 * (d & 1))) & 15 for d in range(dim)])
            want = (codes.astype(np.float64) * scale + bias).astype(np.float32)
            assert np.array_equal(y, want)
    # constant row: scale 0, every code 0, decodes to the fp16 of the value
    q = orc.int4_quantize_row(np.full(16, 0.5, np.float32))
    assert np.array_equal(orc.decode_row(orc.Table(rows=1, dim=16, dtype=orc.INT4, data=q), 0),
                          np.full(16, 0.5, np.float32))


# --------------------------------------------------------------- backward ---

def test_backward_vs_torch_autograd():
    """Section 4.3: the tables are fine-tuned, so gradients flow to looked-up rows."""
    rng = np.random.default_rng(13)
    B = 48
    tables, ids, off, w = _random_case(rng, rows=61, dims=[8], B=B, F=1, max_len=10)
    rows = rng.integers(0, 61, size=ids.size).astype(np.uint64)
    gout = rng.standard_normal((B, 8)).astype(np.float32)
    for pool, mode in ((orc.POOL_SUM, "sum"), (orc.POOL_MEAN, "mean"), (orc.POOL_WSUM, "sum")):
        got = orc.embedding_bag_backward_slot(tables, B, [0], [0], [pool], 0, 8, 0, rows, off, w, gout,
                                              ids_are_rows=True)
        weight = torch.from_numpy(_dense(tables[0])).requires_grad_(True)
        psw = torch.from_numpy(w.astype(np.float64)) if pool == orc.POOL_WSUM else None
        o = torch.nn.functional.embedding_bag(torch.from_numpy(rows.astype(np.int64)), weight,
                                              torch.from_numpy(off[:-1]), mode=mode, per_sample_weights=psw)
        o.backward(torch.from_numpy(gout.astype(np.float64)))
        np.testing.assert_allclose(got, weight.grad.numpy(), rtol=1e-9, atol=1e-12)
