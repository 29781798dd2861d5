"""Seeded random launch shapes against the oracle: table sets of mixed dtype and width (row
sizes that are not a power of two, rows wider than 512 bytes, INT4 rows), facets that share a
feature, unused features, every pooling, bag lengths from empty to several hundred, odd batch
sizes, and the pooling kernel's options (tile, staging capacity, lane mapping, overlapping
launches). Each case draws everything from its seed, so a failure names a reproducible shape."""
import numpy as np
import pytest

import oracle as orc
from paper_2508_05700_b200 import inputs as gi
from tests.helpers import DeviceTables, assert_close, forward

pytestmark = pytest.mark.gpu

DIMS = {gi.F32: [4, 12, 32, 64, 132], gi.F16: [8, 24, 64, 128, 264], gi.BF16: [8, 32, 56, 64, 128, 520],
        gi.INT4: [8, 32, 64, 136]}


def _lengths(rng, n, kind):
    if kind == 0:      # short, many empty
        lens = rng.integers(0, 6, n)
        lens[rng.random(n) < 0.3] = 0
    elif kind == 1:    # around the warp-per-bag threshold
        lens = rng.integers(40, 90, n)
    elif kind == 2:    # heavy tail
        lens = np.minimum(500, np.floor(np.exp(np.log(8) + 1.5 * rng.standard_normal(n)))).astype(np.int64)
    else:              # Poisson-like
        lens = rng.poisson(rng.integers(3, 40), n)
    return lens.astype(np.int64)


@pytest.mark.parametrize("seed", range(24))
def test_random_shape_matches_oracle(seed):
    rng = np.random.default_rng(1000 + seed)
    n_tables = int(rng.integers(1, 6))
    specs = []
    for t in range(n_tables):
        dt_ = [gi.F32, gi.F16, gi.BF16, gi.INT4][int(rng.integers(0, 4))]
        dim = int(rng.choice(DIMS[dt_]))
        rows = int(rng.choice([1, 17, 1000, 65537]))
        specs.append(gi.TableSpec(rows, dim, dt_, int(rng.integers(0, 2**62)), int(rng.integers(1, 2**62))))
    n_features = int(rng.integers(1, 5))
    n_slots = int(rng.integers(1, 8))
    slot_feature = np.sort(rng.integers(0, n_features, n_slots)).astype(np.int32)  # facets share a feature
    table_ids = rng.integers(0, n_tables, n_slots).astype(np.int32)
    pooling = rng.integers(0, 3, n_slots).astype(np.int32)
    B = int(rng.choice([1, 3, 31, 64, 129, 300, 777]))
    lens = np.concatenate([_lengths(rng, B, int(rng.integers(0, 4))) for _ in range(n_features)])
    off = np.zeros(n_features * B + 1, np.int64)
    np.cumsum(lens, out=off[1:])
    ids = rng.integers(0, 2**63, size=int(off[-1]), dtype=np.uint64)
    w = rng.random(ids.size).astype(np.float32)
    with DeviceTables(specs) as dt:
        m = dt.m
        ref = orc.embedding_bag(dt.oracle_tables, B, n_features, slot_feature, table_ids, pooling, ids, off, w)
        base = forward(dt, B, n_features, slot_feature, table_ids, pooling, ids, off, w)
        assert_close(base, ref, "seed %d, defaults" % seed)
        lens_fb = lens.reshape(n_features, B)
        col = 0
        for s in range(n_slots):
            D = specs[int(table_ids[s])].dim
            assert not base[lens_fb[int(slot_feature[s])] == 0, col:col + D].any()
            col += D
        m.mfet_set_option(dt.h, m.OPT_TILE, int(rng.choice([8, 24, 56, 128])))
        m.mfet_set_option(dt.h, m.OPT_STAGE_IDS, int(rng.choice([32, 200, 1024, 8192])))
        m.mfet_set_option(dt.h, m.OPT_GROUP_POLICY, int(rng.integers(0, 3)))
        m.mfet_set_option(dt.h, m.OPT_OVERLAP_LAUNCHES, int(rng.integers(0, 2)))
        got = forward(dt, B, n_features, slot_feature, table_ids, pooling, ids, off, w)
        assert_close(got, ref, "seed %d, options" % seed)
