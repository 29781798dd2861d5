"""Distribution checks of the synthetic workload generator (inputs only; both the GPU
path and the oracle read the same arrays, so a generator error cannot fake parity)."""
import numpy as np

from paper_2508_05700_b200 import inputs as gi


def test_zipf_rank1_frequency_and_range():
    rng = np.random.default_rng(0)
    for alpha in (0.9, 1.0, 1.05, 1.2):
        s = gi.ZipfSampler(alpha)
        r = s.draw(rng, 400_000)
        assert r.min() >= 1 and r.max() <= gi.ID_SPACE
        p1 = (r == 1).mean()
        assert abs(p1 - s.p_rank1()) < 4 * np.sqrt(s.p_rank1() / r.size) + 1e-4
        # rank 2 is 2^-alpha as likely as rank 1
        p2 = (r == 2).mean()
        assert abs(p2 / p1 - 2.0 ** -alpha) < 0.05
        # mass beyond the exact head matches the integral
        tail = (r > (1 << 20)).mean()
        assert abs(tail - s.tail_mass / s.total) < 0.01


def test_rank_to_id_is_a_bijection_on_a_sample():
    ranks = np.arange(1, 200_001, dtype=np.uint64)
    ids = gi.rank_to_id(ranks, 12345)
    assert ids.max() < gi.ID_SPACE and np.unique(ids).size == ranks.size


def test_bag_length_recipes():
    rng = np.random.default_rng(1)
    u = gi.bag_lengths(rng, "uniform", (1, 20), 100_000)
    assert u.min() == 1 and u.max() == 20 and abs(u.mean() - 10.5) < 0.1
    p = gi.bag_lengths(rng, "poisson", (20.0, 100), 100_000)
    assert p.min() >= 0 and p.max() <= 100 and abs(p.mean() - 20) < 0.1
    l = gi.bag_lengths(rng, "lognormal", (8.0, 1.5, 500), 400_000)
    assert l.max() == 500 and abs(np.median(l) - 7.5) <= 1.0
    assert 0.06 < (l == 0).mean() < 0.11 and 20 < l.mean() < 26


def test_workloads_shapes_and_determinism():
    for c, (L, D) in {1: (1, 32), 2: (8, 512), 3: (12, 896), 4: (32, 2048), 5: (17, 1088)}.items():
        w = gi.make_workload(c, rows_scale=1e-3, batch_scale=1 / 64)
        assert w.n_slots == L and w.out_dim == D
        b0, b1 = gi.make_batch(w, 0), gi.make_batch(w, 0)
        assert np.array_equal(b0.ids, b1.ids) and np.array_equal(b0.offsets, b1.offsets)
        assert b0.offsets.size == w.n_features * w.batch + 1 and b0.offsets[-1] == b0.ids.size
        assert (np.diff(b0.offsets) >= 0).all() and b0.ids.max() < gi.ID_SPACE
        assert not np.array_equal(gi.make_batch(w, 1).ids[:50], b0.ids[:50])
        assert (b0.weights is not None) == (c == 3)
        if b0.weights is not None:
            assert b0.weights.dtype == np.float32 and 0 <= b0.weights.min() and b0.weights.max() < 1
    w3 = gi.make_workload(3)
    assert [t.dim for t in w3.tables[:3]] == [32, 64, 128] and w3.slot_feature.tolist() == [0] * 3 + [1] * 3 + [2] * 3 + [3] * 3
    w5 = gi.make_workload(5)
    assert w5.tables[0].location == gi.LOC_HOST and w5.tables[0].rows == 10**9


def test_hot_ids_are_the_most_frequent():
    w = gi.make_workload(5, rows_scale=1e-3, batch_scale=1 / 8)
    b = gi.make_batch(w, 0)
    f0 = b.ids[b.offsets[0]:b.offsets[w.batch]]
    top = gi.hot_ids(w, 0, 1)[0]
    vals, counts = np.unique(f0, return_counts=True)
    assert vals[counts.argmax()] == top
