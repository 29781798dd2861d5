"""Seeded synthetic workloads shaped like ads-ranking lookups.

This module produces INPUTS only: table shapes, raw IDs, CSR offsets, per-sample
weights and the list of hottest raw IDs. It holds none of the lookup method's
arithmetic (no hashing, no pooling, no table values) and imports only numpy, so
both the GPU path's callers and the CPU checker's callers can draw the very same
inputs from it.

The paper's tables are looked up with private production traffic; these five
workloads stand in for it: thousands of candidates per request, tens of sparse
ID features, Zipf-distributed raw 40-bit IDs, ragged multi-hot bags (Section 2.1
of the paper lists the feature families; its sequence features built on
engagement history are the long bags of workload 4).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

F32, F16, BF16, INT4 = 0, 1, 2, 3
POOL_SUM, POOL_MEAN, POOL_WSUM = 0, 1, 2
LOC_DEVICE, LOC_HOST = 0, 1

ID_BITS = 40
ID_SPACE = 1 << ID_BITS
_HEAD = 1 << 20  # ranks with an exact cumulative table
_RANK_MULT = np.uint64(0xD1342543DE82EF95)  # odd => rank -> id is a bijection mod 2^40


@dataclass
class TableSpec:
    rows: int
    dim: int
    dtype: int
    hash_seed: int
    value_key: int
    location: int = LOC_DEVICE


@dataclass
class Workload:
    name: str
    batch: int
    tables: List[TableSpec]
    n_features: int
    slot_feature: np.ndarray  # int32 [n_slots], nondecreasing
    table_ids: np.ndarray     # int32 [n_slots]
    pooling: np.ndarray       # int32 [n_slots]
    alpha: np.ndarray         # float64 [n_features], Zipf exponent per feature
    length_kind: str          # "uniform" | "poisson" | "lognormal"
    length_params: tuple
    weighted: bool
    run_seed: int
    cache_fraction: float = 0.0  # share of the host table's rows kept in the HBM cache
    feature_salt: np.ndarray = field(default=None)  # uint64 [n_features]

    @property
    def n_slots(self) -> int:
        return int(self.slot_feature.size)

    @property
    def out_dim(self) -> int:
        return int(sum(self.tables[int(t)].dim for t in self.table_ids))


@dataclass
class Batch:
    ids: np.ndarray                 # uint64 [nnz], feature-major bags
    offsets: np.ndarray             # int64 [n_features*batch + 1]
    weights: Optional[np.ndarray]   # float32 [nnz] or None


# --------------------------------------------------------------- samplers ---

class ZipfSampler:
    """Ranks k in [1, 2^40] with P(k) proportional to k^-alpha.

    Ranks up to 2^20 use an exact cumulative table; the tail inverts the
    midpoint-rule integral of x^-alpha over [2^20 + 1/2, 2^40 + 1/2] and rounds
    to the nearest rank.
    """

    def __init__(self, alpha: float):
        self.alpha = float(alpha)
        k = np.arange(1, _HEAD + 1, dtype=np.float64)
        self.cum = np.cumsum(k ** (-self.alpha))
        self.head_mass = float(self.cum[-1])
        self.a = _HEAD + 0.5
        self.b = ID_SPACE + 0.5
        if abs(self.alpha - 1.0) < 1e-12:
            self.tail_mass = float(np.log(self.b / self.a))
        else:
            e = 1.0 - self.alpha
            self.tail_mass = float((self.b ** e - self.a ** e) / e)
        self.total = self.head_mass + self.tail_mass

    def p_rank1(self) -> float:
        return 1.0 / self.total

    def draw(self, rng: np.random.Generator, n: int) -> np.ndarray:
        u = rng.random(n) * self.total
        ranks = np.empty(n, dtype=np.uint64)
        head = u < self.head_mass
        ranks[head] = np.searchsorted(self.cum, u[head], side="right").astype(np.uint64) + np.uint64(1)
        v = u[~head] - self.head_mass
        if abs(self.alpha - 1.0) < 1e-12:
            x = self.a * np.exp(v)
        else:
            e = 1.0 - self.alpha
            x = (self.a ** e + v * e) ** (1.0 / e)
        x = np.clip(np.rint(x), _HEAD + 1, ID_SPACE)
        ranks[~head] = x.astype(np.uint64)
        np.clip(ranks, 1, ID_SPACE, out=ranks)
        return ranks


def rank_to_id(ranks: np.ndarray, salt) -> np.ndarray:
    """Bijection from rank to raw 40-bit ID, so that popular IDs are scattered."""
    with np.errstate(over="ignore"):
        v = ranks.astype(np.uint64) * _RANK_MULT + np.uint64(salt)
    return v & np.uint64(ID_SPACE - 1)


def hot_ids(w: Workload, feature: int, count: int) -> np.ndarray:
    """Raw IDs of the `count` most probable ranks of a feature, most probable first."""
    return rank_to_id(np.arange(1, count + 1, dtype=np.uint64), w.feature_salt[feature])


def bag_lengths(rng: np.random.Generator, kind: str, params: tuple, n: int) -> np.ndarray:
    if kind == "uniform":
        lo, hi = params
        return rng.integers(lo, hi + 1, size=n, dtype=np.int64)
    if kind == "poisson":
        lam, cap = params
        return np.minimum(rng.poisson(lam, size=n), cap).astype(np.int64)
    if kind == "lognormal":
        median, sigma, cap = params
        z = rng.standard_normal(n)
        return np.minimum(np.floor(np.exp(np.log(median) + sigma * z)), cap).astype(np.int64)
    raise ValueError(kind)


# --------------------------------------------------------------- workloads --

def _seeds(run_seed: int, tag: int, n: int) -> np.ndarray:
    return np.random.default_rng([run_seed, tag]).integers(0, 2**63, size=n, dtype=np.uint64) * np.uint64(2) + np.uint64(1)


def make_workload(config: int, rows_scale: float = 1.0, batch_scale: float = 1.0) -> Workload:
    """Workload `config` in 1..5. `rows_scale` / `batch_scale` < 1 shrink table
    rows and batch for small parity cases; 1.0 is the full size."""
    run_seed = config - 1

    def R(r):
        return max(1, int(round(r * rows_scale)))

    def Bz(b):
        return max(1, int(round(b * batch_scale)))

    def specs(shapes, location=None):
        n = len(shapes)
        hs = _seeds(run_seed, 1, n)
        vk = _seeds(run_seed, 2, n)
        return [TableSpec(R(r), d, dt, int(hs[i]) if config != 1 else 0, int(vk[i]),
                          (location[i] if location else LOC_DEVICE))
                for i, (r, d, dt) in enumerate(shapes)]

    if config == 1:
        tables = specs([(100_000, 32, F32)])
        F = 1
        w = Workload("c1: 1 x 100k x 32 fp32, B=512, U{1..20}, sum", Bz(512), tables, F,
                     np.zeros(1, np.int32), np.zeros(1, np.int32), np.full(1, POOL_SUM, np.int32),
                     np.full(F, 1.05), "uniform", (1, 20), False, run_seed)
    elif config == 2:
        tables = specs([(10_000_000, 64, F16)] * 8)
        F = 8
        pooling = np.array([POOL_SUM] * 4 + [POOL_MEAN] * 4, np.int32)
        w = Workload("c2: 8 x 10M x 64 fp16, B=4096, Poisson(20)<=100, sum/mean", Bz(4096), tables, F,
                     np.arange(F, dtype=np.int32), np.arange(F, dtype=np.int32), pooling,
                     np.full(F, 1.1), "poisson", (20.0, 100), False, run_seed)
    elif config == 3:
        shapes = []
        for _ in range(4):
            shapes += [(50_000_000, 32, BF16), (50_000_000, 64, BF16), (50_000_000, 128, BF16)]
        tables = specs(shapes)
        F = 4
        w = Workload("c3: 4 features x 3 facets (50M x 32/64/128 bf16), B=8192, Poisson(10)<=64, wsum",
                     Bz(8192), tables, F, np.repeat(np.arange(F, dtype=np.int32), 3),
                     np.arange(12, dtype=np.int32), np.full(12, POOL_WSUM, np.int32),
                     np.full(F, 1.2), "poisson", (10.0, 64), True, run_seed)
    elif config == 4:
        tables = specs([(20_000_000, 64, BF16)] * 32)
        F = 32
        pooling = np.array([POOL_SUM if f % 2 == 0 else POOL_MEAN for f in range(F)], np.int32)
        alpha = np.random.default_rng([run_seed, 3]).uniform(0.9, 1.3, size=F)
        w = Workload("c4: 32 x 20M x 64 bf16, B=16384, lognormal(8,1.5)<=500, sum/mean", Bz(16384),
                     tables, F, np.arange(F, dtype=np.int32), np.arange(F, dtype=np.int32), pooling,
                     alpha, "lognormal", (8.0, 1.5, 500), False, run_seed)
    elif config == 5:
        shapes = [(1_000_000_000, 64, F16)] + [(10_000_000, 64, BF16)] * 16
        tables = specs(shapes, [LOC_HOST] + [LOC_DEVICE] * 16)
        F = 17
        w = Workload("c5: host 1B x 64 fp16 + 16 x 10M x 64 bf16, B=8192, Poisson(30)<=200, sum",
                     Bz(8192), tables, F, np.arange(F, dtype=np.int32), np.arange(F, dtype=np.int32),
                     np.full(F, POOL_SUM, np.int32), np.full(F, 1.05), "poisson", (30.0, 200),
                     False, run_seed, cache_fraction=0.02)
    else:
        raise ValueError("config must be 1..5")
    w.feature_salt = np.random.default_rng([run_seed, 4]).integers(0, ID_SPACE, size=w.n_features,
                                                                   dtype=np.uint64)
    return w


_SAMPLERS = {}


def make_batch(w: Workload, j: int = 0) -> Batch:
    """Batch `j` of the workload's rotation (distinct j => independent draws)."""
    rng = np.random.default_rng([w.run_seed, 5, j])
    B, F = w.batch, w.n_features
    lens = bag_lengths(rng, w.length_kind, w.length_params, F * B)
    offsets = np.zeros(F * B + 1, np.int64)
    np.cumsum(lens, out=offsets[1:])
    nnz = int(offsets[-1])
    ids = np.empty(nnz, np.uint64)
    for f in range(F):
        lo, hi = int(offsets[f * B]), int(offsets[(f + 1) * B])
        a = float(w.alpha[f])
        s = _SAMPLERS.get(a)
        if s is None:
            s = _SAMPLERS[a] = ZipfSampler(a)
        ids[lo:hi] = rank_to_id(s.draw(rng, hi - lo), w.feature_salt[f])
    weights = None
    if w.weighted:
        weights = (rng.integers(0, 1 << 24, size=nnz).astype(np.float32) * np.float32(2.0 ** -24))
    return Batch(ids, offsets, weights)
