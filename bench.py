#!/usr/bin/env python
"""Benchmark of the embedding-table lookup path: pooled IDs per second.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference]

One step = one pass of the whole lookup path (hash -> gather -> pool -> concat, plus
dedup -> cache probe -> host fetch for a host-resident table) over one synthetic batch.
`value` is measured with the batch resident in HBM; `e2e` goes through the C-ABI call
that takes HOST buffers (copies in and out inside the timed region). N > 1 runs N
independent replicas (the path has no exchange step), one process per GPU.

The default run on one GPU times workload 3 (the headline: batch 8192, multi-faceted) under
the step contract, and then every workload 1..5 (workloads 2 and 4 also with uniform IDs, i.e.
without repeated rows) into the `workloads` object of the same JSON line: each as R repeats of
a K-step region with launches back to back, the same with every launch by itself, and a
series with the L2 flushed before every step; median / p10 / p90 of each.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2508_05700_b200 import inputs as gi  # noqa: E402

METRIC = "pooled_ids_per_sec"
UNIT = "IDs/s"
DEFAULT_CONFIG = 3
NOMINAL_HBM_GBS = 8000.0  # the bar of the task is stated against this figure
KERNEL_SOURCES = ["paper_2508_05700_b200/csrc/bag.cu", "paper_2508_05700_b200/csrc/common.cuh"]
REPEATS = 15          # K-step regions per series
COLD_STEPS = 40       # steps of the series with the L2 flushed before every step
L2_FLUSH_BYTES = 256 << 20


# ------------------------------------------------------------------ helpers --

def gi_row_bytes(t: gi.TableSpec) -> int:
    if t.dtype == gi.INT4:
        return (t.dim // 2 + 4 + 15) // 16 * 16
    return t.dim * (4 if t.dtype == gi.F32 else 2)


def algorithmic_bytes(w: gi.Workload, b: gi.Batch, slots=None) -> int:
    """Bytes the method must move for one batch: one stored row per lookup, 8 per input ID
    (+4 if weighted), 8 per bag offset, 4 per output element."""
    B = w.batch
    slots = range(w.n_slots) if slots is None else slots
    feats = sorted({int(w.slot_feature[s]) for s in slots})
    total = 0
    out_dim = 0
    for s in slots:
        f = int(w.slot_feature[s])
        t = w.tables[int(w.table_ids[s])]
        n_f = int(b.offsets[(f + 1) * B] - b.offsets[f * B])
        total += n_f * gi_row_bytes(t)
        out_dim += t.dim
    nnz = sum(int(b.offsets[(f + 1) * B] - b.offsets[f * B]) for f in feats)
    total += nnz * (8 + (4 if b.weights is not None else 0))
    total += (len(feats) * B + 1) * 8
    total += B * out_dim * 4
    return total


def row_lookups(w: gi.Workload, b: gi.Batch, slots=None) -> int:
    slots = range(w.n_slots) if slots is None else slots
    return sum(int(b.offsets[(int(w.slot_feature[s]) + 1) * w.batch] - b.offsets[int(w.slot_feature[s]) * w.batch])
               for s in slots)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def kernel_fingerprint() -> str:
    h = hashlib.sha256()
    for p in KERNEL_SOURCES:
        with open(os.path.join(ROOT, p), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def recorded_traffic(workload_key: str):
    """(DRAM bytes per launch of the pooling kernel, note) from the committed ncu summary; (None, None)
    when there is none for this workload or the kernel sources changed since it was taken. The
    captures are taken on row-reduced tables at the full batch (a few GB on the device); a launch
    processes the same IDs as at full size, so the figure is used per launch as it stands."""
    path = os.path.join(ROOT, "profiles", "bag_kernel_dram_traffic.txt")
    if not os.path.exists(path):
        return None, None
    fp = kernel_fingerprint()
    with open(path) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            f = line.split(None, 3)
            if len(f) >= 3 and f[0] == workload_key and f[1] == fp:
                return float(f[2]), (f[3].strip() if len(f) > 3 else None)
    return None, None


def stats(xs):
    a = np.asarray(xs, np.float64)
    return {"median": float(np.median(a)), "p10": float(np.percentile(a, 10)), "p90": float(np.percentile(a, 90)),
            "n": int(a.size)}


class ClockSampler:
    """nvidia-smi clock / throttle sampling while the GPU is under load."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], None, set()
        for ts, line in self.lines:
            if ts < t0 or ts > t1 + 0.15:
                continue
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax = float(f[2])
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": smax, "reasons": sorted(reasons),
                "samples": len(sm)}


def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def aggregate_over_ranks(local_ms: float, local_units: float, dist=None):
    """Slowest rank's time and the units all ranks processed (replicas: no data exchange)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return local_ms, local_units
    import torch
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([local_ms], dtype=torch.float64, device=dev)
    u = torch.tensor([local_units], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


# --------------------------------------------------------------- CPU oracle --

def cpu_model() -> str:
    try:
        with open("/proc/cpuinfo") as fh:
            for line in fh:
                if line.lower().startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def mem_available() -> int:
    try:
        with open("/proc/meminfo") as fh:
            return {l.split(":")[0]: int(l.split()[1]) * 1024 for l in fh}["MemAvailable"]
    except (OSError, KeyError):
        return 8 << 30


def oracle_tables_materialised(w: gi.Workload, threads: int, budget_bytes: int):
    """The oracle's tables with their rows MATERIALISED in host memory (written by the oracle's own
    generator), so that the timed oracle gathers rows from memory instead of recomputing values.
    When the tables do not fit the budget, every table gets the same fraction of its rows (the IDs
    then hash into the smaller tables): a row-reduced replica, labelled "scaled"."""
    import oracle as orc
    total = sum(t.rows * gi_row_bytes(t) for t in w.tables)
    frac = min(1.0, budget_bytes / max(1, total))
    tabs, nbytes = [], 0
    with ThreadPoolExecutor(max_workers=threads) as ex:
        for t in w.tables:
            rows = t.rows if frac >= 1.0 else max(1, int(t.rows * frac))
            spec = orc.Table(rows=rows, dim=t.dim, dtype=t.dtype, hash_seed=t.hash_seed, value_key=t.value_key)
            data = np.empty((rows, gi_row_bytes(t)), np.uint8)
            cuts = np.linspace(0, rows, threads * 4 + 1).astype(np.int64)

            def fill(k, spec=spec, data=data, cuts=cuts):
                r0, r1 = int(cuts[k]), int(cuts[k + 1])
                if r1 > r0:
                    data[r0:r1] = orc.table_fill(spec, r0, r1).reshape(r1 - r0, -1)
            list(ex.map(fill, range(threads * 4)))
            tabs.append(orc.Table(rows=rows, dim=t.dim, dtype=t.dtype, hash_seed=t.hash_seed, value_key=t.value_key,
                                  data=data))
            nbytes += data.nbytes
    kind = "materialised host copy of the tables" if frac >= 1.0 else \
        "materialised row-reduced replica of the tables (scaled: %.4f of the rows of every table)" % frac
    return tabs, kind, nbytes


def oracle_run_samples(w, b, tabs, samples, threads):
    """The oracle, as it stands, over the given samples; sharded over samples on `threads`
    host threads (the C routine runs without the interpreter lock)."""
    import oracle as orc
    chunks = [c for c in np.array_split(np.asarray(samples), threads) if c.size]

    def run(c):
        orc.embedding_bag(tabs, w.batch, w.n_features, w.slot_feature, w.table_ids, w.pooling, b.ids, b.offsets,
                          b.weights, samples=c.tolist())
    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=len(chunks)) as ex:
        list(ex.map(run, chunks))
    return time.perf_counter() - t0


def ids_in_samples(w, b, samples):
    off = b.offsets.reshape(-1)
    n = 0
    for f in range(w.n_features):
        idx = f * w.batch + np.asarray(samples)
        n += int((off[idx + 1] - off[idx]).sum())
    return n


def oracle_rate(w, batches, tabs, threads, target_seconds):
    """IDs per second of the oracle on about `target_seconds` of work with `threads` threads: whole
    batches of the rotation when a batch is quick, else the first samples of batch 0."""
    b = batches[0]
    probe = list(range(min(w.batch, 4 * threads)))
    oracle_run_samples(w, b, tabs, probe, threads)  # first touch: library load, thread start, page faults
    dt = max(oracle_run_samples(w, b, tabs, probe, threads), 1e-5)
    per_sample = dt / len(probe)
    if per_sample * w.batch > target_seconds:
        n = int(max(threads, target_seconds / per_sample))
        samples = list(range(min(n, w.batch)))
        total = oracle_run_samples(w, b, tabs, samples, threads)
        n_ids = ids_in_samples(w, b, samples)
        what = "samples 0..%d of batch 0" % (len(samples) - 1)
    else:
        samples = list(range(w.batch))
        total, n_ids, reps = 0.0, 0, 0
        while total < target_seconds and reps < 4096:
            bb = batches[reps % len(batches)]
            total += oracle_run_samples(w, bb, tabs, samples, threads)
            n_ids += int(bb.offsets[-1])
            reps += 1
        what = "%d whole batches (rotation of %d)" % (reps, len(batches))
    return n_ids / total, "%s, %d IDs, %.1f s" % (what, n_ids, total)


def cpu_baseline(w, batches):
    """The oracle timed on this machine's host cores over a bounded sample of the workload, reading
    materialised tables: with one thread and with all hardware threads (`value`)."""
    import oracle as orc
    orc.build()
    threads = os.cpu_count() or 1
    budget = int(min(6 << 30, 0.2 * mem_available()))
    t0 = time.perf_counter()
    tabs, kind, nbytes = oracle_tables_materialised(w, threads, budget)
    t_fill = time.perf_counter() - t0
    one, what1 = oracle_rate(w, batches, tabs, 1, 4.0)
    many, whatn = oracle_rate(w, batches, tabs, threads, 8.0)
    return {"value": many, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": "%s of %s; all %d threads: %s; one thread: %s" % (kind, w.name, threads, whatn, what1),
            "one_thread": {"value": one, "unit": UNIT, "cores": 1},
            "tables": kind, "table_bytes_on_host": int(nbytes), "table_fill_s": t_fill,
            "cpu_model": cpu_model(), "nproc": threads}


def run_reference(args):
    """--impl reference: the CPU oracle timed on this machine's host cores, each step a bounded
    sample of the workload (materialised tables, all hardware threads)."""
    rank, _, world = dist_env()
    if rank != 0:
        return 0
    import oracle as orc
    orc.build()
    args.config = args.config or DEFAULT_CONFIG
    w = gi.make_workload(args.config)
    for t in w.tables:
        t.location = gi.LOC_DEVICE  # placement is transparent to the oracle
    b = gi.make_batch(w, 0)
    threads = os.cpu_count() or 1
    tabs, kind, nbytes = oracle_tables_materialised(w, threads, int(min(6 << 30, 0.2 * mem_available())))
    probe = list(range(min(w.batch, 4 * threads)))
    oracle_run_samples(w, b, tabs, probe, threads)
    dt = max(oracle_run_samples(w, b, tabs, probe, threads), 1e-5)
    budget = 60.0 / max(1, args.steps + args.warmup)
    n = int(min(w.batch, max(threads, budget / (dt / len(probe)))))
    times, ids_done = [], 0
    for step in range(args.warmup + args.steps):
        lo = (step * n) % max(1, w.batch - n + 1)
        samples = list(range(lo, lo + n))
        dt = oracle_run_samples(w, b, tabs, samples, threads)
        if step >= args.warmup:
            times.append(dt)
            ids_done += ids_in_samples(w, b, samples)
    total = sum(times)
    value = ids_done / total
    sample = "%d samples of batch 0 per step (%d IDs per step on average), %s" % (
        n, ids_done // max(1, args.steps), kind)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / max(1, args.steps),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "config": args.config, "batch": w.batch},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample,
                             "cpu_model": cpu_model()},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------ GPU arm --

def host_rows_that_fit(w: gi.Workload):
    """Rows of the host-resident table that this box can pin (it needs rows*row_bytes of
    host RAM next to everything else); the full row count when memory allows."""
    avail = mem_available()
    out = {}
    for i, t in enumerate(w.tables):
        if t.location == gi.LOC_HOST:
            fit = int(0.70 * avail) // gi_row_bytes(t)
            out[i] = min(t.rows, fit)
    return out


class Ctx:
    """One workload set up on the GPU: tables filled, batches resident."""

    def __init__(self, args, config, rank, alpha=None, int4=False, device_slots_only=False, n_batches=None):
        import torch

        from paper_2508_05700_b200 import mfet as m
        from paper_2508_05700_b200.runtime import LookupEngine
        self.m, self.torch = m, torch
        w = gi.make_workload(config, rows_scale=args.rows_scale)
        if alpha is not None:  # e.g. 0 = uniform IDs: no row repeats, the pure random-gather case
            w.alpha = np.full(w.n_features, float(alpha))
            w.name += ", Zipf alpha overridden to %g" % alpha
        if int4:  # the same tables stored as INT4 rows (paper, Section 4.1.2)
            for t in w.tables:
                t.dtype = gi.INT4
            w.name += ", tables stored as INT4"
        if device_slots_only:  # the HBM-resident part of a hybrid workload, as a workload of its own
            keep = [s for s in range(w.n_slots) if w.tables[int(w.table_ids[s])].location == gi.LOC_DEVICE]
            for t in w.tables:
                if t.location != gi.LOC_DEVICE:
                    t.rows = 1024
            w.slot_feature, w.table_ids, w.pooling = w.slot_feature[keep], w.table_ids[keep], w.pooling[keep]
            w.name += ", device-table slots only"
        self.scaled_host = False
        for i, rows in host_rows_that_fit(w).items():
            if rows < w.tables[i].rows:
                w.tables[i].rows = rows
                self.scaled_host = True
        self.w, self.config = w, config
        self.n_rot = n_batches or args.batches
        self.batches = [gi.make_batch(w, rank * 1000 + j) for j in range(self.n_rot)]
        self.eng = LookupEngine(w, device=torch.cuda.current_device())
        if args.tile:
            m.mfet_set_option(self.eng.h, m.OPT_TILE, args.tile)
        if args.stage_ids:
            m.mfet_set_option(self.eng.h, m.OPT_STAGE_IDS, args.stage_ids)
        self.stream = torch.cuda.current_stream()
        self.d_ids = [torch.from_numpy(b.ids.view(np.int64)).cuda() for b in self.batches]
        self.d_off = [torch.from_numpy(b.offsets).cuda() for b in self.batches]
        self.d_w = [None if b.weights is None else torch.from_numpy(b.weights).cuda() for b in self.batches]
        self.out = torch.empty(w.batch, w.out_dim, dtype=torch.float32, device="cuda")
        self.nnz = [int(b.offsets[-1]) for b in self.batches]
        self.dev_slots = [s for s in range(w.n_slots) if w.tables[int(w.table_ids[s])].location == gi.LOC_DEVICE]
        self.all_dev = len(self.dev_slots) == w.n_slots
        if not self.all_dev:
            self.sub_shape, self._keep = m.make_shape(w.batch, w.n_features, w.slot_feature[self.dev_slots])
            self.sub_out = torch.empty(w.batch, sum(w.tables[int(w.table_ids[s])].dim for s in self.dev_slots),
                                       device="cuda")

    def pool_device_slots(self, k):
        """One launch of the pooling kernel: all HBM-resident slots of batch k."""
        w, e = self.w, self.eng
        if self.all_dev:
            e.forward(self.d_ids[k], self.d_off[k], self.d_w[k], self.out)
        else:
            e.forward(self.d_ids[k], self.d_off[k], self.d_w[k], self.sub_out, table_ids=w.table_ids[self.dev_slots],
                      pooling=w.pooling[self.dev_slots], shape=self.sub_shape)

    def close(self):
        self.eng.close()
        self.d_ids = self.d_off = self.d_w = self.out = None
        self.torch.cuda.empty_cache()


def region_series(ctx, step, steps, repeats):
    """`repeats` regions of `steps` steps each, one CUDA-event pair around a region on the launching
    stream; returns the per-step time of every region in microseconds."""
    torch = ctx.torch
    us = []
    for _ in range(repeats):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(ctx.stream)
        for j in range(steps):
            step(j)
        b.record(ctx.stream)
        b.synchronize()
        us.append(a.elapsed_time(b) * 1e3 / steps)
    return us


def pooling_series(ctx, args, flush):
    """The pooling kernel over all HBM-resident slots (one launch per step), three ways:
    launches back to back (a launch may stage and hash while its predecessor drains), every
    launch by itself, and with an L2-sized buffer written before every step (cold L2; one event
    pair per step)."""
    m, torch = ctx.m, ctx.torch
    w = ctx.w
    peak, peak_kind = measured_peaks()
    alg = float(np.mean([algorithmic_bytes(w, b, ctx.dev_slots) for b in ctx.batches]))
    ids = float(np.mean([sum(int(b.offsets[(f + 1) * w.batch] - b.offsets[f * w.batch])
                             for f in sorted({int(w.slot_feature[s]) for s in ctx.dev_slots})) for b in ctx.batches]))
    lookups = float(np.mean([row_lookups(w, b, ctx.dev_slots) for b in ctx.batches]))

    def step(j):
        ctx.pool_device_slots(j % ctx.n_rot)
    for j in range(max(3, args.warmup)):
        step(j)
    torch.cuda.synchronize()
    out = {"ids_per_launch": ids, "row_lookups_per_launch": lookups, "algorithmic_bytes_per_launch": alg,
           "bytes_per_id": alg / max(1.0, ids)}

    def describe(us):
        s = stats(us)
        med = s["median"] * 1e-6
        return {"us_per_step": s, "ids_per_s": ids / med, "row_lookups_per_s": lookups / med,
                "alg_gbps": alg / med / 1e9, "frac_of_copy_bw": alg / med / 1e9 / peak,
                "frac_of_8tbs": alg / med / 1e9 / NOMINAL_HBM_GBS}
    m.mfet_set_option(ctx.eng.h, m.OPT_OVERLAP_LAUNCHES, 1)
    out["back_to_back"] = describe(region_series(ctx, step, args.steps, REPEATS))
    m.mfet_set_option(ctx.eng.h, m.OPT_OVERLAP_LAUNCHES, 0)
    out["by_itself"] = describe(region_series(ctx, step, args.steps, REPEATS))
    cold = []
    for j in range(COLD_STEPS + 3):
        flush.fill_(j & 1)  # evicts the L2; outside the event pair
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(ctx.stream)
        step(j)
        b.record(ctx.stream)
        b.synchronize()
        if j >= 3:
            cold.append(a.elapsed_time(b) * 1e3)
    out["cold_l2"] = describe(cold)
    out["cold_l2"]["note"] = "%d MiB written before every step, one event pair per step" % (L2_FLUSH_BYTES >> 20)
    out["peak_gbps"] = peak
    out["peak_kind"] = peak_kind + " copy bandwidth"
    return out


def measure(args, config, rank, world, dist, with_cpu_baseline, sampler_gpu=None):
    """One workload under the step contract: set-up, warm-up, exactly K timed steps (device-resident
    inputs), the pooling kernel's three series, the end-to-end series through host buffers."""
    import torch

    from paper_2508_05700_b200 import mfet as m

    ctx = Ctx(args, config, rank, alpha=args.alpha, int4=args.int4, device_slots_only=args.device_slots_only)
    w, eng, batches, n_rot = ctx.w, ctx.eng, ctx.batches, ctx.n_rot
    d_ids, d_off, d_w, out, nnz, stream = ctx.d_ids, ctx.d_off, ctx.d_w, ctx.out, ctx.nnz, ctx.stream
    base = cpu_baseline(w, batches) if with_cpu_baseline else None
    if not args.no_overlap_launches:
        # the batches are resident before the timed region: a step's kernel may hash its IDs while the
        # step before it finishes (it waits for that kernel before it writes the output)
        m.mfet_set_option(eng.h, m.OPT_OVERLAP_LAUNCHES, 1)
    host_tabs = [] if args.device_slots_only else eng.host_table_ids()
    cached_rows = 0
    B = w.batch
    host_feats = sorted({int(w.slot_feature[s]) for s in range(w.n_slots) if int(w.table_ids[s]) in host_tabs})
    if host_tabs:
        worst = max(int(b.offsets[(f + 1) * B] - b.offsets[f * B]) for b in batches for f in host_feats)
        ws_ids = int(worst * 1.25) + 4096
        eng.set_workspace(ws_ids)
        for t in host_tabs:
            f = int(w.slot_feature[list(w.table_ids).index(t)])
            cached_rows = eng.build_hot_cache(t, f, int(w.tables[t].rows * w.cache_fraction))
        m.mfet_set_option(eng.h, m.OPT_PROFILE, 1)

    # Hybrid workload: the fetch of the next batch's host-table rows starts before the current
    # batch is pooled (the paper's early embedding fetch, Section 3.4): the library's dedup of
    # batch j+1 and the PCIe reads of its rows run while batch j is pooled. Results are
    # bit-identical to the serial path (tests). `seq` numbers the steps across warm-up, load
    # phase and timed region, because every step announces its successor.
    n_host_slots = sum(1 for s in range(w.n_slots) if int(w.table_ids[s]) in host_tabs)
    can_pipeline = bool(host_tabs) and n_host_slots == 1
    pipelined = can_pipeline and not args.serial_host_path
    seq = [0]
    if can_pipeline:
        pre_shape, _keep_pre = m.make_shape(w.batch, w.n_features, w.slot_feature)
        pre_shape.flags |= m.BATCH_PREFETCHED
    if pipelined:
        m.mfet_host_prefetch(eng.h, eng.shape, d_ids[0], d_off[0], w.table_ids, stream.cuda_stream)

    def step(_j=None):
        k, kn = seq[0] % n_rot, (seq[0] + 1) % n_rot
        seq[0] += 1
        if pipelined:
            m.mfet_host_prefetch(eng.h, eng.shape, d_ids[kn], d_off[kn], w.table_ids, stream.cuda_stream)
            m.mfet_embedding_bag_forward(eng.h, pre_shape, d_ids[k], d_off[k], d_w[k], w.table_ids, w.pooling, out,
                                         stream.cuda_stream)
        else:
            eng.forward(d_ids[k], d_off[k], d_w[k], out)
        return k

    def drain_pipeline():
        # pool the batch that the last step announced: nothing is left outstanding
        k = seq[0] % n_rot
        m.mfet_embedding_bag_forward(eng.h, pre_shape, d_ids[k], d_off[k], d_w[k], w.table_ids, w.pooling, out,
                                     stream.cuda_stream)
        torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(torch.cuda.current_device()) if sampler_gpu is not None else None
    if sampler:
        sampler.start()
    # warm-up: W steps, then keep the GPU under the same load for about a second so that the
    # clock samples around the timed region describe the loaded state
    for j in range(args.warmup):
        step(j)
    torch.cuda.synchronize()
    t_load0 = time.time()
    while time.time() - t_load0 < args.load_seconds:
        for _ in range(50):
            step()
        torch.cuda.synchronize()

    # ---- timed region: exactly K steps, inputs resident in HBM ----------------
    launches0 = m.mfet_launch_count(eng.h)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    timed_batches = [step() for _ in range(args.steps)]
    e1.record(stream)
    barrier()
    local_ms = e0.elapsed_time(e1)
    launches = m.mfet_launch_count(eng.h) - launches0
    ids_done = sum(nnz[k] for k in timed_batches)
    # the same region repeated: median / p10 / p90 of the step time
    step_us = [local_ms * 1e3 / args.steps]
    if world == 1:
        for _ in range(REPEATS - 1):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(args.steps):
                step()
            b.record(stream)
            b.synchronize()
            step_us.append(a.elapsed_time(b) * 1e3 / args.steps)
    serial_step_us = None
    if pipelined:
        drain_pipeline()
        pipelined = False
        if world == 1:  # the same steps without the early fetch: one request at a time
            for _ in range(3):
                step()
            serial_step_us = stats(region_series(ctx, lambda j: step(), min(args.steps, 50), 5))
    assert m.mfet_query_status(eng.h) == 0, "device error bits set during the timed region"

    # ---- the pooling kernel alone: all HBM-resident slots, one launch per step ----
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")
    series = pooling_series(ctx, args, flush)
    if not args.no_overlap_launches:
        m.mfet_set_option(eng.h, m.OPT_OVERLAP_LAUNCHES, 1)
    alg = series["algorithmic_bytes_per_launch"]
    # the kernel's average launch duration over the timed region when a step is exactly one launch
    kern_ms = local_ms / args.steps if ctx.all_dev else series["back_to_back"]["us_per_step"]["median"] * 1e-3
    kern_ms_serialized = series["by_itself"]["us_per_step"]["median"] * 1e-3

    # ---- host-table path alone (PCIe roofline): stage times from the library's events ----
    host_path = None
    if host_tabs:
        t0 = host_tabs[0]
        row_b = gi_row_bytes(w.tables[t0])
        nbytes = min(1 << 30, w.tables[t0].rows * row_b)
        src = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
        dst = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        best = 0.0
        for rep in range(5):
            c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            c0.record(stream)
            dst.copy_(src, non_blocking=True)  # one DMA copy, pinned host -> device
            c1.record(stream)
            torch.cuda.synchronize()
            best = max(best, nbytes / (c0.elapsed_time(c1) * 1e-3) / 1e9)
        peak_h2d = best
        del dst, src
        stages = np.zeros(3)
        reps = min(args.steps, 50)
        for j in range(reps):
            step(j)
            torch.cuda.synchronize()
            stages += np.array(m.mfet_profile_read(eng.h))
        stages /= reps
        n_uniq, n_miss = m.mfet_host_path_counts(eng.h)  # distinct rows, distinct uncached rows of the last batch
        fetched = n_miss * row_b
        # what the platform gives the same fetch kernel on as many rows of the same registered table:
        # uniformly random rows, and consecutive rows
        rng = np.random.default_rng(7)
        n_probe = max(1, n_miss)
        rows_tab = int(w.tables[t0].rows)
        lists = {"random": np.sort(rng.integers(0, rows_tab, size=n_probe, dtype=np.int64)),
                 "sequential": (rows_tab // 3 + np.arange(n_probe, dtype=np.int64)) % rows_tab}
        probe_dst = torch.empty(n_probe * row_b, dtype=torch.uint8, device="cuda")
        ceilings = {}
        for name, rows_list in lists.items():
            d_rows = torch.from_numpy(rows_list).cuda()
            best_ms = None
            for rep in range(4):
                if name == "random":  # other rows every time: nothing is served from a cache on the way
                    d_rows = torch.from_numpy(np.sort(rng.integers(0, rows_tab, size=n_probe, dtype=np.int64))).cuda()
                c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                c0.record(stream)
                m.mfet_host_fetch_rows(eng.h, t0, d_rows, n_probe, probe_dst, stream.cuda_stream)
                c1.record(stream)
                torch.cuda.synchronize()
                ms = c0.elapsed_time(c1)
                if rep > 0:
                    best_ms = ms if best_ms is None else min(best_ms, ms)
            ceilings[name + "_rows_gbps"] = n_probe * row_b / (best_ms * 1e-3) / 1e9
        del probe_dst
        # how many of a batch's distinct uncached rows were already fetched for one of the 8 batches before it
        seen, shares = [], []
        cache_keys = None
        for j in range(min(n_rot, 9)):
            eng.forward(d_ids[j], d_off[j], d_w[j], out)
            torch.cuda.synchronize()
            nm = m.mfet_host_path_counts(eng.h)[1]
            miss = torch.empty(ws_ids, dtype=torch.int64, device="cuda")
            m.mfet_host_path_result(eng.h, None, None, miss, ws_ids)
            cur = miss[:nm].cpu().numpy()
            if seen:
                prev = np.unique(np.concatenate(seen[-8:]))
                shares.append(float(np.isin(cur, prev).mean()) if cur.size else 0.0)
            seen.append(cur)
        host_path = {"bound": "pcie", "kernel": "fetch_rows_kernel (zero-copy reads of the missed rows)",
                     "lookups_per_step": int(np.mean([int(b.offsets[(host_feats[0] + 1) * B] - b.offsets[host_feats[0] * B])
                                                      for b in batches])),
                     "unique_rows_per_step": n_uniq, "unique_missed_rows_per_step": n_miss, "row_bytes": row_b,
                     "achieved": fetched / (stages[1] * 1e-3) / 1e9 if stages[1] > 0 else None,
                     "peak": peak_h2d, "unit": "GB/s",
                     "frac": (fetched / (stages[1] * 1e-3) / 1e9 / peak_h2d) if stages[1] > 0 and peak_h2d else None,
                     "peak_kind": "measured DMA copy of 1 GiB, pinned host to device, in this run",
                     "stage_ms": {"hash_dedup_probe": float(stages[0]), "fetch": float(stages[1]), "pool": float(stages[2])},
                     "same_kernel_on_%d_rows_of_this_table" % n_probe: ceilings,
                     "frac_of_random_rows_rate": (fetched / (stages[1] * 1e-3) / 1e9 / ceilings["random_rows_gbps"])
                     if stages[1] > 0 else None,
                     "missed_rows_seen_in_the_8_batches_before": {"share": float(np.mean(shares)) if shares else None,
                                                                   "batches": len(shares)},
                     "host_rows": int(w.tables[t0].rows), "scaled_to_fit_host_ram": ctx.scaled_host}

    # ---- end to end: host buffers in, host result out, through the C-ABI call ---
    p_ids = [torch.from_numpy(b.ids.view(np.int64)).pin_memory() for b in batches]
    p_off = [torch.from_numpy(b.offsets).pin_memory() for b in batches]
    p_w = [None if b.weights is None else torch.from_numpy(b.weights).pin_memory() for b in batches]
    io_bytes = max(m.mfet_host_io_bytes(eng.h, eng.shape, w.table_ids, n) for n in nnz)
    # two steps in flight on two streams, each with its own device scratch and pinned result buffer:
    # the result copy of one step overlaps the input copy and the kernels of the next (PCIe is full duplex)
    lanes = [torch.cuda.Stream(), torch.cuda.Stream()]
    p_out = [torch.empty(w.batch, w.out_dim, dtype=torch.float32).pin_memory() for _ in lanes]
    io = [torch.empty(io_bytes, dtype=torch.uint8, device="cuda") for _ in lanes]

    def e2e_step(j):
        k, a = j % n_rot, j % 2
        lanes[a].synchronize()  # the step that used this lane two steps ago has delivered its result
        m.mfet_embedding_bag_forward_host_async(eng.h, eng.shape, p_ids[k], p_off[k], p_w[k], nnz[k], w.table_ids,
                                                w.pooling, p_out[a], io[a], io_bytes, lanes[a].cuda_stream)
    for j in range(max(4, args.warmup)):
        e2e_step(j)
    # the K-step region five times (every region drained: all results in host memory); the median is reported
    e2e_regions = []
    for _ in range(5 if world == 1 else 1):
        barrier()
        t_e2e = time.perf_counter()
        for j in range(args.steps):
            e2e_step(j)
        barrier()  # both lanes drained: every result is in host memory
        e2e_regions.append(1e3 * (time.perf_counter() - t_e2e))
    e2e_ms = float(np.median(e2e_regions))
    t_load1 = time.time()
    clocks = sampler.stop(t_load0, t_load1) if sampler else None

    h2d = float(np.mean([nnz[k] * (8 + (4 if batches[k].weights is not None else 0)) + batches[k].offsets.size * 8
                         for k in range(n_rot)]))
    d2h = float(w.batch * w.out_dim * 4)

    # ---- hashing alone and dedup alone (not part of the timed step) ----------
    alone = None
    if world == 1:
        def timed(fn, reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            for _ in range(3):
                fn()
            a.record(stream)
            for _ in range(reps):
                fn()
            b.record(stream)
            torch.cuda.synchronize()
            return a.elapsed_time(b) / reps * 1e3  # us

        s0 = 0
        t0, f0 = int(w.table_ids[s0]), int(w.slot_feature[s0])
        n_all = nnz[0]
        rows_all = torch.empty(n_all, dtype=torch.int64, device="cuda")
        us_hash = timed(lambda: m.mfet_hash_ids(eng.h, t0, d_ids[0], n_all, rows_all, stream.cuda_stream), 100)
        n_big = 1 << 24
        big = torch.randint(0, 1 << 40, (n_big,), dtype=torch.int64, device="cuda")
        big_out = torch.empty_like(big)
        us_big = timed(lambda: m.mfet_hash_ids(eng.h, t0, big, n_big, big_out, stream.cuda_stream), 20)
        lo, hi = int(batches[0].offsets[f0 * B]), int(batches[0].offsets[(f0 + 1) * B])
        n_f = hi - lo
        if eng.ws is None:
            eng.set_workspace(n_f + 1024)
        m.mfet_hash_ids(eng.h, t0, d_ids[0][lo:hi], n_f, rows_all, stream.cuda_stream)
        uniq = torch.empty(n_f, dtype=torch.int64, device="cuda")
        inv = torch.empty(n_f, dtype=torch.int32, device="cuda")
        n_uniq_d = torch.zeros(1, dtype=torch.int64, device="cuda")
        us_dedup = timed(lambda: m.mfet_dedup_rows(eng.h, rows_all, n_f, uniq, inv, n_uniq_d, w.tables[t0].rows - 1,
                                                   stream.cuda_stream), 50)
        peak_bw, _ = measured_peaks()
        alone = {"hash": {"ids": n_all, "us": us_hash, "ids_large": n_big, "us_large": us_big,
                          "gbps_large": n_big * 16 / us_big / 1e3, "frac_large": n_big * 16 / us_big / 1e3 / peak_bw,
                          "bytes_per_id": 16},
                 "dedup": {"ids": n_f, "unique": int(n_uniq_d.item()), "us": us_dedup,
                           "table_rows": int(w.tables[t0].rows)}}
        del big, big_out, rows_all, uniq, inv

    ms, units = aggregate_over_ranks(local_ms, float(ids_done), dist if world > 1 else None)
    e2e_ms_all, _ = aggregate_over_ranks(e2e_ms, float(ids_done), dist if world > 1 else None)
    ctx.close()
    del d_ids, d_off, d_w, out, io, lanes, flush
    torch.cuda.empty_cache()

    peak, peak_kind = measured_peaks()
    achieved = alg / (kern_ms * 1e-3) / 1e9
    wl_key = "config%d" % config
    traffic, traffic_note = recorded_traffic(wl_key) if (args.rows_scale == 1.0 and args.alpha is None and not args.int4) \
        else (None, None)
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": traffic, "peak_kind": peak_kind + " copy bandwidth",
                "what": "algorithmic bytes per launch (a row counts once per lookup) / launch duration, against the "
                        "copy bandwidth; rows that repeat inside a batch are served by L1/L2, so DRAM moves less "
                        "than that (`traffic`, `dram_gbps`)",
                "kernel": "bag_kernel (all HBM-resident slots, one launch)",
                "algorithmic_bytes_per_launch": alg, "kernel_ms": kern_ms,
                "dram_gbps": (traffic / (kern_ms * 1e-3) / 1e9) if traffic else None, "traffic_note": traffic_note,
                "frac_of_8tbs": achieved / NOMINAL_HBM_GBS,
                "serialized": {"kernel_ms": kern_ms_serialized,
                               "achieved": alg / (kern_ms_serialized * 1e-3) / 1e9,
                               "frac": alg / (kern_ms_serialized * 1e-3) / 1e9 / peak,
                               "frac_of_8tbs": alg / (kern_ms_serialized * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
                               "note": "every launch waits for the one before it (no programmatic dependent launch): "
                                       "what a single request sees"}}
    return {
        "metric": METRIC, "value": units / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "config": config, "batch": w.batch, "ids_per_step": float(np.mean(nnz)),
                   "row_lookups_per_step": float(np.mean([row_lookups(w, b) for b in batches])),
                   "table_bytes": int(sum(t.rows * gi_row_bytes(t) for t in w.tables)),
                   "rows_scale": args.rows_scale, "cached_rows": cached_rows,
                   "l2": "no flush: tables are far larger than L2 and %d distinct batches rotate "
                         "(a cold-L2 series is under pooling_kernel.cold_l2)" % n_rot,
                   "launch_overlap": not args.no_overlap_launches,
                   "parallelism": "replicas x%d" % world},
        "step_us": stats(step_us) if len(step_us) > 1 else None,
        "serial_host_path_step_us": serial_step_us,
        "e2e": {"value": units / (e2e_ms_all * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                # the two directions of the link run at the same time; the busier one bounds the step
                "link_gbps": max(h2d, d2h) * args.steps / (e2e_ms_all * 1e-3) / 1e9,  # per GPU
                "link_direction": "d2h" if d2h >= h2d else "h2d",
                "regions_ms": [round(x, 3) for x in e2e_regions]},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "pooling_kernel": series,
        "roofline_host_path": host_path,
        "stages_alone": alone,
        "cpu_baseline": base,
        "clocks": clocks,
    }


def measure_series_only(args, config, rank, alpha=None, int4=False, n_batches=4):
    """A workload's pooling-kernel series without the step contract around it (for the `workloads`
    object of the default run)."""
    import torch
    ctx = Ctx(args, config, rank, alpha=alpha, int4=int4, n_batches=n_batches)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")
    try:
        s = pooling_series(ctx, args, flush)
        s["workload"] = ctx.w.name
        s["batch"] = ctx.w.batch
        s["table_bytes"] = int(sum(t.rows * gi_row_bytes(t) for t in ctx.w.tables))
        assert ctx.m.mfet_query_status(ctx.eng.h) == 0
        return s
    finally:
        ctx.close()
        del flush
        torch.cuda.empty_cache()


def measure_backward(args, config, rank, slot):
    """mfet_embedding_bag_backward for one slot of a workload: microseconds per call, lookups and
    distinct rows per second (paper, Section 4.3: the tables are fine-tuned)."""
    import torch
    ctx = Ctx(args, config, rank, n_batches=2)
    m, w, eng = ctx.m, ctx.w, ctx.eng
    try:
        f = int(w.slot_feature[slot])
        B = w.batch
        n_f = max(int(b.offsets[(f + 1) * B] - b.offsets[f * B]) for b in ctx.batches)
        eng.set_workspace(n_f + 4096)
        dim = w.tables[int(w.table_ids[slot])].dim
        grad_out = torch.randn(w.batch, w.out_dim, dtype=torch.float32, device="cuda")
        g_rows = torch.empty(n_f, dtype=torch.int64, device="cuda")
        g_vals = torch.empty(n_f * dim, dtype=torch.float32, device="cuda")
        n_rows = torch.zeros(1, dtype=torch.int64, device="cuda")

        def call(j):
            k = j % ctx.n_rot
            m.mfet_embedding_bag_backward(eng.h, eng.shape, ctx.d_ids[k], ctx.d_off[k], ctx.d_w[k], w.table_ids, w.pooling,
                                          grad_out, slot, g_rows, g_vals, n_rows, ctx.stream.cuda_stream)
        for j in range(3):
            call(j)
        us = region_series(ctx, call, min(args.steps, 50), 7)
        med = float(np.median(us)) * 1e-6
        lookups = float(np.mean([int(b.offsets[(f + 1) * B] - b.offsets[f * B]) for b in ctx.batches]))
        return {"workload": w.name, "slot": slot, "dim": dim, "lookups_per_call": lookups,
                "distinct_rows_last_call": int(n_rows.item()), "us_per_call": stats(us),
                "lookups_per_s": lookups / med, "distinct_rows_per_s": int(n_rows.item()) / med,
                "note": "hash + sort by row (the dedup machinery) + one pass that sums coef * grad_out per distinct row"}
    finally:
        ctx.close()
        torch.cuda.empty_cache()


def run_gpu(args):
    import torch
    import torch.distributed as dist

    from paper_2508_05700_b200 import build as b_
    rank, local_rank, world = dist_env()
    if world > 1:
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    else:
        torch.cuda.set_device(0)
    if rank == 0:
        b_.build()
    if world > 1:
        dist.barrier()
    config = args.config or DEFAULT_CONFIG
    line = measure(args, config, rank, world, dist, rank == 0 and world == 1 and not args.no_cpu_baseline,
                   sampler_gpu=torch.cuda.current_device() if rank == 0 else None)
    # Next to the headline: every workload's pooling kernel (HBM-resident slots), and the hybrid workload
    # as a whole. One process only: the hybrid workload needs 128 GB of pinned host RAM.
    if args.config is None and world == 1 and not args.headline_only:
        workloads = {"c%d" % config: line["pooling_kernel"]}
        plain = argparse.Namespace(**vars(args))
        plain.alpha, plain.int4, plain.device_slots_only = None, False, False

        def guarded(fn, *a, **k):
            try:
                return fn(*a, **k)
            except Exception as exc:  # the headline number stands on its own
                return {"error": "%s: %s" % (type(exc).__name__, exc)}
        for c in (1, 2, 4):
            workloads["c%d" % c] = guarded(measure_series_only, plain, c, rank)
        for c in (2, 4):  # no repeated rows: the pure random-gather case
            if "error" not in workloads["c%d" % c]:
                workloads["c%d" % c]["uniform_ids"] = guarded(measure_series_only, plain, c, rank, alpha=0.0)
        workloads["c2"]["int4_tables"] = guarded(measure_series_only, plain, 2, rank, int4=True) \
            if "error" not in workloads["c2"] else None
        workloads["c%d" % config]["backward_slot_2"] = guarded(measure_backward, plain, config, rank, 2)
        if not args.no_hybrid:
            hyb = guarded(measure, plain, 5, rank, world, dist, False, None)
            if "error" not in hyb:
                line["hybrid"] = {k: hyb[k] for k in ("value", "unit", "ms_per_step", "step_us", "serial_host_path_step_us",
                                                      "config", "e2e", "gpu_launches", "roofline", "roofline_host_path",
                                                      "stages_alone")}
                workloads["c5"] = hyb["pooling_kernel"]
                workloads["c5"]["whole_step_us"] = hyb["step_us"]
            else:
                line["hybrid"] = hyb
        line["workloads"] = workloads
    if world > 1:
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", type=int, default=None, choices=[1, 2, 3, 4, 5],
                    help="one workload only; default: %d under the step contract, then all five workloads" % DEFAULT_CONFIG)
    ap.add_argument("--no-hybrid", action="store_true", help="skip the hybrid workload after the default one")
    ap.add_argument("--headline-only", action="store_true", help="default workload only, no `workloads` object")
    ap.add_argument("--impl", default="mfet", choices=["mfet", "reference"])
    ap.add_argument("--rows-scale", type=float, default=1.0, help="shrink table rows (reported in config)")
    ap.add_argument("--alpha", type=float, default=None, help="override the Zipf exponent of every feature (0 = uniform IDs)")
    ap.add_argument("--int4", action="store_true", help="store the workload's tables as INT4 rows")
    ap.add_argument("--batches", type=int, default=8, help="distinct batches rotated through")
    ap.add_argument("--load-seconds", type=float, default=1.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-overlap-launches", action="store_true",
                    help="every pooling kernel starts only when the kernel before it on the stream has finished")
    ap.add_argument("--serial-host-path", action="store_true",
                    help="hybrid workload: no early fetch of the next batch's host-table rows")
    ap.add_argument("--device-slots-only", action="store_true",
                    help="drop the host-table slots of the workload (times the HBM-resident part of workload 5 alone)")
    ap.add_argument("--tile", type=int, default=0, help="samples per block of the pooling kernel (0 = library default)")
    ap.add_argument("--stage-ids", type=int, default=0, help="IDs staged per pass of the pooling kernel (0 = library default)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        return run_reference(args)
    return run_gpu(args)


if __name__ == "__main__":
    sys.exit(main())
