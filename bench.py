#!/usr/bin/env python
"""Benchmark of the embedding-table lookup path: pooled IDs per second.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference]

One step = one pass of the whole lookup path (hash -> gather -> pool -> concat, plus
dedup -> cache probe -> host fetch for a host-resident table) over one synthetic batch.
`value` is measured with the batch resident in HBM; `e2e` goes through the C-ABI call
that takes HOST buffers (copies in and out inside the timed region). N > 1 runs N
independent replicas (the path has no exchange step), one process per GPU.
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
KERNEL_SOURCES = ["paper_2508_05700_b200/csrc/bag.cu", "paper_2508_05700_b200/csrc/common.cuh"]


# ------------------------------------------------------------------ helpers --

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


def gi_row_bytes(t: gi.TableSpec) -> int:
    if t.dtype == gi.INT4:
        return (t.dim // 2 + 4 + 15) // 16 * 16
    return t.dim * (4 if t.dtype == gi.F32 else 2)


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
    """DRAM bytes per launch of the pooling kernel from the committed ncu summary; None when
    there is none for this workload or the kernel sources changed since it was taken."""
    path = os.path.join(ROOT, "profiles", "bag_kernel_dram_traffic.txt")
    if not os.path.exists(path):
        return None
    fp = kernel_fingerprint()
    with open(path) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            key, fingerprint, nbytes = line.split()[:3]
            if key == workload_key and fingerprint == fp:
                return float(nbytes)
    return None


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

def oracle_tables(w: gi.Workload):
    import oracle as orc
    return [orc.Table(rows=s.rows, dim=s.dim, dtype=s.dtype, hash_seed=s.hash_seed, value_key=s.value_key)
            for s in w.tables]


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


def cpu_baseline(w, batches, target_seconds=12.0):
    """The oracle on about `target_seconds` of host work: whole batches of the rotation when one
    batch is quick, else the first samples of batch 0."""
    import oracle as orc
    orc.build()
    tabs = oracle_tables(w)
    threads = os.cpu_count() or 1
    b = batches[0]
    probe = list(range(min(w.batch, 4 * threads)))
    oracle_run_samples(w, b, tabs, probe, threads)  # first touch: library load, thread start
    dt = max(oracle_run_samples(w, b, tabs, probe, threads), 1e-4)
    per_sample = dt / len(probe)
    if per_sample * w.batch > target_seconds:
        n = int(max(threads, target_seconds / per_sample))
        samples = list(range(n))
        total = oracle_run_samples(w, b, tabs, samples, threads)
        n_ids = ids_in_samples(w, b, samples)
        what = "samples 0..%d of batch 0" % (n - 1)
    else:
        samples = list(range(w.batch))
        total = oracle_run_samples(w, b, tabs, samples, threads)
        n_ids = int(b.offsets[-1])
        reps = 1
        while total < target_seconds and reps < 256:
            bb = batches[reps % len(batches)]
            total += oracle_run_samples(w, bb, tabs, samples, threads)
            n_ids += int(bb.offsets[-1])
            reps += 1
        what = "%d whole batches (rotation of %d)" % (reps, len(batches))
    return {"value": n_ids / total, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": "%s (%d IDs) of %s, procedural table values, %.1f s" % (what, n_ids, w.name, total)}


def run_reference(args):
    """--impl reference: the CPU oracle timed on this machine's host cores, each step a bounded
    sample of the workload."""
    rank, _, world = dist_env()
    if rank != 0:
        return 0
    import oracle as orc
    orc.build()
    args.config = args.config or DEFAULT_CONFIG
    w = gi.make_workload(args.config)
    b = gi.make_batch(w, 0)
    tabs = oracle_tables(w)
    threads = os.cpu_count() or 1
    probe = list(range(min(w.batch, threads)))
    dt = max(oracle_run_samples(w, b, tabs, probe, threads), 1e-4)
    budget = 90.0 / max(1, args.steps + args.warmup)
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
    sample = "%d samples of batch 0 per step (%d IDs per step on average), procedural table values" % (
        n, ids_done // max(1, args.steps))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / max(1, args.steps),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "config": args.config},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------ GPU arm --

def host_rows_that_fit(w: gi.Workload):
    """Rows of the host-resident table that this box can pin (it needs rows*row_bytes of
    host RAM next to everything else); the full row count when memory allows."""
    try:
        with open("/proc/meminfo") as fh:
            avail = {l.split(":")[0]: int(l.split()[1]) * 1024 for l in fh}["MemAvailable"]
    except (OSError, KeyError):
        return None
    out = {}
    for i, t in enumerate(w.tables):
        if t.location == gi.LOC_HOST:
            fit = int(0.70 * avail) // gi_row_bytes(t)
            out[i] = min(t.rows, fit)
    return out


def measure(args, config, rank, world, dist, with_cpu_baseline, sampler_gpu=None):
    """One workload: set-up, warm-up, exactly K timed steps (device-resident inputs), the
    pooling kernel alone, the end-to-end series through host buffers. Returns the JSON fields."""
    import torch

    from paper_2508_05700_b200 import mfet as m
    from paper_2508_05700_b200.runtime import LookupEngine

    w = gi.make_workload(config, rows_scale=args.rows_scale)
    if args.alpha is not None:  # e.g. 0 = uniform IDs: no row repeats, the pure random-gather case
        w.alpha = np.full(w.n_features, float(args.alpha))
        w.name += ", Zipf alpha overridden to %g" % args.alpha
    if args.device_slots_only:  # the HBM-resident part of a hybrid workload, as a workload of its own
        keep = [s for s in range(w.n_slots) if w.tables[int(w.table_ids[s])].location == gi.LOC_DEVICE]
        for t in w.tables:
            if t.location != gi.LOC_DEVICE:
                t.rows = 1024
        w.slot_feature, w.table_ids, w.pooling = w.slot_feature[keep], w.table_ids[keep], w.pooling[keep]
        w.name += ", device-table slots only"
    scaled_host = False
    fits = host_rows_that_fit(w)
    if fits:
        for i, rows in fits.items():
            if rows < w.tables[i].rows:
                w.tables[i].rows = rows
                scaled_host = True
    n_rot = args.batches
    batches = [gi.make_batch(w, rank * 1000 + j) for j in range(n_rot)]
    base = cpu_baseline(w, batches) if with_cpu_baseline else None

    dev = torch.cuda.current_device()
    eng = LookupEngine(w, device=dev)
    if not args.no_overlap_launches:
        # the batches are resident before the timed region: a step's kernel may hash its IDs while the
        # step before it finishes (it waits for that kernel before it writes the output)
        m.mfet_set_option(eng.h, m.OPT_OVERLAP_LAUNCHES, 1)
    if args.tile:
        m.mfet_set_option(eng.h, m.OPT_TILE, args.tile)
    if args.stage_ids:
        m.mfet_set_option(eng.h, m.OPT_STAGE_IDS, args.stage_ids)
    stream = torch.cuda.current_stream()
    host_tabs = [] if args.device_slots_only else eng.host_table_ids()
    cached_rows = 0
    B = w.batch
    host_feats = sorted({int(w.slot_feature[s]) for s in range(w.n_slots) if int(w.table_ids[s]) in host_tabs})
    if host_tabs:
        worst = max(int(b.offsets[(f + 1) * B] - b.offsets[f * B]) for b in batches for f in host_feats)
        eng.set_workspace(int(worst * 1.25) + 4096)
        for t in host_tabs:
            f = int(w.slot_feature[list(w.table_ids).index(t)])
            cached_rows = eng.build_hot_cache(t, f, int(w.tables[t].rows * w.cache_fraction))
        m.mfet_set_option(eng.h, m.OPT_PROFILE, 1)

    d_ids = [torch.from_numpy(b.ids.view(np.int64)).cuda() for b in batches]
    d_off = [torch.from_numpy(b.offsets).cuda() for b in batches]
    d_w = [None if b.weights is None else torch.from_numpy(b.weights).cuda() for b in batches]
    out = torch.empty(w.batch, w.out_dim, dtype=torch.float32, device="cuda")
    nnz = [int(b.offsets[-1]) for b in batches]

    # Hybrid workload: the fetch of the next batch's host-table rows starts before the current
    # batch is pooled (the paper's early embedding fetch, Section 3.4): the library's dedup of
    # batch j+1 and the PCIe reads of its rows run while batch j is pooled. Results are
    # bit-identical to the serial path (tests). `seq` numbers the steps across warm-up, load
    # phase and timed region, because every step announces its successor.
    n_host_slots = sum(1 for s in range(w.n_slots) if int(w.table_ids[s]) in host_tabs)
    pipelined = bool(host_tabs) and n_host_slots == 1 and not args.serial_host_path
    seq = [0]
    if pipelined:
        pre_shape, _keep_pre = m.make_shape(w.batch, w.n_features, w.slot_feature)
        pre_shape.flags |= m.BATCH_PREFETCHED
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

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(dev) if sampler_gpu is not None else None
    if sampler:
        sampler.start()
    # warm-up: W steps, then keep the GPU under the same load for about a second so that the
    # clock samples around the timed region describe the loaded state
    for j in range(args.warmup):
        step(j)
    torch.cuda.synchronize()
    t_load0 = time.time()
    j = args.warmup
    while time.time() - t_load0 < args.load_seconds:
        for _ in range(50):
            step(j)
            j += 1
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
    if pipelined:  # pool the batch that the last step announced, then go on with the serial path
        k = seq[0] % n_rot
        m.mfet_embedding_bag_forward(eng.h, pre_shape, d_ids[k], d_off[k], d_w[k], w.table_ids, w.pooling, out,
                                     stream.cuda_stream)
        torch.cuda.synchronize()
        pipelined = False
    assert m.mfet_query_status(eng.h) == 0, "device error bits set during the timed region"

    # ---- the pooling kernel alone: all HBM-resident slots, one launch per step ----
    # timed as in the timed region (launches may overlap by their start-up phase) and with every launch
    # waiting for the one before it ("serialized": the duration of a launch by itself)
    dev_slots = [s for s in range(w.n_slots) if w.tables[int(w.table_ids[s])].location == gi.LOC_DEVICE]
    all_dev = len(dev_slots) == w.n_slots
    if not all_dev:
        sub_shape, keep = m.make_shape(w.batch, w.n_features, w.slot_feature[dev_slots])
        sub_out = torch.empty(w.batch, sum(w.tables[int(w.table_ids[s])].dim for s in dev_slots), device="cuda")

    def kernel_alone_ms():
        k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for rep in range(2):
            k0.record(stream)
            for j in range(args.steps):
                k = j % n_rot
                if all_dev:
                    eng.forward(d_ids[k], d_off[k], d_w[k], out)
                else:
                    eng.forward(d_ids[k], d_off[k], d_w[k], sub_out, table_ids=w.table_ids[dev_slots],
                                pooling=w.pooling[dev_slots], shape=sub_shape)
            k1.record(stream)
            torch.cuda.synchronize()
        return k0.elapsed_time(k1) / args.steps

    kern_ms = local_ms / args.steps if all_dev else kernel_alone_ms()
    kern_ms_serialized = kern_ms
    if not args.no_overlap_launches:
        m.mfet_set_option(eng.h, m.OPT_OVERLAP_LAUNCHES, 0)
        kern_ms_serialized = kernel_alone_ms()
        m.mfet_set_option(eng.h, m.OPT_OVERLAP_LAUNCHES, 1)
    alg = float(np.mean([algorithmic_bytes(w, batches[j % n_rot], dev_slots) for j in range(min(args.steps, n_rot))]))

    # ---- host-table path alone (PCIe roofline): stage times from the library's events ----
    host_path = None
    if host_tabs:
        peak_h2d = None
        t0 = host_tabs[0]
        nbytes = min(1 << 30, w.tables[t0].rows * gi_row_bytes(w.tables[t0]))
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
        n_miss = m.mfet_host_path_counts(eng.h)[1]  # unique, uncached rows of the last batch
        row_b = gi_row_bytes(w.tables[t0])
        fetched = n_miss * row_b
        host_path = {"bound": "pcie", "kernel": "fetch_rows_kernel (zero-copy reads of the missed rows)",
                     "unique_missed_rows_per_step": n_miss, "row_bytes": row_b,
                     "achieved": fetched / (stages[1] * 1e-3) / 1e9 if stages[1] > 0 else None,
                     "peak": peak_h2d, "unit": "GB/s",
                     "frac": (fetched / (stages[1] * 1e-3) / 1e9 / peak_h2d) if stages[1] > 0 and peak_h2d else None,
                     "peak_kind": "measured DMA copy of 1 GiB, pinned host to device, in this run",
                     "stage_ms": {"hash_dedup_probe": float(stages[0]), "fetch": float(stages[1]), "pool": float(stages[2])},
                     "host_rows": int(w.tables[t0].rows), "scaled_to_fit_host_ram": scaled_host}

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
    barrier()
    t_e2e = time.perf_counter()
    for j in range(args.steps):
        e2e_step(j)
    barrier()  # both lanes drained: every result is in host memory
    e2e_ms = 1e3 * (time.perf_counter() - t_e2e)
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
        n_uniq = torch.zeros(1, dtype=torch.int64, device="cuda")
        us_dedup = timed(lambda: m.mfet_dedup_rows(eng.h, rows_all, n_f, uniq, inv, n_uniq, w.tables[t0].rows - 1,
                                                   stream.cuda_stream), 50)
        peak_bw, _ = measured_peaks()
        alone = {"hash": {"ids": n_all, "us": us_hash, "ids_large": n_big, "us_large": us_big,
                          "gbps_large": n_big * 16 / us_big / 1e3, "frac_large": n_big * 16 / us_big / 1e3 / peak_bw,
                          "bytes_per_id": 16},
                 "dedup": {"ids": n_f, "unique": int(n_uniq.item()), "us": us_dedup,
                           "table_rows": int(w.tables[t0].rows)}}
        del big, big_out, rows_all, uniq, inv

    ms, units = aggregate_over_ranks(local_ms, float(ids_done), dist if world > 1 else None)
    e2e_ms_all, _ = aggregate_over_ranks(e2e_ms, float(ids_done), dist if world > 1 else None)
    eng.close()
    del eng, d_ids, d_off, d_w, out, io, lanes
    torch.cuda.empty_cache()

    peak, peak_kind = measured_peaks()
    achieved = alg / (kern_ms * 1e-3) / 1e9
    wl_key = "config%d" % config + ("" if args.rows_scale == 1.0 else "_rows%g" % args.rows_scale)
    return {
        "metric": METRIC, "value": units / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "config": config, "batch": w.batch, "ids_per_step": float(np.mean(nnz)),
                   "row_lookups_per_step": float(np.mean([sum(int(b.offsets[(int(w.slot_feature[s]) + 1) * w.batch] -
                                                                   b.offsets[int(w.slot_feature[s]) * w.batch])
                                                               for s in range(w.n_slots)) for b in batches])),
                   "table_bytes": int(sum(t.rows * gi_row_bytes(t) for t in w.tables)),
                   "rows_scale": args.rows_scale, "cached_rows": cached_rows,
                   "l2": "no flush: tables are far larger than L2 and %d distinct batches rotate" % n_rot,
                   "launch_overlap": not args.no_overlap_launches,
                   "parallelism": "replicas x%d" % world},
        "e2e": {"value": units / (e2e_ms_all * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                # the two directions of the link run at the same time; the busier one bounds the step
                "link_gbps": max(h2d, d2h) * args.steps / (e2e_ms_all * 1e-3) / 1e9,  # per GPU
                "link_direction": "d2h" if d2h >= h2d else "h2d"},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": recorded_traffic(wl_key), "peak_kind": peak_kind + " copy bandwidth",
                     "kernel": "bag_kernel (all HBM-resident slots, one launch)",
                     "algorithmic_bytes_per_launch": alg, "kernel_ms": kern_ms,
                     "serialized": {"kernel_ms": kern_ms_serialized,
                                    "achieved": alg / (kern_ms_serialized * 1e-3) / 1e9,
                                    "frac": alg / (kern_ms_serialized * 1e-3) / 1e9 / peak,
                                    "note": "every launch waits for the one before it (no programmatic dependent launch)"}},
        "roofline_host_path": host_path,
        "stages_alone": alone,
        "cpu_baseline": base,
        "clocks": clocks,
    }


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
    # the hybrid workload (largest table in host memory) next to the headline one: it needs
    # 128 GB of pinned host RAM per process, so it runs only as a single process
    if args.config is None and world == 1 and not args.no_hybrid:
        try:
            hyb = measure(args, 5, rank, world, dist, False, sampler_gpu=None)
            line["hybrid"] = {k: hyb[k] for k in ("value", "unit", "ms_per_step", "config", "e2e", "gpu_launches",
                                                  "roofline", "roofline_host_path", "stages_alone")}
        except Exception as exc:  # the headline number stands on its own
            line["hybrid"] = {"error": "%s: %s" % (type(exc).__name__, exc)}
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
                    help="workload; default: %d, followed by the hybrid workload 5 on one GPU" % DEFAULT_CONFIG)
    ap.add_argument("--no-hybrid", action="store_true", help="skip the hybrid workload after the default one")
    ap.add_argument("--impl", default="mfet", choices=["mfet", "reference"])
    ap.add_argument("--rows-scale", type=float, default=1.0, help="shrink table rows (reported in config)")
    ap.add_argument("--alpha", type=float, default=None, help="override the Zipf exponent of every feature (0 = uniform IDs)")
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
