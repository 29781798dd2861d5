"""bench.py's multi-rank bookkeeping (replicas only: max time over ranks, units summed),
run as two gloo ranks on CPU."""
import os
import socket
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist

    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env() == (rank, rank, world)
    ms, units = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 1000.0 * (rank + 1), dist)
    dist.barrier()
    dist.destroy_process_group()
    q.put((rank, ms, units))


def test_two_rank_aggregation_gloo():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == [(0, 15.0, 3000.0), (1, 15.0, 3000.0)]


def test_single_process_aggregation_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_over_ranks(3.5, 7.0, None) == (3.5, 7.0)
    b = bench.algorithmic_bytes
    from paper_2508_05700_b200 import inputs as gi
    w = gi.make_workload(1)
    batch = gi.make_batch(w, 0)
    nnz = int(batch.offsets[-1])
    assert b(w, batch) == nnz * 128 + nnz * 8 + (512 + 1) * 8 + 512 * 32 * 4


def test_bench_bookkeeping_helpers(tmp_path, monkeypatch):
    """Percentiles, row-lookup counts and the reading of the committed DRAM-traffic file (keyed by workload
    and by a fingerprint of the kernel sources: a stale figure must come back as None)."""
    sys.path.insert(0, ROOT)
    import bench
    from paper_2508_05700_b200 import inputs as gi
    s = bench.stats([1.0, 2.0, 3.0, 4.0, 100.0])
    assert s["median"] == 3.0 and s["n"] == 5 and s["p10"] < s["median"] < s["p90"]
    w = gi.make_workload(3, rows_scale=1e-4, batch_scale=1 / 64)
    b = gi.make_batch(w, 0)
    nnz = int(b.offsets[-1])
    assert bench.row_lookups(w, b) == 3 * nnz                      # three facet slots read every feature's IDs
    assert bench.row_lookups(w, b, [0]) == int(b.offsets[w.batch] - b.offsets[0])
    t = w.tables
    rows_bytes = sum(int(b.offsets[(f + 1) * w.batch] - b.offsets[f * w.batch]) * (t[3 * f].dim + t[3 * f + 1].dim + t[3 * f + 2].dim) * 2
                     for f in range(w.n_features))
    assert bench.algorithmic_bytes(w, b) == rows_bytes + nnz * 12 + (w.n_features * w.batch + 1) * 8 + w.batch * w.out_dim * 4
    fp = bench.kernel_fingerprint()
    prof = tmp_path / "profiles"
    prof.mkdir()
    (prof / "bag_kernel_dram_traffic.txt").write_text("# comment\nconfig3 %s 12345 scaled capture: x\nconfig2 deadbeefdeadbeef 777 old\n" % fp)
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    monkeypatch.setattr(bench, "kernel_fingerprint", lambda: fp)
    assert bench.recorded_traffic("config3") == (12345.0, "scaled capture: x")
    assert bench.recorded_traffic("config2") == (None, None)       # captured for other kernel sources
    assert bench.recorded_traffic("config9") == (None, None)
