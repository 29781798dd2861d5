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
