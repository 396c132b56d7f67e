"""The multi-GPU mode is N independent replicas (sequences never interact, weights are
read-only), so the only cross-rank logic is the timing reduction of the benchmark.  It is
exercised here with two CPU processes over gloo."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    import torch.distributed as dist

    sys.path.insert(0, ROOT)
    import bench

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, device="cpu")     # ranks take 10 ms and 15 ms
    dist.barrier()
    q.put((rank, ms, bench.aggregate_steps_per_s(world, 30, ms)))
    dist.destroy_process_group()


def test_max_over_ranks_and_aggregate_value():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 500
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value in res:
        assert ms == 15.0                       # the slowest rank decides
        assert abs(value - 2 * 30 / 0.015) < 1e-9


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.max_over_ranks(3.5, device="cpu") == 3.5
    assert bench.aggregate_steps_per_s(1, 100, 50.0) == 2000.0
