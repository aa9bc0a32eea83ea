"""The N > 1 plumbing of bench.py on CPU: two gloo ranks, max-over-ranks timing, whole-job throughput."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    ms = bench.max_over_ranks(local_ms, world, torch.device("cpu"))
    dist.barrier()
    q.put((rank, ms, bench.job_tflops(world, 2.0e12, 4, ms)))
    dist.destroy_process_group()


def test_two_ranks_agree_on_the_slowest_time_and_aggregate_value():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [15.0, 15.0]
    # two replicas x 2 TFLOP x 4 steps in 15 ms
    assert abs(res[0][2] - 2 * 2.0 * 4 / 0.015) < 1e-6 and res[0][2] == res[1][2]


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert bench.job_tflops(1, 1e12, 10, 1000.0) == 10.0
