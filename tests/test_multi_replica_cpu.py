"""The N > 1 path of the benchmark is N independent replicas (the MoE step has no exchange
step): the only cross-rank logic is the barrier and the max-over-ranks of the timings.  Covered
here with two gloo ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    times = [10.0 + 5.0 * rank, 3.0 - rank]          # rank 1 is slower on the first, faster on the second
    dist.barrier()
    got = bench.max_over_ranks(times, "cpu")
    q.put((rank, got, bench.aggregate_tokens_per_s(world, 16, 100, got[0])))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_aggregate_with_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, agg in res:
        assert got == [15.0, 3.0]                        # the slowest replica decides, on every rank
        assert abs(agg - 2 * 16 * 100 / 0.015) < 1e-6     # whole-job tokens/s of two replicas


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], "cpu") == [1.5, 2.5]
