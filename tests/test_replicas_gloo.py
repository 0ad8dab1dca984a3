"""The multi-GPU path is "replicas only": ranks decode independent batches and only the timing is reduced.  This runs
that reduction (bench.reduce_replicas) as two gloo ranks on the CPU."""
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
    ms, tok = bench.reduce_replicas([100.0 + 10 * rank, 200.0 - 5 * rank], 256 * (rank + 1), world)
    dist.barrier()
    dist.destroy_process_group()
    q.put((rank, ms, tok))


def test_two_rank_reduction_is_max_time_and_summed_tokens():
    world, port = 2, 29731
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    for rank, ms, tok in res:
        assert ms == [110.0, 200.0]          # the slowest rank of each timed region
        assert tok == 256 + 512              # whole-job tokens
    # value = whole-job tokens / max time, as bench.py prints it
    assert abs((256 + 512) / (110.0 * 1e-3) - 6981.818) < 1e-2


def test_single_rank_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_replicas([3.5, 7.0], 42, 1) == ([3.5, 7.0], 42.0)
