"""The N > 1 path of bench.py on CPU: two gloo ranks, barrier, max-over-ranks time, summed examples."""
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
    # rank r pretends its timed region took (10 + 5r) ms for 1000*(r+1) examples
    ms, ex = bench.reduce_over_ranks([10.0 + 5.0 * rank, 7.0 - rank], 1000 * (rank + 1), device="cpu")
    q.put((rank, ms, ex))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_take_max_time_and_sum_examples():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, ex in got:
        assert ms == [15.0, 7.0] and ex == 3000     # slowest rank's time per region, examples of all ranks


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_over_ranks([3.0, 4.0], 17, device="cpu") == ([3.0, 4.0], 17)
