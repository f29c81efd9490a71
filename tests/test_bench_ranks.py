"""The multi-GPU path of bench.py is replicas only: no collective on the data path, one reduction of the timings and
counts at the end.  Two CPU ranks over gloo check that reduction: the slowest rank's time, the sum of tokens and
launches."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    # rank k: k-dependent step time and token count
    got = bench.aggregate_ranks(dist, torch.device("cpu"), 100.0 + 10 * rank, 120.0 - 5 * rank, 2048 * (rank + 1),
                                1024 * (rank + 1), 32768 + rank)
    dist.barrier()
    dist.destroy_process_group()
    out[rank] = got


def test_two_ranks_take_the_slowest_time_and_sum_the_tokens():
    world, port = 2, 29731
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        results = [out[r] for r in range(world)]
    want = (110.0, 120.0, 2048 * 3, 1024 * 3, 2 * 32768 + 1)
    assert results[0] == want and results[1] == want


def test_one_rank_is_left_alone():
    import bench
    assert bench.aggregate_ranks(None, None, 1.0, 2.0, 3, 4, 5) == (1.0, 2.0, 3, 4, 5)
