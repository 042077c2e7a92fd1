"""The N > 1 arm of the benchmark without GPUs: two gloo ranks on CPU.

Prompts are independent, so ranks share nothing on the data path; what has to
be right is that every rank draws different prompts and that the whole-job
figure is (sum of units) / (slowest rank's time)."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    import bench
    from paper_2503_05330_b200 import synth
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = synth.WORKLOADS[1]
    tokens, _ = synth.make_streams(w, bench.rank_seed(w, rank))
    times, units = bench.whole_job([10.0 + rank, 5.0 - rank], [100.0 * (rank + 1), 7.0], "cpu")
    out[rank] = (int(tokens.sum()), times, units)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_draw_different_prompts_and_reduce_max_time_sum_units():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] != res[1][0]                       # different streams per rank
    for r in range(world):
        assert res[r][1] == [11.0, 5.0]                 # MAX over ranks
        assert res[r][2] == [300.0, 14.0]               # SUM over ranks


def test_single_process_passthrough():
    import bench
    assert bench.whole_job([3.0], [4.0], "cpu") == ([3.0], [4.0])
