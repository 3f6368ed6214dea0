"""The multi-process path of the benchmark (replicas only: a max-reduction of timings), on CPU with gloo."""
import os

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1701_06538_b200 import replicas


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, ms_e2e = replicas.max_over_ranks([10.0 + 5.0 * rank, 30.0 - 7.0 * rank])
    dist.barrier()
    out[rank] = (ms, ms_e2e, replicas.job_throughput(1000, 4, ms, world))
    dist.destroy_process_group()


def test_timing_is_the_max_over_ranks_and_throughput_is_whole_job():
    world = 2
    with mp.get_context("spawn").Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, 29517 + os.getpid() % 200, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]                      # every rank ends with the same numbers
    ms, ms_e2e, tput = res[0]
    assert ms == 15.0 and ms_e2e == 30.0         # slowest rank per quantity
    assert tput == world * 1000 * 4 / 0.015      # all replicas' tokens over that time


def test_single_process_is_identity():
    assert replicas.max_over_ranks([3.5, 1.0]) == [3.5, 1.0]
    assert replicas.job_throughput(100, 2, 50.0, 1) == 4000.0
