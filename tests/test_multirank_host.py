"""The N > 1 path of the benchmark on CPU: two gloo ranks, no data-path collective - each rank draws its own row
shard, the elapsed times are reduced with MAX and the job throughput is the sum of the ranks' work over that time."""
import os

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2604_18117_b200 import dist_util as D
from paper_2604_18117_b200 import inputs as I


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), WORLD_SIZE=str(world), RANK=str(rank),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w, r, l = D.env_ranks()
        assert (w, r, l) == (world, rank, rank)
        wl = I.workload(0)
        X, _, _ = I.layer_inputs(wl, wl.layers[0], seed=D.shard_seed(0, rank), M=32)
        my_ms = 10.0 + 5.0 * rank                                   # rank 1 is the slow one
        dist.barrier()
        slowest = D.max_over_ranks(my_ms, world)
        out[rank] = (float(np.abs(X.astype(np.float32)).sum()), slowest,
                     D.job_throughput(1000.0, 4, slowest, world))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_rows_and_take_the_slowest_time():
    world, port = 2, 29000 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        r0, r1 = out[0], out[1]
    assert r0[0] != r1[0]                          # different rows on the two ranks
    assert r0[1] == r1[1] == 15.0                  # both see the slowest rank's time
    assert abs(r0[2] - 2 * 1000.0 * 4 / 15e-3) < 1e-6 and r0[2] == r1[2]


def test_single_rank_needs_no_process_group():
    assert D.max_over_ranks(3.5, 1) == 3.5
    assert D.job_throughput(10.0, 2, 1000.0, 1) == 20.0
