"""world_size-2 gloo check of the benchmark's rank plumbing (CPU only)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2204_06514_b200 import dist_util


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert dist_util.env_rank() == (rank, world, rank)
    dist.barrier()
    ms = dist_util.max_over_ranks(10.0 + 5.0 * rank)          # rank 1 is the slow replica
    out[rank] = (ms, dist_util.whole_job_rate(8192, world, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_rate_world2():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
        assert out[0] == out[1]
        ms, rate = out[0]
        assert ms == 15.0
        assert abs(rate - 2 * 8192 / 15e-3) < 1e-6


def test_single_process_is_identity():
    assert dist_util.max_over_ranks(3.5) == 3.5
    assert dist_util.whole_job_rate(100, 1, 50.0) == 2000.0
