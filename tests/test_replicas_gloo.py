"""World-size-2 gloo test of the multi-GPU plumbing (timing reduction and head partition)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2509_10406_b200 import replicas


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = 10.0 if rank == 0 else 25.0
    out[rank] = (replicas.max_over_ranks(ms), replicas.job_throughput(1000.0, ms), replicas.head_range(5, rank, world))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_timing_and_partition():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 25.0
    assert abs(res[0][1] - 2 * 1000.0 / 0.025) < 1e-6
    assert res[0][2] == (0, 3) and res[1][2] == (3, 5)


def test_single_process_is_identity():
    assert replicas.max_over_ranks(7.0) == 7.0
    assert replicas.head_range(16, 0, 1) == (0, 16)
