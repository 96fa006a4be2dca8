"""The N>1 bookkeeping (max-over-ranks time, whole-job rate) on two gloo ranks."""
import os
import socket

import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_13031_b200 import replicas


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    seconds = 2.0 if rank == 0 else 3.0           # rank 1 is the slow one
    replicas.barrier()
    out[rank] = (replicas.max_over_ranks(seconds), replicas.whole_job_rate(6.0, seconds))
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_summed_work():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    out = mp.Manager().dict()
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    for rank in (0, 1):
        slowest, rate = out[rank]
        assert slowest == 3.0
        assert rate == 2 * 6.0 / 3.0


def test_single_process_is_identity():
    assert replicas.max_over_ranks(1.5) == 1.5
    assert replicas.whole_job_rate(4.0, 2.0) == 2.0
