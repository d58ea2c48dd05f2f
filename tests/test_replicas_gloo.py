"""The N > 1 path of the benchmark on CPU: two gloo ranks, max-over-ranks timing, whole-job rate."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2405_14917_b200 import replicas
    ms = 10.0 * (rank + 1)                          # rank 1 is the slow one
    out[rank] = (replicas.max_over_ranks(ms), replicas.whole_job_rate(1000.0, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_sum_of_the_work():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        ms_max, rate = res[rank]
        assert ms_max == 20.0
        assert abs(rate - 2 * 1000.0 / 20e-3) < 1e-6


def test_single_process_is_the_identity():
    from paper_2405_14917_b200 import replicas
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.whole_job_rate(7.0, 1000.0) == 7.0
