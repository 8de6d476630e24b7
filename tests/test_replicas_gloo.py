"""The N > 1 path of the benchmark is "replicas only": the ranks exchange nothing but their step times.
Two gloo ranks on the CPU check the reduction and the whole-job figure."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_15211_b200.replicas import max_over_ranks, whole_job_tflops


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms = 3.0 + rank                       # rank 1 is the slower replica
        slowest = max_over_ranks(ms)
        dist.barrier()
        out[rank] = (slowest, whole_job_tflops(6.0e11, world, slowest))
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_aggregate():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in range(world):
        slowest, value = res[rank]
        assert slowest == 4.0                                    # max over ranks, the same on every rank
        assert abs(value - 2 * 6.0e11 / 4.0e-3 / 1e12) < 1e-9    # whole job = both replicas over the slowest time


def test_single_process_is_its_own_maximum():
    assert max_over_ranks(2.5) == 2.5
    assert abs(whole_job_tflops(1.0e12, 1, 1.0) - 1000.0) < 1e-9
