"""The N > 1 path of the benchmark on CPU: two gloo ranks, barrier, max-over-ranks
timing, whole-job throughput of independent replicas."""
import os
import socket

import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2112_10769_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        replicas.barrier()
        seconds = 0.5 if rank == 0 else 2.0          # rank 1 is the slow replica
        out[rank] = (replicas.world(), replicas.max_over_ranks(seconds), replicas.job_throughput(10.0, seconds))
        replicas.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_report_the_slowest_replica():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_rank_main, args=(world, _free_port(), out), nprocs=world, join=True)
    for rank in range(world):
        w, slowest, thr = out[rank]
        assert w == 2 and slowest == 2.0 and thr == 2 * 10.0 / 2.0


def test_single_process_is_a_world_of_one():
    assert replicas.world() == 1
    assert replicas.max_over_ranks(3.0) == 3.0
    assert replicas.job_throughput(6.0, 3.0) == 2.0
    replicas.barrier()
