"""The N > 1 path of the benchmark on CPU: two gloo ranks, each a replica with its own
timing; the slowest rank sets the whole-job rate (no data-path collective exists)."""
import os
import socket
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from paper_2506_19651_b200 import replicas
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    my_ms = 2.0 + rank            # rank 1 is the slow replica
    slowest = replicas.max_over_ranks(my_ms)
    rate = replicas.whole_job_rate(1000.0, world, slowest)
    dist.barrier()
    out[rank] = (slowest, rate)
    dist.destroy_process_group()


def test_two_replicas_report_slowest_rank_and_aggregate_rate():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    assert out[0] == out[1] == (3.0, 2 * 1000.0 / 3.0e-3)


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    from paper_2506_19651_b200 import replicas
    assert replicas.max_over_ranks(1.5) == 1.5
    assert replicas.whole_job_rate(10.0, 1, 5.0) == 2000.0
