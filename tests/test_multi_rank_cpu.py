"""The N > 1 path of bench.py on CPU: two gloo ranks as independent replicas (the method itself has no
collective; ranks only agree on the slowest rank's time)."""
import os
import socket
import sys

import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import torch.distributed as dist

    import bench

    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env() == (rank, world, rank)
    my_ms = 2.0 if rank == 0 else 3.5  # rank 1 is the slow replica
    slowest = bench.max_over_ranks(my_ms, world, torch.device("cpu"))
    dist.barrier()
    out[rank] = (slowest, bench.whole_job_value(slowest, world))
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_whole_job():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 3.5
    assert abs(res[0][1] - 2 * 1000.0 / 3.5) < 1e-9


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.max_over_ranks(1.25, 1, torch.device("cpu")) == 1.25
    assert bench.whole_job_value(2.0, 1) == 500.0
