"""The N > 1 path of bench.py is "replicas only": ranks do not exchange data, they only agree on
the slowest rank's time.  Two gloo ranks on CPU check that agreement and the whole-job figure."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    local_ms = 1.0 + rank            # rank 1 is the slow one
    dist.barrier()
    ms = bench.max_over_ranks(local_ms, world)
    out[rank] = (ms, bench.whole_job_gbs(10_000_000, world, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_aggregate_rate():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    assert set(out.keys()) == {0, 1}
    for rank in range(world):
        ms, gbs = out[rank]
        assert ms == 2.0                                  # max over ranks, identical on both
        assert abs(gbs - 2 * 10_000_000 / 2.0e-3 / 1e9) < 1e-12


def test_single_rank_is_the_identity():
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert abs(bench.whole_job_gbs(8_000_000, 1, 2.0) - 4.0) < 1e-12
