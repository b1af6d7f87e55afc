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


# ------------------------------------------------------------------ N-sharded layer (output columns over ranks)

def test_shard_columns_cover_the_layer_in_balanced_whole_tiles():
    from paper_2608_15531_b200.sharded import shard_columns
    for N, world in [(4096, 2), (28672, 8), (768, 2), (6144, 5), (512, 4), (256, 3)]:
        rs = shard_columns(N, world)
        assert len(rs) == world and rs[0][0] == 0 and rs[-1][1] == N
        assert all(a1 == b0 for (_, a1), (b0, _) in zip(rs, rs[1:]))
        widths = [b - a for a, b in rs]
        assert all(w % 256 == 0 for w in widths) and max(widths) - min(widths) <= 256
        assert widths == sorted(widths, reverse=True)
    import pytest
    with pytest.raises(ValueError):
        shard_columns(1000, 2)


def _sharded_worker(rank: int, world: int, port: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import numpy as np
    import oracle
    from paper_2608_15531_b200 import synth
    from paper_2608_15531_b200.sharded import ShardedLayer, shard_outliers
    K, N, g, M = 256, 768, 128, 3                      # three column tiles over two ranks: widths 512 and 256
    lay = synth.layer(31, K, N, density=0.02, layout="mixed")
    X = synth.activations(7, M, K)

    def compute(Xb, shard):
        # the per-rank compute, replaced by the oracle on the rank's own columns (this is a CPU test)
        n0, n1 = shard.n0, shard.n1
        q, s, z = oracle.quantize(np.ascontiguousarray(lay.W[:, n0:n1]), np.ascontiguousarray(lay.mask[:, n0:n1]), g)
        k, n, v = shard_outliers(lay.coo_k, lay.coo_n, lay.coo_v, n0, n1)
        return torch.from_numpy(oracle.fused_matmul(Xb.numpy().view(np.uint16), q, s, z, g, k, n, v))

    layer = ShardedLayer(lay.W, lay.mask, lay.coo_k, lay.coo_n, lay.coo_v, g, rank, world, compute=compute)
    Y = layer.forward(torch.from_numpy(X.view(np.int16)))
    out[rank] = (Y.numpy().copy(), layer.shard.n0, layer.shard.n1)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_gather_their_column_shards_into_the_full_result():
    import numpy as np
    import oracle
    from paper_2608_15531_b200 import synth
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_sharded_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    K, N, g, M = 256, 768, 128, 3
    lay = synth.layer(31, K, N, density=0.02, layout="mixed")
    X = synth.activations(7, M, K)
    q, s, z = oracle.quantize(lay.W, lay.mask, g)
    want = oracle.fused_matmul(X, q, s, z, g, lay.coo_k, lay.coo_n, lay.coo_v)
    assert (out[0][1], out[0][2], out[1][1], out[1][2]) == (0, 512, 512, 768)
    for rank in range(world):
        assert out[rank][0].shape == (M, N)
        # per-column quantisation does not depend on the other columns: the sharded result is the full one, bit for bit
        assert np.array_equal(out[rank][0], want)

