"""The benchmark's multi-rank bookkeeping on CPU: two gloo ranks (independent replicas, no collective
on the data path) reduce their step times with MAX and report the whole-job throughput."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    pre_ms, dec_ms = 1.0 + 0.5 * rank, 0.30 - 0.05 * rank      # rank 1 is slower in prefill, rank 0 in decode
    dist.barrier()
    got = bench.max_over_ranks([pre_ms, dec_ms], world, "cpu")
    val = bench.job_tokens_per_s(4096, world, got[0])
    out[rank] = (got, val)
    dist.destroy_process_group()


def test_two_rank_aggregation_with_gloo():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        got, val = res[rank]
        assert got == [1.5, 0.30]                       # MAX over ranks, element-wise, same on every rank
        assert abs(val - 2 * 4096 / 1.5e-3) < 1e-6      # both replicas' tokens over the slowest rank's time


def test_single_rank_is_a_no_op():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([2.0, 3.0], 1) == [2.0, 3.0]
    assert bench.job_tokens_per_s(100, 1, 10.0) == 10000.0
