"""The N > 1 benchmark path has no exchange step (replicas only): what is shared between ranks is
the timing reduction (slowest rank), the aggregate throughput and the per-rank seeds.  Checked here
with two gloo ranks on CPU."""
import os
import socket
import sys

import numpy as np
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
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2108_13342_b200 import workloads as W
    ms = bench.max_over_ranks(1.0 + rank)                       # rank 1 is the slow one
    val = bench.aggregate_throughput(1e9, ms, world)
    wl = W.masked_softmax(batch=1, heads=1, s=8, seed=bench.rank_seed(W.BASE_SEED, rank))
    out[rank] = (ms, val, float(wl.inputs["S"].sum()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_agree_on_slowest_time_and_draw_different_inputs():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    assert out[0][0] == out[1][0] == 2.0                        # max over ranks, same on every rank
    assert abs(out[0][1] - 2 * 1e9 / 2e-3 / 1e9) < 1e-9         # two replicas' bytes over the slowest time
    assert out[0][2] != out[1][2]                               # rank-dependent seeds


def test_single_process_path_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.aggregate_throughput(2e9, 1.0, 1) == 2e9 / 1e-3 / 1e9
