"""The N > 1 benchmark path on CPU: two gloo ranks, each with its own seeded shard of
independent (batch, head) units; times reduce with MAX, work with SUM, no data-path collective."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
from paper_2506_23858_b200 import inputs as gen


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    layers = bench.rank_workloads([gen.C1], rank)
    data = gen.make_inputs(layers[0], with_do=False)
    ms, e2e, flops = bench.aggregate_over_ranks(10.0 + rank, 20.0 - rank, 100.0 * (rank + 1), "cpu")
    out[rank] = (ms, e2e, flops, float(data["q"].sum()), layers[0].seed)
    dist.destroy_process_group()


def test_two_rank_aggregation_and_sharding():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    assert out[0][:3] == out[1][:3] == (11.0, 20.0, 300.0)      # max time, max e2e time, summed work
    assert out[0][4] != out[1][4] and out[0][3] != out[1][3]       # different seeded batches per rank


def test_single_process_aggregation_is_identity():
    assert bench.aggregate_over_ranks(1.5, 2.5, 7.0, "cpu") == (1.5, 2.5, 7.0)
