"""The multi-rank host logic of bench.py on CPU: two gloo ranks shard the batch (rank-specific
seeds, no data-path collective), the step time is the max over ranks, the value is the whole job's."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
from paper_2604_04250_b200 import inputs


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # each rank's shard is its own draw of the same recipe
    d = inputs.scan_inputs(1, 8, 64, bench.rank_seed(5, rank))
    my_ms = 10.0 + 5.0 * rank                        # rank 1 is the slow one
    total, e2e = bench.reduce_max([my_ms, 2 * my_ms], world, "cpu")
    dist.barrier()
    out[rank] = (total, e2e, float(np.abs(d["p"]).sum()))
    dist.destroy_process_group()


def test_two_gloo_ranks_max_time_and_whole_job_value():
    world, port = 2, _free_port()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    assert out[0][:2] == (15.0, 30.0) and out[1][:2] == (15.0, 30.0)      # max over ranks, on every rank
    assert out[0][2] != out[1][2]                                         # different shards
    v = bench.whole_job_value(world, 16384, 15.0)
    assert abs(v - 2 * 16384 / 15e-3 / 1e6) < 1e-9
    assert bench.whole_job_value(1, 16384, 15.0) * 2 == v                 # weak scaling: work per rank fixed
