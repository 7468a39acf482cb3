"""World-size-2 checks of the multi-rank plumbing on CPU (gloo): unit sharding and the max-over-ranks timing rule."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_36938_b200 import dist_utils as D
from paper_2609_36938_b200 import workloads as W


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = D.shard_units(5, rank, world)
        # each rank "processes" its own sessions: different seeds give different inputs, no exchange of data
        tokens = 0
        for u in mine:
            shp = W.config_shape(1, L=64, M=8 + u, k=4)
            sess = W.make_session(shp, seed=u, with_attention=False)
            tokens += sess["q_idx"].shape[0]
        elapsed_ms = 10.0 * (rank + 1)                      # rank 1 is the slow one
        value, t_max, total = D.aggregate_throughput(float(tokens), elapsed_ms)
        out[rank] = (mine, tokens, value, t_max, total)
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_sessions_and_report_the_slowest_time():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    (mine0, tok0, v0, t0, tot0), (mine1, tok1, v1, t1, tot1) = out[0], out[1]
    assert sorted(mine0 + mine1) == [0, 1, 2, 3, 4] and not set(mine0) & set(mine1)
    assert tok0 == 8 + 10 + 12 and tok1 == 9 + 11
    assert t0 == t1 == 20.0                                 # maximum over ranks
    assert tot0 == tot1 == 50.0
    assert v0 == v1 == 50.0 / 20e-3


def test_single_process_passthrough():
    v, t, u = D.aggregate_throughput(100.0, 50.0)
    assert (v, t, u) == (2000.0, 50.0, 100.0)
