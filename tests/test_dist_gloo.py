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


# ---- key-sharded prediction (Sec. 4.2, Eq. 3) across two ranks: disjoint history shards, one union at the end ------------
def _pages_to_bitmap(pages, n_phys):
    import numpy as np

    words = np.zeros((n_phys + 31) // 32, dtype=np.uint32)
    for p in pages:
        words[p >> 5] |= np.uint32(1) << np.uint32(p & 31)
    return torch.from_numpy(words.view(np.int32).copy())


def _bitmap_to_pages(bitmap, n_phys):
    import numpy as np

    bits = np.unpackbits(bitmap.numpy().view(np.uint8), bitorder="little")[:n_phys]
    return np.nonzero(bits)[0].tolist()


def _shard_session():
    shp = W.config_shape(4, L=1500, M=6, k=64)          # 24 pages of 64 tokens, the last one partial
    import dataclasses

    shp = dataclasses.replace(shp, table="shuffled")
    return shp, W.make_session(shp, seed=7, with_attention=False)


def _shard_pages(sess, shp, a, b, k_shard):
    """The oracle's predicted page set of history shard [a, b): non-causal scores over the shard's keys, top-(k/N), pages
    through the slice of the page table that starts at the shard's first page."""
    from oracle import janus_oracle as O

    sc = O.indexer_scores(sess["q_pred"], sess["k_idx"][a:b], sess["w"], dtype=shp.idx_dtype, q_pos0=shp.L, causal=False)
    idx = O.topk(sc, k_shard, q_pos0=shp.L, causal=False)
    return O.page_demand(idx, b - a, shp.page_size, sess["page_table"][a // shp.page_size:])["pages"]


def _shard_worker(rank, world, port, out):
    from paper_2609_36938_b200 import prediction as P

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        shp, sess = _shard_session()
        n_phys = sess["n_phys_pages"]
        a, b = P.shard_bounds(shp.L, world, shp.page_size)[rank]
        mine = _shard_pages(sess, shp, a, b, shp.k // world)       # no exchange up to here: the rank could prefetch these now
        union = D.or_reduce_bitmap(_pages_to_bitmap(mine, n_phys))
        out[rank] = (mine, _bitmap_to_pages(union, n_phys))
    finally:
        dist.destroy_process_group()


def test_two_ranks_predict_on_disjoint_history_shards_and_unite_their_page_sets():
    from oracle import janus_oracle as O
    from paper_2609_36938_b200 import prediction as P

    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_shard_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    (mine0, union0), (mine1, union1) = out[0], out[1]
    shp, sess = _shard_session()
    # the same shards, computed in this process one after another
    want = [_shard_pages(sess, shp, a, b, shp.k // world) for a, b in P.shard_bounds(shp.L, world, shp.page_size)]
    assert mine0 == want[0] and mine1 == want[1]
    assert not set(mine0) & set(mine1)                              # disjoint shards never ask for the same page (Sec. 4.2)
    assert union0 == union1 == sorted(set(want[0]) | set(want[1]))  # every rank ends with the same union
    # what the exact pass would still have to read: its pages minus the union
    sc = O.indexer_scores(sess["q_idx"], sess["k_idx"], sess["w"], dtype=shp.idx_dtype, q_pos0=shp.L, causal=True)
    exact = O.page_demand(O.topk(sc, shp.k, q_pos0=shp.L, causal=True), shp.L, shp.page_size, sess["page_table"], predicted_pages=union0)
    assert exact["miss"] == sorted(set(exact["pages"]) - set(union0))


def test_or_reduce_bitmap_single_process_passthrough():
    b = torch.tensor([5, 0, -1], dtype=torch.int32)
    u = D.or_reduce_bitmap(b)
    assert torch.equal(u, b) and u.data_ptr() != b.data_ptr()


# ---- query-parallel partition (Sec. 4.2): each rank selects for its slice of the new tokens, the page sets are united -----------
def _query_worker(rank, world, port, out):
    from oracle import janus_oracle as O

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        shp, sess = _shard_session()
        r0, r1 = rank * shp.M // world, (rank + 1) * shp.M // world
        sc = O.indexer_scores(sess["q_idx"], sess["k_idx"], sess["w"], dtype=shp.idx_dtype, q_pos0=shp.L, causal=True, rows=range(r0, r1))
        idx = O.topk(sc, shp.k, q_pos0=shp.L, causal=True, rows=range(r0, r1))
        mine = O.page_demand(idx, shp.L, shp.page_size, sess["page_table"])["pages"]
        union = D.or_reduce_bitmap(_pages_to_bitmap(mine, sess["n_phys_pages"]))
        out[rank] = (mine, _bitmap_to_pages(union, sess["n_phys_pages"]))
    finally:
        dist.destroy_process_group()


def test_two_ranks_split_the_query_rows_and_unite_their_page_sets():
    from oracle import janus_oracle as O

    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_query_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    shp, sess = _shard_session()
    sc = O.indexer_scores(sess["q_idx"], sess["k_idx"], sess["w"], dtype=shp.idx_dtype, q_pos0=shp.L, causal=True)
    full = O.page_demand(O.topk(sc, shp.k, q_pos0=shp.L, causal=True), shp.L, shp.page_size, sess["page_table"])["pages"]
    (mine0, union0), (mine1, union1) = out[0], out[1]
    assert union0 == union1 == full == sorted(set(mine0) | set(mine1))      # rows are independent: the union is the session's demand
