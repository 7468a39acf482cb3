"""Lookahead prediction (Eq. 2) and its synchronisation-free sharded form (Eq. 3, Sec. 4.2) through the C ABI, checked
against the oracle: per-shard selections on sampled rows, per-shard page sets bit-exactly on all rows, disjointness of the
shards' page sets, the union, and the recall / precision of both predicted sets against the exact page set."""
import numpy as np
import pytest
import torch

from oracle import janus_oracle as O
from paper_2609_36938_b200 import binding as B
from paper_2609_36938_b200 import build, prediction as P
from paper_2609_36938_b200 import workloads as W

import helpers as Hp

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    B.load()
    yield
    B.check_dev_status()


def test_shard_bounds_are_disjoint_page_aligned_and_cover_the_history():
    for L, n, pg in ((1000, 8, 64), (4096, 4, 64), (130, 8, 64), (77, 3, 16)):
        b = P.shard_bounds(L, n, pg)
        assert b[0][0] == 0 and b[-1][1] == L
        for (a0, b0), (a1, _) in zip(b, b[1:]):
            assert b0 == a1 and a1 % pg == 0
        assert all(bb > aa for aa, bb in b)


@pytest.mark.parametrize("n_shards", [2, 8])
def test_sharded_prediction_matches_oracle_and_reports_quality(n_shards):
    # a reduced session of the ragged-batch configuration: correlated lookahead queries, fragmented page table
    shp = W.config_shape(4, L=24000, M=48, k=64)
    tables, n_phys = W.fragmented_page_tables([shp, W.config_shape(4, L=9000, M=64, k=64)], seed=3)
    sess = W.make_session(shp, seed=3, with_attention=False, page_table=tables[0], n_phys_pages=n_phys)
    d = Hp.upload_session(sess)
    pg, L, k = shp.page_size, shp.L, shp.k

    # exact pass
    sc = B.janus_indexer_scores(d["q_idx"], d["k_idx"], d["w"], q_pos0=L, causal=True)
    idx, _, _ = B.janus_topk(sc, shp.S, k, q_pos0=L, causal=True)
    exact = B.janus_page_demand(idx, demand_limit=L, page_size=pg, page_table=d["page_table"], n_phys_pages=n_phys)
    exact_pages = Hp.bitmap_to_pages(exact["bitmap"], n_phys)

    # unsharded prediction (Eq. 2)
    pred_bitmap, pred_idx = P.predicted_pages(d["q_pred"], d["k_idx"], d["w"], L=L, k=k, page_size=pg, page_table=d["page_table"],
                                              n_phys_pages=n_phys)
    pred_pages = Hp.bitmap_to_pages(pred_bitmap, n_phys)
    assert pred_pages == O.page_demand(pred_idx.cpu().numpy(), L, pg, sess["page_table"])["pages"]

    # sharded prediction (Eq. 3)
    union, bitmaps, indices = P.sharded_predicted_pages(d["q_pred"], d["k_idx"], d["w"], L=L, k=k, n_shards=n_shards, page_size=pg,
                                                        page_table=d["page_table"], n_phys_pages=n_phys)
    B.check_dev_status()
    bounds = P.shard_bounds(L, n_shards, pg)
    rows = W.sample_rows(shp.M, 4)
    all_shard_pages = []
    for (a, b), bm, ix in zip(bounds, bitmaps, indices):
        ix_np = ix.cpu().numpy()
        assert ix_np.shape == (shp.M, k // n_shards)
        # selection of the shard on sampled rows: the same indexer restricted to the shard's keys, top-(k/N)
        for t in rows:
            ref = O.indexer_scores(sess["q_pred"][t:t + 1], sess["k_idx"][a:b], sess["w"][t:t + 1], q_pos0=L + int(t), causal=False)[0]
            ok, msg = O.topk_row_agrees(ix_np[t], ref, b - a, k // n_shards)
            assert ok, f"shard [{a},{b}) row {t}: {msg}"
        # page set of the shard, bit-exact on all rows (global token = local index + shard start)
        glob = np.where(ix_np >= 0, ix_np + a, -1)
        ref_pages = O.page_demand(glob, L, pg, sess["page_table"])["pages"]
        got_pages = Hp.bitmap_to_pages(bm, n_phys)
        assert got_pages == ref_pages
        all_shard_pages.append(set(got_pages))
    # disjoint shards never request the same page twice (Sec. 4.2), and the union is the union
    for i in range(len(all_shard_pages)):
        for j in range(i + 1, len(all_shard_pages)):
            assert not (all_shard_pages[i] & all_shard_pages[j])
    union_pages = Hp.bitmap_to_pages(union, n_phys)
    assert set(union_pages) == set().union(*all_shard_pages)

    # the miss set against the sharded prediction is "exact minus union"
    miss = B.janus_page_demand(idx, demand_limit=L, page_size=pg, page_table=d["page_table"], n_phys_pages=n_phys, predicted_bitmap=union)
    got = Hp.page_lists_from_device(miss)
    assert got["miss"] == sorted(set(exact_pages) - set(union_pages))

    r0, p0 = O.recall_precision(pred_pages, exact_pages)
    r1, p1 = O.recall_precision(union_pages, exact_pages)
    print(f"\nN={n_shards}: unsharded recall {r0:.4f} precision {p0:.4f} | sharded recall {r1:.4f} precision {p1:.4f} "
          f"| pages exact {len(exact_pages)} pred {len(pred_pages)} sharded {len(union_pages)}")
    assert 0.0 <= r1 <= 1.0 and 0.0 <= p1 <= 1.0
