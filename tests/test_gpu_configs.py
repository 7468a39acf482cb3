"""The five benchmark configurations at full size, through the C ABI in the launch configuration the benchmark
times, checked against the CPU oracle.

The oracle cannot run a full configuration (1-36 TFLOP of scalar fp64), so: indexer scores, top-k selections and
attention outputs are compared on sampled query rows (first, last, evenly spread; rows are independent, so this is
exact for those rows), page sets / runs / miss sets are compared bit-exactly on ALL rows of the GPU's own
selection (integer work), and size-independent properties are checked on every row (selection size, index range,
causality, no duplicates on sampled rows)."""
import numpy as np
import pytest
import torch

from oracle import janus_oracle as O
from paper_2609_36938_b200 import binding as B
from paper_2609_36938_b200 import build
from paper_2609_36938_b200 import workloads as W

import helpers as Hp

pytestmark = pytest.mark.gpu

N_SAMPLE_ROWS = 10


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    B.load()
    yield


def oracle_row_scores(sess, t, *, predicted=False):
    """Oracle scores of one query row (called with a one-row query block positioned at L+t)."""
    shp = sess["shape"]
    q = sess["q_pred" if predicted else "q_idx"][t:t + 1]
    w = sess["w"][t:t + 1]
    if predicted:
        ks = None if sess["k_scale"] is None else sess["k_scale"][:shp.L]
        return O.indexer_scores(q, sess["k_idx"][:shp.L], w, dtype=shp.idx_dtype, q_scale=sess["q_scale"], k_scale=ks, q_pos0=shp.L + t,
                                causal=False)[0]
    return O.indexer_scores(q, sess["k_idx"], w, dtype=shp.idx_dtype, q_scale=sess["q_scale"], k_scale=sess["k_scale"],
                            recency=sess["recency"], q_pos0=shp.L + t, causal=True)[0]


def boundary_rows(shp):
    """Query rows whose causal diagonal (their own key, position L + t) is the last key of a 128-key tile and the first key
    of the next one, the same for the key chunk one CTA of the indexer walks (up to 256 tiles; 64 tiles checked too), and the last and first
    row of a CTA's 16-token query group: the places where a tile-edge or mask-edge mistake would show."""
    rows = set()
    for period in (128, 64 * 128, 256 * 128):
        t_last = (period - 1 - shp.L) % period           # L + t = period - 1 (mod period)
        rows |= {t_last, t_last + 1}
    rows |= {15, 16}
    return np.array(sorted(t for t in rows if 0 <= t < shp.M), dtype=np.int64)


def run_and_check(sess, n_rows=N_SAMPLE_ROWS):
    shp = sess["shape"]
    d = Hp.upload_session(sess)
    n_phys = sess["n_phys_pages"]
    # predicted pass (Eq. 2): lookahead queries against the history keys only
    pred_bitmap, pred_idx = None, None
    if "q_pred" in d:
        psc = B.janus_indexer_scores(d["q_pred"], d["k_idx"][:shp.L], d["w"], q_scale=d["q_scale"],
                                     k_scale=None if d["k_scale"] is None else d["k_scale"][:shp.L], q_pos0=shp.L, causal=False)
        pred_idx, _, _ = B.janus_topk(psc, shp.L, shp.k, q_pos0=shp.L, causal=False)
        pred_bitmap = B.janus_page_demand(pred_idx, demand_limit=shp.L, page_size=shp.page_size, page_table=d["page_table"],
                                          n_phys_pages=n_phys, want_miss=False)["bitmap"]
        del psc
    # exact pass
    sc = B.janus_indexer_scores(d["q_idx"], d["k_idx"], d["w"], q_scale=d["q_scale"], k_scale=d["k_scale"], row_bias=d["row_bias"],
                                col_bias=d["col_bias"], q_pos0=shp.L, causal=True)
    idx, count, kth = B.janus_topk(sc, shp.S, shp.k, q_pos0=shp.L, causal=True)
    pd = B.janus_page_demand(idx, demand_limit=shp.L, page_size=shp.page_size, page_table=d["page_table"], n_phys_pages=n_phys,
                             predicted_bitmap=pred_bitmap)
    out, lse = B.janus_sparse_attn_prefill(d["Q"], d["k_pool"], d["v_pool"], idx, page_table=d["page_table"], page_size=shp.page_size,
                                           softmax_scale=shp.softmax_scale, d_v=shp.d_v)
    B.check_dev_status()

    rows = np.unique(np.concatenate([W.sample_rows(shp.M, n_rows), boundary_rows(shp)]))
    idx_np = idx.cpu().numpy()
    # ---- properties on every row
    cnt = count.cpu().numpy()
    expect = np.minimum(shp.k, shp.L + np.arange(shp.M) + 1)
    assert np.array_equal(cnt, expect)
    assert np.array_equal((idx_np >= 0).sum(axis=1), expect)
    assert np.all(idx_np.max(axis=1) <= shp.L + np.arange(shp.M)), "causality"
    # ---- sampled rows against the oracle
    tol = 1e-2 if shp.idx_dtype == "bf16" else 5e-2
    got_rows = sc[torch.from_numpy(rows).cuda(), :shp.S].cpu().numpy()
    for i, t in enumerate(rows):
        t = int(t)
        ref = oracle_row_scores(sess, t)
        Hp.assert_scores_close(got_rows[i:i + 1], ref[None, :], tol, f"config {shp.config_id} row {t}")
        Hp.assert_scores_close(got_rows[i:i + 1], ref[None, :], 2e-4, f"config {shp.config_id} row {t} (tight)")
        ok, msg = O.topk_row_agrees(idx_np[t], ref, shp.L + t + 1, shp.k)
        assert ok, f"config {shp.config_id} row {t}: {msg}"
        if pred_idx is not None:
            pref = oracle_row_scores(sess, t, predicted=True)
            ok, msg = O.topk_row_agrees(pred_idx[t].cpu().numpy(), pref, shp.L, shp.k)
            assert ok, f"config {shp.config_id} predicted row {t}: {msg}"
    ref_o, ref_lse = O.sparse_attention(sess["Q"][rows], sess["k_pool"], sess["v_pool"], sess["page_table"], idx_np[rows],
                                        page_size=shp.page_size, softmax_scale=shp.softmax_scale, d_qk=shp.d_qk, d_v=shp.d_v)
    got_o = Hp.bf16_tensor_to_f64(out[torch.from_numpy(rows).cuda()])
    Hp.assert_attention_close(got_o, ref_o, f"config {shp.config_id}")
    np.testing.assert_allclose(lse[torch.from_numpy(rows).cuda()].cpu().numpy(), ref_lse, rtol=2e-3, atol=2e-3)
    # ---- page demand on all rows, bit-exact
    pred_pages = None
    if pred_idx is not None:
        pred_pages = O.page_demand(pred_idx.cpu().numpy(), shp.L, shp.page_size, sess["page_table"])["pages"]
        assert Hp.bitmap_to_pages(pred_bitmap, n_phys) == pred_pages
    ref_pd = O.page_demand(idx_np, shp.L, shp.page_size, sess["page_table"], predicted_pages=pred_pages)
    got_pd = Hp.page_lists_from_device(pd)
    if pred_pages is None:
        ref_pd["miss"], ref_pd["miss_runs"] = ref_pd["pages"], ref_pd["runs"]
    assert got_pd == {k_: ref_pd[k_] for k_ in ("pages", "runs", "miss", "miss_runs")}
    assert set(got_pd["miss"]) == set(got_pd["pages"]) - set(pred_pages or [])
    stats = {"n_pages": len(got_pd["pages"]), "n_runs": len(got_pd["runs"]), "n_miss": len(got_pd["miss"])}
    if pred_pages is not None:
        stats["page_recall"], stats["page_precision"] = O.recall_precision(pred_pages, got_pd["pages"])
    return stats


def test_config1_tiny_mha_full():
    shp = W.config_shape(1)
    stats = run_and_check(W.make_session(shp, seed=0), n_rows=shp.M)      # the oracle finishes this one in full
    assert stats["n_pages"] == 64 and stats["n_runs"] == 1                    # M*k >> pages: every history page, identity table
    assert stats["page_recall"] == 1.0 and stats["n_miss"] == 0


def test_config2_latent_bf16():
    stats = run_and_check(W.make_session(W.config_shape(2), seed=0))
    assert stats["n_pages"] == 512


def test_config3_fp8_indexer_128k():
    stats = run_and_check(W.make_session(W.config_shape(3), seed=0))
    assert stats["n_pages"] == 2048


def test_config4_ragged_batch_with_prediction():
    shapes = W.batch_shapes(0)
    sessions = W.make_batch(0, shapes)
    for sess in sessions:
        shp = sess["shape"]
        stats = run_and_check(sess, n_rows=4)
        assert 0.0 <= stats["page_recall"] <= 1.0
        # token-granularity report (page size 1, identity table) is exercised on the first session only
    sess = sessions[0]
    shp = sess["shape"]
    d = Hp.upload_session(sess)
    sc = B.janus_indexer_scores(d["q_idx"], d["k_idx"], d["w"], q_pos0=shp.L, causal=True)
    idx, _, _ = B.janus_topk(sc, shp.S, shp.k, q_pos0=shp.L, causal=True)
    ident = torch.arange(shp.S, dtype=torch.int32, device="cuda")
    tok = B.janus_page_demand(idx, demand_limit=shp.L, page_size=1, page_table=ident, n_phys_pages=shp.S, want_miss=False)
    n_tok = int(tok["counts"][0])
    uniq = np.unique(idx.cpu().numpy())
    uniq = uniq[(uniq >= 0) & (uniq < shp.L)]
    assert n_tok == len(uniq) <= shp.M * shp.k                              # |S| <= M*k (Sec. 4.2)
    assert np.array_equal(tok["pages"][:n_tok].cpu().numpy(), uniq)
    B.check_dev_status()


def test_config5_long_structured_fp8():
    stats = run_and_check(W.make_session(W.config_shape(5), seed=0), n_rows=6)
    assert 0 < stats["n_pages"] <= 4096
