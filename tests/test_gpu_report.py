"""The reporting code of the benchmark (recall / precision of the predicted set, miss-set size, runs, at page and at token
granularity; Sec. 4.2 and Sec. 4.3) computes its figures from the library's device outputs.  Here the same figures are
recomputed by the oracle from the selections the GPU made, on a session small enough for plain Python sets."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import janus_oracle as O
from paper_2609_36938_b200 import binding as B
from paper_2609_36938_b200 import build
from paper_2609_36938_b200 import report as R
from paper_2609_36938_b200 import workloads as W

import helpers as Hp

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    B.load()
    yield
    B.check_dev_status()


def test_report_matches_oracle_sets():
    # few rows and a small budget so that the page sets do not saturate: the predicted and the exact sets really differ
    shp = dataclasses.replace(W.config_shape(4, L=6000, M=5, k=48), table="shuffled")
    sess = W.make_session(shp, seed=5, with_attention=False)
    d = Hp.upload_session(sess)
    n_phys = sess["n_phys_pages"]
    psc = B.janus_indexer_scores(d["q_pred"], d["k_idx"][:shp.L], d["w"], q_pos0=shp.L, causal=False)
    pidx, _, _ = B.janus_topk(psc, shp.L, shp.k, q_pos0=shp.L, causal=False)
    pred = B.janus_page_demand(pidx, demand_limit=shp.L, page_size=shp.page_size, page_table=d["page_table"], n_phys_pages=n_phys, want_miss=False)
    sc = B.janus_indexer_scores(d["q_idx"], d["k_idx"], d["w"], q_pos0=shp.L, causal=True)
    idx, _, _ = B.janus_topk(sc, shp.S, shp.k, q_pos0=shp.L, causal=True)
    pd = B.janus_page_demand(idx, demand_limit=shp.L, page_size=shp.page_size, page_table=d["page_table"], n_phys_pages=n_phys,
                             predicted_bitmap=pred["bitmap"])
    B.check_dev_status()
    rep = R.demand_report(pd, pred["bitmap"])
    tok = R.token_granularity_report(idx, pidx, shp.L)
    B.check_dev_status()

    idx_h, pidx_h = idx.cpu().numpy(), pidx.cpu().numpy()
    exact_pages = O.page_demand(idx_h, shp.L, shp.page_size, sess["page_table"])
    pred_pages = O.page_demand(pidx_h, shp.L, shp.page_size, sess["page_table"])["pages"]
    recall, precision = O.recall_precision(pred_pages, exact_pages["pages"])
    assert 0 < len(set(exact_pages["pages"]) - set(pred_pages)) < len(exact_pages["pages"]), "the case must have a non-trivial miss set"
    assert rep["n_demand"] == len(exact_pages["pages"]) and rep["n_predicted"] == len(pred_pages)
    assert rep["n_miss"] == len(set(exact_pages["pages"]) - set(pred_pages))
    assert rep["n_runs"] == len(exact_pages["runs"])
    assert rep["recall"] == pytest.approx(recall, abs=1e-15) and rep["precision"] == pytest.approx(precision, abs=1e-15)
    assert rep["mean_run_length"] == pytest.approx(len(exact_pages["pages"]) / len(exact_pages["runs"]))
    hist = R.run_length_histogram(pd)
    want = {}
    for _, ln in exact_pages["runs"]:
        want[ln] = want.get(ln, 0) + 1
    assert hist == want

    # token granularity: the sets are the selected history tokens themselves
    exact_tok = sorted(set(int(s) for s in idx_h.ravel() if 0 <= s < shp.L))
    pred_tok = sorted(set(int(s) for s in pidx_h.ravel() if 0 <= s < shp.L))
    r_tok, p_tok = O.recall_precision(pred_tok, exact_tok)
    assert tok["n_demand"] == len(exact_tok) <= shp.M * shp.k and tok["n_predicted"] == len(pred_tok)
    assert tok["n_miss"] == len(set(exact_tok) - set(pred_tok))
    assert tok["n_runs"] == len(O.maximal_runs(exact_tok))
    assert tok["recall"] == pytest.approx(r_tok, abs=1e-15) and tok["precision"] == pytest.approx(p_tok, abs=1e-15)
    assert R.popcount(pred["bitmap"]) == len(pred_pages)
