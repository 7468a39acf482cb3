"""Entry-granularity selection (footnote of Sec. 2.2, in this library's stated reading) through the C ABI: entry scores
from the indexer over one key per entry, janus_topk_entries, janus_entry_expand, then page demand and attention on the
expanded token selection; each step against the oracle, plus the invariant that selecting every visible entry gives dense
causal attention.  Also index reuse: one selection driving the attention of two layers' KV pools."""
import numpy as np
import pytest
import torch

from oracle import janus_oracle as O
from paper_2609_36938_b200 import binding as B
from paper_2609_36938_b200 import build
from paper_2609_36938_b200 import workloads as W

import helpers as Hp

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    B.load()
    yield
    B.check_dev_status()


def dev(x, kind):
    return B.to_device(x, kind)


@pytest.mark.parametrize("E,L,M,k_e", [(128, 40000, 24, 16), (16, 5003, 37, 40), (64, 100, 70, 8)])
def test_entry_pipeline_matches_oracle(E, L, M, k_e):
    rng = np.random.default_rng(E + L)
    S = L + M
    n_entries = (S + E - 1) // E
    H, D, page, d_qk, d_v, H_q = 64, 128, 64, 576, 512, 128
    q = W.to_bf16_bits(rng.standard_normal((M, H, D)).astype(np.float32))
    ke = W.to_bf16_bits(rng.standard_normal((n_entries, D)).astype(np.float32))        # one indexer key per entry
    w = (rng.uniform(0, 1, (M, H)) / 8).astype(np.float32)
    sc = B.janus_indexer_scores(dev(q, "bf16"), dev(ke, "bf16"), dev(w, "f32"), q_pos0=0, causal=False)
    idx_e, cnt, _ = B.janus_topk_entries(sc, n_entries, k_e, q_pos0=L, entry_size=E)
    idx_t = B.janus_entry_expand(idx_e, q_pos0=L, entry_size=E)
    B.check_dev_status()
    ref_sc = O.indexer_scores(q, ke, w, dtype="bf16", q_pos0=0, causal=False)
    idx_e_h, idx_t_h = idx_e.cpu().numpy(), idx_t.cpu().numpy()
    for t in range(M):
        prefix = O.entry_visible_prefix(t, n_entries, L, E)
        assert cnt.cpu().numpy()[t] == min(k_e, prefix)
        ok, msg = O.topk_row_agrees(idx_e_h[t], ref_sc[t], prefix, k_e)
        assert ok, f"row {t}: {msg}"
    assert np.array_equal(idx_t_h, O.entry_expand(idx_e_h, q_pos0=L, entry_size=E))      # integer work: exact

    # page demand and attention on the expanded selection
    n_log = (S + page - 1) // page
    n_phys = n_log + 11
    table = rng.permutation(n_phys)[:n_log].astype(np.int32)
    pd = B.janus_page_demand(idx_t, demand_limit=L, page_size=page, page_table=dev(table, "i32"), n_phys_pages=n_phys)
    ref_pd = O.page_demand(idx_t_h, L, page, table)
    got = Hp.page_lists_from_device(pd)
    assert got["pages"] == ref_pd["pages"] and got["runs"] == ref_pd["runs"]
    Q = W.to_bf16_bits((rng.standard_normal((M, H_q, d_qk)) / 4).astype(np.float32))
    pools = [W.to_bf16_bits((rng.standard_normal((n_phys, page, 1, d_qk)) / 4).astype(np.float32)) for _ in range(2)]
    scale = 1.0 / np.sqrt(d_qk)
    for pool in pools:      # index reuse: the same selection serves the KV pools of two layers
        out, _ = B.janus_sparse_attn_prefill(dev(Q, "bf16"), dev(pool, "bf16"), dev(pool, "bf16"), idx_t, page_table=dev(table, "i32"),
                                             page_size=page, softmax_scale=scale, d_v=d_v)
        ref_o, _ = O.sparse_attention(Q, pool, pool, table, idx_t_h, page_size=page, softmax_scale=scale, d_qk=d_qk, d_v=d_v)
        Hp.assert_attention_close(Hp.bf16_tensor_to_f64(out), ref_o, "entry attention")
    B.check_dev_status()


def test_selecting_every_entry_is_dense_causal_attention():
    E, L, M = 32, 200, 40
    S = L + M
    n_entries = (S + E - 1) // E
    rng = np.random.default_rng(1)
    sc = torch.from_numpy(rng.standard_normal((M, (n_entries + 3) // 4 * 4)).astype(np.float32)).cuda()
    idx_e, _, _ = B.janus_topk_entries(sc, n_entries, n_entries, q_pos0=L, entry_size=E)
    idx_t = B.janus_entry_expand(idx_e, q_pos0=L, entry_size=E).cpu().numpy()
    for t in range(M):
        assert sorted(x for x in idx_t[t] if x >= 0) == list(range(L + t + 1))
    B.check_dev_status()


@pytest.mark.parametrize("E,L,M,k_e,dtype", [(128, 30000, 20, 12, "bf16"), (16, 2011, 33, 25, "fp8"), (64, 50, 70, 4, "bf16")])
def test_pooled_entry_scores_pipeline_matches_oracle(E, L, M, k_e, dtype):
    """The other reading of the entry footnote (Sec. 2.2): token scores from the ordinary indexer, an entry scores as the
    maximum over its visible tokens (janus_entry_pool_scores), then the same entry top-k and expansion."""
    rng = np.random.default_rng(7 * E + L)
    S = L + M
    n_entries = (S + E - 1) // E
    H, D = 64, 128
    qf, kf = rng.standard_normal((M, H, D)).astype(np.float32), rng.standard_normal((S, D)).astype(np.float32)
    w = (rng.uniform(0, 1, (M, H)) / 8).astype(np.float32)
    if dtype == "bf16":
        q, kk, qs, ks = W.to_bf16_bits(qf), W.to_bf16_bits(kf), None, None
    else:
        q, kk = W.to_e4m3_bits(2 * qf), W.to_e4m3_bits(2 * kf)
        qs, ks = np.exp2(rng.uniform(-2, 2, H)).astype(np.float32), np.exp2(rng.uniform(-1, 1, S)).astype(np.float32)
    sc = B.janus_indexer_scores(dev(q, dtype), dev(kk, dtype), dev(w, "f32"), q_scale=dev(qs, "f32"), k_scale=dev(ks, "f32"), q_pos0=L, causal=True)
    pooled = B.janus_entry_pool_scores(sc, S, entry_size=E, q_pos0=L, causal=True)
    idx_e, cnt, _ = B.janus_topk_entries(pooled, n_entries, k_e, q_pos0=L, entry_size=E)
    idx_t = B.janus_entry_expand(idx_e, q_pos0=L, entry_size=E)
    B.check_dev_status()
    # pooling is a maximum of fp32 values: exact on the library's own scores
    sc_h = sc[:, :S].cpu().numpy()
    want_pooled = O.entry_pool_scores(sc_h, entry_size=E, q_pos0=L, causal=True)
    assert np.array_equal(pooled[:, :n_entries].cpu().numpy().astype(np.float64), want_pooled)
    # against the oracle's own scores: entry selection within the 1e-3 band, expansion exact
    ref_sc = O.indexer_scores(q, kk, w, dtype=dtype, q_scale=qs, k_scale=ks, q_pos0=L, causal=True)
    ref_pooled = O.entry_pool_scores(ref_sc, entry_size=E, q_pos0=L, causal=True)
    idx_e_h = idx_e.cpu().numpy()
    for t in range(M):
        prefix = O.entry_visible_prefix(t, n_entries, L, E)
        assert cnt.cpu().numpy()[t] == min(k_e, prefix)
        ok, msg = O.topk_row_agrees(idx_e_h[t], ref_pooled[t], prefix, k_e)
        assert ok, f"row {t}: {msg}"
    assert np.array_equal(idx_t.cpu().numpy(), O.entry_expand(idx_e_h, q_pos0=L, entry_size=E))
    # non-causal pooling (the prediction pass over history keys only)
    nc = B.janus_entry_pool_scores(sc, L, entry_size=E, causal=False)
    assert np.array_equal(nc[:, :(L + E - 1) // E].cpu().numpy().astype(np.float64), O.entry_pool_scores(sc_h[:, :L], entry_size=E, causal=False))
    B.check_dev_status()
