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
