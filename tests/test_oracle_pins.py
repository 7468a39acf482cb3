"""Pins for the CPU oracle: closed forms, brute force, library routines on special cases,
hand-computed cases and the worked example the paper states in words (Sec. 4.3).
A dropped term, a wrong sign or index, or a transposed operand in the oracle fails one of these."""
import os

import numpy as np
import pytest
import torch

from oracle import janus_oracle as O
from paper_2609_36938_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16(x):
    return W.to_bf16_bits(np.asarray(x, dtype=np.float32))


# ------------------------------------------------------------------ formats
def test_decode_bf16_matches_torch():
    bits = np.arange(0, 65536, dtype=np.uint16)
    ref = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()
    got = O.decode_bf16(bits)
    both_nan = np.isnan(ref) & np.isnan(got)
    assert np.array_equal(got[~both_nan], ref[~both_nan])


def test_decode_e4m3_matches_torch_and_format_facts():
    codes = np.arange(256, dtype=np.uint8)
    ref = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    got = O.decode_e4m3(codes)
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan) and nan.sum() == 2
    assert np.array_equal(got[~nan], ref[~nan])
    assert got[0x7E] == 448.0 and got[0x01] == 2.0 ** -9 and got[0x38] == 1.0 and got[0xB8] == -1.0


def test_generator_rounding_roundtrip():
    rng = np.random.default_rng(0)
    x = rng.standard_normal(4096).astype(np.float32)
    b = W.to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(O.decode_bf16(b).astype(np.float32), ref)
    c = W.to_e4m3_bits(x * 100)
    assert np.all(np.abs(O.decode_e4m3(c)) <= 448.0)
    # nearest representable: error at most half a step of 2^(e-3) for normal values
    xs = np.clip(x * 100, -448, 448)
    err = np.abs(O.decode_e4m3(c) - xs)
    assert np.all(err <= np.maximum(2.0 ** (np.floor(np.log2(np.maximum(np.abs(xs), 2.0 ** -6))) - 4), 2.0 ** -10) + 1e-12)


# ------------------------------------------------------------------ indexer
def test_indexer_hand_computed_two_tokens_three_keys_two_heads():
    # q[t,h,:], k[s,:] in 2 dims; exact small integers (representable in bf16)
    q = np.array([[[1, 0], [0, -1]],
                  [[2, 1], [-1, 1]]], dtype=np.float32)
    k = np.array([[1, 1], [-2, 3], [0, -4]], dtype=np.float32)
    w = np.array([[0.5, 2.0], [1.0, -1.0]], dtype=np.float32)
    # dots t=0: h0: [1,-2,0]; h1: [-1,-3,4]  -> relu: [1,0,0], [0,0,4] -> 0.5*.. + 2*.. = [0.5, 0, 8]
    # dots t=1: h0: [3,-1,-4]; h1: [0,5,-4]  -> relu: [3,0,0], [0,5,0] -> 1*.. - 1*.. = [3, -5, 0]
    sc = O.indexer_scores(bf16(q), bf16(k), w, q_pos0=1, causal=True)
    # q_pos0=1: row 0 sees keys 0..1, row 1 sees 0..2
    assert np.array_equal(sc[0], np.array([0.5, 0.0, -np.inf]))
    assert np.array_equal(sc[1], np.array([3.0, -5.0, 0.0]))
    full = O.indexer_scores(bf16(q), bf16(k), w, causal=False)
    assert np.array_equal(full, np.array([[0.5, 0.0, 8.0], [3.0, -5.0, 0.0]]))


def test_indexer_single_head_positive_dots_is_a_matrix_product():
    rng = np.random.default_rng(1)
    q = np.abs(rng.standard_normal((5, 1, 16))).astype(np.float32)
    k = np.abs(rng.standard_normal((9, 16))).astype(np.float32)
    w = np.ones((5, 1), dtype=np.float32)
    sc = O.indexer_scores(bf16(q), bf16(k), w, causal=False)
    ref = np.matmul(O.decode_bf16(bf16(q))[:, 0, :], O.decode_bf16(bf16(k)).T)
    np.testing.assert_allclose(sc, ref, rtol=1e-14)
    # all dots negative -> exactly zero
    sc0 = O.indexer_scores(bf16(q), bf16(-k), w, causal=False)
    assert np.all(sc0 == 0.0)


def test_indexer_linear_in_w_and_key_scale_law():
    rng = np.random.default_rng(2)
    q = bf16(rng.standard_normal((4, 3, 8)))
    k = bf16(rng.standard_normal((7, 8)))
    w1 = rng.uniform(-1, 1, (4, 3)).astype(np.float32)
    w2 = rng.uniform(-1, 1, (4, 3)).astype(np.float32)
    a = O.indexer_scores(q, k, w1, causal=False)
    b = O.indexer_scores(q, k, w2, causal=False)
    ab = O.indexer_scores(q, k, (w1.astype(np.float64) + 2 * w2.astype(np.float64)), causal=False)
    np.testing.assert_allclose(ab, a + 2 * b, rtol=1e-12, atol=1e-12)
    # scaling key s by c>0 scales column s by c (the FP8 per-token scale law)
    ks = np.array([1, 2, 0.5, 4, 1, 8, 0.25])
    codes_q = W.to_e4m3_bits(np.round(rng.standard_normal((4, 3, 8)) * 4) / 4)
    codes_k = W.to_e4m3_bits(np.round(rng.standard_normal((7, 8)) * 4) / 4)
    base = O.indexer_scores(codes_q, codes_k, w1, dtype="fp8", causal=False)
    scaled = O.indexer_scores(codes_q, codes_k, w1, dtype="fp8", k_scale=ks, q_scale=np.ones(3), causal=False)
    np.testing.assert_allclose(scaled, base * ks[None, :], rtol=1e-12, atol=1e-12)


def test_indexer_fp8_unit_scales_equals_bf16_on_representable_values():
    rng = np.random.default_rng(3)
    qv = np.round(rng.standard_normal((3, 2, 8)) * 2) / 2    # multiples of 0.5: exact in both formats
    kv = np.round(rng.standard_normal((6, 8)) * 2) / 2
    w = rng.uniform(0, 1, (3, 2)).astype(np.float32)
    a = O.indexer_scores(bf16(qv), bf16(kv), w, dtype="bf16", causal=False)
    b = O.indexer_scores(W.to_e4m3_bits(qv), W.to_e4m3_bits(kv), w, dtype="fp8",
                         q_scale=np.ones(2, np.float32), k_scale=np.ones(6, np.float32), causal=False)
    assert np.array_equal(a, b)


def test_indexer_per_token_query_scales_hand_case_and_broadcast_axis():
    # FP8 queries with one scale per (token, head) (Sec. 5.1 storage; Eq. 1 scoring): the scale multiplies head h of token t.
    # Hand case, 2 tokens x 2 heads x 2 dims, 2 keys, every value exact in E4M3:
    q = np.array([[[1, 2], [2, -1]],
                  [[1, 2], [2, -1]]], dtype=np.float32)          # both tokens store the same codes: only the scales differ
    k = np.array([[1, 1], [1, -1]], dtype=np.float32)
    w = np.array([[1.0, 1.0], [1.0, 1.0]], dtype=np.float32)
    qs = np.array([[1.0, 2.0], [4.0, 0.5]])                      # qs[t, h]
    # code dots: h0: [3, -1]; h1: [1, 3]
    # t=0: scales (1, 2): relu([3,-1]) + relu([2, 6]) = [5, 6];  t=1: scales (4, 0.5): relu([12,-4]) + relu([0.5,1.5]) = [12.5, 1.5]
    sc = O.indexer_scores(W.to_e4m3_bits(q), W.to_e4m3_bits(k), w, dtype="fp8", q_scale=qs, k_scale=np.ones(2), causal=False)
    assert np.array_equal(sc, np.array([[5.0, 6.0], [12.5, 1.5]]))
    # a swapped broadcast axis would read qs[h, t]: (1, 4) for t=0 -> [3+4, 12] and fails the line above; check it is different
    assert not np.array_equal(sc, np.array([[7.0, 12.0], [6.5, 1.5]]))
    # a per-head vector repeated for every token is bit-identical to the 1-D call (non-square shape: a transposed use cannot broadcast)
    rng = np.random.default_rng(14)
    M, H, D, n = 5, 3, 8, 7
    cq = W.to_e4m3_bits(rng.standard_normal((M, H, D)))
    ck = W.to_e4m3_bits(rng.standard_normal((n, D)))
    wv = rng.uniform(-1, 1, (M, H)).astype(np.float32)
    per_head = (2.0 ** rng.uniform(-2, 2, H)).astype(np.float32)
    ks = (2.0 ** rng.uniform(-4, 4, n)).astype(np.float32)
    one_d = O.indexer_scores(cq, ck, wv, dtype="fp8", q_scale=per_head, k_scale=ks, q_pos0=2, causal=True)
    two_d = O.indexer_scores(cq, ck, wv, dtype="fp8", q_scale=np.tile(per_head, (M, 1)), k_scale=ks, q_pos0=2, causal=True)
    assert np.array_equal(one_d, two_d)
    # scaling one token's scale row by c > 0 scales exactly that token's score row (ReLU is positively homogeneous)
    qs2 = np.tile(per_head, (M, 1)).astype(np.float64)
    qs2[3] *= 4.0
    scaled = O.indexer_scores(cq, ck, wv, dtype="fp8", q_scale=qs2, k_scale=ks, causal=False)
    base = O.indexer_scores(cq, ck, wv, dtype="fp8", q_scale=per_head, k_scale=ks, causal=False)
    factor = np.ones((M, 1)); factor[3] = 4.0
    np.testing.assert_allclose(scaled, base * factor, rtol=1e-13, atol=0)
    # a scale on one head of one token equals that head's weight scaled instead (the scale sits outside the ReLU)
    qs3 = np.tile(per_head, (M, 1)).astype(np.float64)
    qs3[1, 2] *= 8.0
    w3 = wv.astype(np.float64).copy()
    w3[1, 2] *= 8.0
    np.testing.assert_allclose(O.indexer_scores(cq, ck, wv, dtype="fp8", q_scale=qs3, k_scale=ks, causal=False),
                               O.indexer_scores(cq, ck, w3, dtype="fp8", q_scale=per_head, k_scale=ks, causal=False), rtol=1e-13, atol=1e-300)


def test_indexer_mask_counts_and_self_inclusion():
    rng = np.random.default_rng(4)
    L, M = 5, 4
    q = bf16(rng.standard_normal((M, 2, 4)))
    k = bf16(rng.standard_normal((L + M, 4)))
    w = np.ones((M, 2), np.float32)
    sc = O.indexer_scores(q, k, w, q_pos0=L, causal=True)
    for t in range(M):
        assert np.isfinite(sc[t]).sum() == L + t + 1
        assert np.all(sc[t, L + t + 1:] == -np.inf)
    # zero history: the first token sees exactly itself
    sc0 = O.indexer_scores(q, k[:M], w, q_pos0=0, causal=True)
    assert np.isfinite(sc0[0]).sum() == 1


def test_indexer_bias_forms_agree_and_rows_subset():
    rng = np.random.default_rng(5)
    L, M = 40, 6
    q = bf16(rng.standard_normal((M, 2, 4)))
    k = bf16(rng.standard_normal((L + M, 4)))
    w = rng.uniform(0, 1, (M, 2)).astype(np.float32)
    t = np.arange(M)
    s = np.arange(L + M)
    rb = 2.0 * np.exp(-(L + t) / 16.0)
    cb = np.exp(s / 16.0)
    a = O.indexer_scores(q, k, w, q_pos0=L, recency=(2.0, 16.0))
    b = O.indexer_scores(q, k, w, q_pos0=L, row_bias=rb, col_bias=cb)
    fin = np.isfinite(a)
    np.testing.assert_allclose(a[fin], b[fin], rtol=1e-12)
    # the newest visible key gets exactly +amp
    plain = O.indexer_scores(q, k, w, q_pos0=L)
    np.testing.assert_allclose(a[t, L + t] - plain[t, L + t], 2.0, rtol=1e-12)
    sub = O.indexer_scores(q, k, w, q_pos0=L, recency=(2.0, 16.0), rows=[1, 4])
    assert np.array_equal(sub, a[[1, 4]])


# ------------------------------------------------------------------ top-k
def test_topk_against_brute_force_sort():
    rng = np.random.default_rng(6)
    for n, k in [(1, 1), (7, 3), (50, 50), (50, 64), (200, 17)]:
        sc = rng.standard_normal(n)
        sel, tau = O.topk_select(sc, n, k)
        brute = sorted(range(n), key=lambda i: (-sc[i], i))[:min(k, n)]
        assert list(sel) == brute
        assert tau == sc[brute[-1]]


def test_topk_special_cases():
    rng = np.random.default_rng(7)
    sc = rng.standard_normal(33)
    sel, _ = O.topk_select(sc, 33, 1)
    assert sel[0] == np.argmax(sc)
    sel, _ = O.topk_select(sc, 20, 64)                      # k >= prefix: whole prefix
    assert set(sel) == set(range(20))
    sel, _ = O.topk_select(np.ones(40), 40, 8)              # all equal: lowest indices
    assert list(sel) == list(range(8))
    a, _ = O.topk_select(sc, 33, 9)
    b, _ = O.topk_select(2 * sc + 1, 33, 9)                 # monotone transform keeps the set
    assert list(a) == list(b)


def test_topk_causal_block_and_padding():
    rng = np.random.default_rng(8)
    L, M, k = 6, 5, 8
    sc = rng.standard_normal((M, L + M))
    out = O.topk(sc, k, q_pos0=L, causal=True)
    for t in range(M):
        valid = out[t][out[t] >= 0]
        assert len(valid) == min(k, L + t + 1)
        assert valid.max() <= L + t
        assert np.all(out[t][len(valid):] == -1)


def test_topk_agreement_rule():
    sc = np.array([10.0, 9.0, 8.0, 8.0 * (1 - 5e-4), 1.0, 0.5])
    ok, _ = O.topk_row_agrees([0, 1, 2, -1], sc, 6, 3)
    assert ok
    ok, _ = O.topk_row_agrees([0, 1, 3], sc, 6, 3)          # inside the band around the 3rd score
    assert ok
    ok, msg = O.topk_row_agrees([0, 1, 4], sc, 6, 3)        # clearly below
    assert not ok
    ok, _ = O.topk_row_agrees([0, 2, 3], sc, 6, 3)          # misses a clear winner
    assert not ok
    ok, _ = O.topk_row_agrees([0, 0, 1], sc, 6, 3)          # duplicate
    assert not ok
    ok, _ = O.topk_row_agrees([0, 1, 5], sc, 5, 3)          # outside the prefix
    assert not ok


# ------------------------------------------------------------------ page demand
def _parse_golden():
    cases = []
    with open(os.path.join(GOLDEN, "read_packing_example.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, ids, runs = [p.strip() for p in line.split("|")]
            cases.append((name, [int(x) for x in ids.split()],
                          [tuple(int(v) for v in r.split(":")) for r in runs.split()]))
    return cases


@pytest.mark.parametrize("name,ids,runs", _parse_golden())
def test_read_packing_worked_examples(name, ids, runs):
    # page_size 1 and an identity table: token ids are block ids
    table = np.arange(64, dtype=np.int32)
    d = O.page_demand(np.array(ids)[None, :], 64, 1, table)
    assert d["pages"] == sorted(ids)
    assert d["runs"] == runs


def test_page_demand_hand_cases():
    pg = 4
    table = np.arange(8, dtype=np.int32)
    all_tokens = np.arange(32)[None, :]
    d = O.page_demand(all_tokens, 32, pg, table)
    assert d["pages"] == list(range(8)) and d["runs"] == [(0, 8)]
    # only history tokens (s < demand_limit) create demand; -1 is padding
    idx = np.array([[0, 1, 5, -1], [30, 31, 17, -1]])
    d = O.page_demand(idx, 20, pg, table)
    assert d["pages"] == [0, 1, 4] and d["runs"] == [(0, 2), (4, 1)]
    # alternating pages: as many runs as pages
    idx = np.array([[0, 8, 16, 24]])
    d = O.page_demand(idx, 32, pg, table)
    assert d["pages"] == [0, 2, 4, 6] and len(d["runs"]) == 4
    # a shuffled table keeps the page count and moves the runs
    sh = np.array([5, 0, 6, 2, 7, 1, 4, 3], dtype=np.int32)   # logical 0,2,4,6 -> physical 5,6,7,4
    d2 = O.page_demand(idx, 32, pg, sh)
    assert d2["pages"] == [4, 5, 6, 7] and d2["runs"] == [(4, 4)]


def test_page_demand_miss_set_is_set_difference_and_run_invariants():
    rng = np.random.default_rng(9)
    pg, n_pages = 8, 40
    table = rng.permutation(n_pages).astype(np.int32)
    L = pg * n_pages - 3
    for trial in range(20):
        idx = rng.integers(-1, L + 20, size=(6, 9))
        pidx = rng.integers(-1, L, size=(6, 9))
        pred = O.page_demand(pidx, L, pg, table)["pages"]
        d = O.page_demand(idx, L, pg, table, predicted_pages=pred)
        A = {int(table[s // pg]) for s in idx.reshape(-1) if 0 <= s < L}
        assert set(d["pages"]) == A and d["pages"] == sorted(A)
        assert set(d["miss"]) == A - set(pred)
        assert len(A) <= min(idx.size, n_pages)
        for runs, pages in ((d["runs"], d["pages"]), (d["miss_runs"], d["miss"])):
            assert sum(l for _, l in runs) == len(pages)
            covered = [p for a, l in runs for p in range(a, a + l)]
            assert covered == pages
            for (a0, l0), (a1, _) in zip(runs, runs[1:]):
                assert a0 + l0 < a1                       # ascending, disjoint, not adjacent
    full = O.page_demand(idx, L, pg, table, predicted_pages=range(n_pages))
    assert full["miss"] == [] and full["miss_runs"] == []
    none = O.page_demand(idx, L, pg, table, predicted_pages=[])
    assert none["miss"] == none["pages"]


def test_recall_precision():
    r, p = O.recall_precision([1, 2, 3, 4], [3, 4, 5])
    assert r == pytest.approx(2 / 3) and p == pytest.approx(0.5)
    assert O.recall_precision([], []) == (1.0, 1.0)


# ------------------------------------------------------------------ sparse attention
def _paged(K, V, page_size, table):
    """Scatter contiguous K [S,Hkv,d], V into paged pools through ``table``."""
    S, Hkv, dk = K.shape
    dv = V.shape[2]
    n_log = (S + page_size - 1) // page_size
    n_phys = int(max(table)) + 1
    kp = np.zeros((n_phys, page_size, Hkv, dk), dtype=np.uint16)
    vp = np.zeros((n_phys, page_size, Hkv, dv), dtype=np.uint16)
    for s in range(S):
        kp[table[s // page_size], s % page_size] = K[s]
        vp[table[s // page_size], s % page_size] = V[s]
    return kp, vp


def _small_attention_case(seed, L=9, M=5, H=4, Hkv=2, dk=8, dv=6, pg=4, shuffled=True):
    rng = np.random.default_rng(seed)
    S = L + M
    Q = bf16(rng.standard_normal((M, H, dk)))
    K = bf16(rng.standard_normal((S, Hkv, dk)))
    V = bf16(rng.standard_normal((S, Hkv, dv)))
    n_log = (S + pg - 1) // pg
    table = rng.permutation(n_log).astype(np.int32) if shuffled else np.arange(n_log, dtype=np.int32)
    kp, vp = _paged(K, V, pg, table)
    return Q, K, V, kp, vp, table


def test_sparse_attention_with_full_selection_equals_dense_causal():
    L, M, pg = 9, 5, 4
    Q, K, V, kp, vp, table = _small_attention_case(10, L=L, M=M, pg=pg)
    S = L + M
    idx = np.full((M, S), -1, dtype=np.int64)
    for t in range(M):
        idx[t, :L + t + 1] = np.arange(L + t + 1)
    out, lse = O.sparse_attention(Q, kp, vp, table, idx, page_size=pg, softmax_scale=0.7, d_qk=8, d_v=6)
    dense = O.dense_causal_attention(O.decode_bf16(Q), O.decode_bf16(K), O.decode_bf16(V), softmax_scale=0.7, q_pos0=L)
    np.testing.assert_allclose(out, dense, rtol=1e-12, atol=1e-13)
    # library cross-check: torch SDPA in fp64 with an explicit causal mask, kv heads expanded
    Qt = torch.from_numpy(O.decode_bf16(Q)).permute(1, 0, 2)[None]           # [1,H,M,dk]
    Kt = torch.from_numpy(O.decode_bf16(K)).permute(1, 0, 2).repeat_interleave(2, 0)[None]
    Vt = torch.from_numpy(O.decode_bf16(V)).permute(1, 0, 2).repeat_interleave(2, 0)[None]
    mask = torch.arange(S)[None, :] <= (L + torch.arange(M))[:, None]
    ref = torch.nn.functional.scaled_dot_product_attention(Qt, Kt, Vt, attn_mask=mask, scale=0.7)
    np.testing.assert_allclose(out, ref[0].permute(1, 0, 2).numpy(), rtol=1e-10, atol=1e-12)
    # lse = log sum exp of the logits
    logit = 0.7 * (O.decode_bf16(K)[:L + 1, 0] @ O.decode_bf16(Q)[0, 0])
    assert lse[0, 0] == pytest.approx(np.log(np.exp(logit).sum()), rel=1e-12)


def test_sparse_attention_special_selections():
    L, M, pg = 9, 5, 4
    Q, K, V, kp, vp, table = _small_attention_case(11, L=L, M=M, pg=pg)
    Vd = O.decode_bf16(V)
    # a single selected key: output is exactly its V row (per kv head)
    idx = np.full((M, 3), -1, dtype=np.int64)
    idx[:, 1] = [3, 0, 7, 9, 2]
    out, _ = O.sparse_attention(Q, kp, vp, table, idx, page_size=pg, softmax_scale=1.0, d_qk=8, d_v=6)
    for t in range(M):
        for h in range(4):
            assert np.array_equal(out[t, h], Vd[idx[t, 1], h // 2])
    # permuting the selection leaves the output unchanged; empty selection gives zeros / -inf
    rng = np.random.default_rng(12)
    idx = np.stack([rng.permutation(L)[:6] for _ in range(M)])
    a, la = O.sparse_attention(Q, kp, vp, table, idx, page_size=pg, softmax_scale=0.5, d_qk=8, d_v=6)
    b, lb = O.sparse_attention(Q, kp, vp, table, idx[:, ::-1], page_size=pg, softmax_scale=0.5, d_qk=8, d_v=6)
    np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-14)
    e, le = O.sparse_attention(Q, kp, vp, table, np.full((M, 4), -1), page_size=pg, softmax_scale=0.5, d_qk=8, d_v=6)
    assert np.all(e == 0) and np.all(le == -np.inf)


def test_sparse_attention_identical_keys_average_values_and_shift_invariance():
    rng = np.random.default_rng(13)
    S, H, dk, dv, pg = 12, 2, 8, 4, 4
    Q = bf16(rng.standard_normal((3, H, dk)))
    krow = rng.standard_normal((1, 1, dk))
    K = bf16(np.repeat(krow, S, axis=0))
    V = bf16(rng.standard_normal((S, 1, dv)))
    table = np.array([2, 0, 1], dtype=np.int32)
    kp, vp = _paged(K, V, pg, table)
    idx = np.array([[0, 5, 11, 7], [1, 2, 3, -1], [4, -1, -1, -1]])
    out, _ = O.sparse_attention(Q, kp, vp, table, idx, page_size=pg, softmax_scale=1.3, d_qk=dk, d_v=dv)
    Vd = O.decode_bf16(V)
    np.testing.assert_allclose(out[0, 0], Vd[[0, 5, 11, 7], 0].mean(axis=0), rtol=1e-12)
    np.testing.assert_allclose(out[1, 1], Vd[[1, 2, 3], 0].mean(axis=0), rtol=1e-12)
    # adding to Q a direction on which all keys agree shifts every logit equally: output unchanged
    K2 = rng.standard_normal((S, 1, dk))
    K2[:, :, 0] = 1.0                                         # every key has the same first coordinate
    K2 = bf16(K2)
    kp2, vp2 = _paged(K2, V, pg, table)
    Qa = O.decode_bf16(Q).copy()
    Qb = Qa.copy()
    Qb[:, :, 0] += 4.0
    a, _ = O.sparse_attention(bf16(Qa), kp2, vp2, table, idx, page_size=pg, softmax_scale=1.0, d_qk=dk, d_v=dv)
    b, _ = O.sparse_attention(bf16(Qb), kp2, vp2, table, idx, page_size=pg, softmax_scale=1.0, d_qk=dk, d_v=dv)
    np.testing.assert_allclose(a, b, rtol=1e-9, atol=1e-12)


def test_sparse_attention_page_table_relabeling_and_latent_value_prefix():
    L, M, pg = 9, 5, 4
    rng = np.random.default_rng(14)
    Q, K, V, kp_id, vp_id, t_id = _small_attention_case(15, L=L, M=M, pg=pg, shuffled=False)
    table = np.array([3, 1, 0, 2], dtype=np.int32)
    kp_sh, vp_sh = _paged(K, V, pg, table)
    idx = np.stack([rng.permutation(L)[:5] for _ in range(M)])
    a, _ = O.sparse_attention(Q, kp_id, vp_id, t_id, idx, page_size=pg, softmax_scale=0.4, d_qk=8, d_v=6)
    b, _ = O.sparse_attention(Q, kp_sh, vp_sh, table, idx, page_size=pg, softmax_scale=0.4, d_qk=8, d_v=6)
    assert np.array_equal(a, b)
    # latent layout: values are the first d_v dims of the key row (v_pool aliases k_pool)
    c, _ = O.sparse_attention(Q, kp_id[:, :, :1], kp_id[:, :, :1], t_id, idx, page_size=pg, softmax_scale=0.4, d_qk=8, d_v=6)
    Kd = O.decode_bf16(K)
    for t in range(M):
        logit = 0.4 * (Kd[idx[t], 0] @ O.decode_bf16(Q)[t, 3])
        p = np.exp(logit - logit.max())
        np.testing.assert_allclose(c[t, 3], (p / p.sum()) @ Kd[idx[t], 0, :6], rtol=1e-12)


# ------------------------------------------------------------------ generator facts the tests rely on
def test_workload_shapes_and_determinism():
    shp = W.config_shape(1, L=128, M=16, k=8)
    a = W.make_session(shp, seed=0)
    b = W.make_session(shp, seed=0)
    c = W.make_session(shp, seed=1)
    assert a["q_idx"].shape == (16, 4, 64) and a["k_idx"].shape == (144, 64) and a["q_idx"].dtype == np.uint16
    assert np.array_equal(a["q_idx"], b["q_idx"]) and not np.array_equal(a["q_idx"], c["q_idx"])
    assert a["k_pool"].shape == (3, 64, 8, 128) and a["q_pred"].shape == a["q_idx"].shape
    s3 = W.make_session(W.config_shape(3, L=256, M=8, k=16), seed=0)
    assert s3["q_idx"].dtype == np.uint8 and s3["k_scale"].shape == (264,) and s3["q_scale"].shape == (64,)
    assert sorted(s3["page_table"].tolist()) == list(range(5))
    assert s3["k_pool"] is s3["v_pool"] and s3["k_pool"].shape == (5, 64, 1, 576)
    s5 = W.make_session(W.config_shape(5, L=4096, M=8, k=16), seed=0, with_attention=False)
    assert s5["row_bias"].shape == (8,) and s5["col_bias"].shape == (4104,)
    shapes = W.batch_shapes(0)
    assert len(shapes) == 8 and all(16384 <= s.L <= 204800 and 512 <= s.M <= 8192 for s in shapes)
    tabs, n_phys = W.fragmented_page_tables(shapes[:3], 0)
    allp = np.concatenate(tabs)
    assert len(np.unique(allp)) == len(allp) == n_phys


# ---- entry granularity ------------------------------------------------------------------------------------------------
def test_entry_selection_of_all_entries_expands_to_the_causal_prefix():
    # selecting every visible entry must give exactly the tokens 0 .. pos of each row (so that attention over the expansion
    # is dense causal attention), whatever the entry size and wherever the row sits inside its entry
    for E, L, M in ((4, 10, 7), (8, 16, 9), (3, 0, 5), (16, 5, 3)):
        n_entries = (L + M + E - 1) // E
        scores = np.random.default_rng(E).standard_normal((M, n_entries))
        sel = O.entry_topk(scores, n_entries, q_pos0=L, entry_size=E)
        tok = O.entry_expand(sel, q_pos0=L, entry_size=E)
        for t in range(M):
            assert sorted(x for x in tok[t] if x >= 0) == list(range(L + t + 1))
            assert O.entry_visible_prefix(t, n_entries, L, E) == (L + t) // E + 1


def test_entry_topk_hand_case_and_unit_entries():
    # E = 1 is token granularity: same selection as the token top-k
    rng = np.random.default_rng(9)
    sc = rng.standard_normal((6, 30))
    assert np.array_equal(O.entry_topk(sc, 5, q_pos0=20, entry_size=1), O.topk(sc, 5, q_pos0=20, causal=True))
    # hand case: E = 4, query at position 9 sees entries 0, 1, 2 (tokens 0..9); the best two of [0.5, 2.0, 1.0, 9.0] among
    # the visible three are entries 1 and 2; their expansion drops tokens 10, 11 of entry 2
    sel = O.entry_topk(np.array([[0.5, 2.0, 1.0, 9.0]]), 2, q_pos0=9, entry_size=4)
    assert sel.tolist() == [[1, 2]]
    assert O.entry_expand(sel, q_pos0=9, entry_size=4).tolist() == [[4, 5, 6, 7, 8, 9, -1, -1]]


# ---- FP4 keys -----------------------------------------------------------------------------------------------------------
def test_e2m1_decode_table_and_packing_order():
    # the sixteen codes against the format's definition written out by hand
    want = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0, -0.0, -0.5, -1.0, -1.5, -2.0, -3.0, -4.0, -6.0]
    packed = np.array([[(2 * i) | ((2 * i + 1) << 4) for i in range(8)]], dtype=np.uint8)     # codes 0..15 in element order
    got = O.decode_e2m1(packed)[0]
    assert got.tolist() == want and np.signbit(got[8])
    # every E2M1 value is an E4M3 value: FP4 keys and the same numbers stored as FP8 must score identically
    rng = np.random.default_rng(4)
    codes = rng.integers(0, 16, size=(50, 32)).astype(np.uint8)
    packed = (codes[:, 0::2] | (codes[:, 1::2] << 4)).astype(np.uint8)
    vals = O.decode_e2m1(packed)
    import torch
    k8 = torch.from_numpy(vals.astype(np.float32)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(O.decode_e4m3(k8), vals)
    q = rng.integers(0, 120, size=(3, 4, 32)).astype(np.uint8)
    w = rng.uniform(0, 1, (3, 4)).astype(np.float32)
    qs, ks = rng.uniform(0.5, 2, 4).astype(np.float32), rng.uniform(0.5, 2, 50).astype(np.float32)
    a = O.indexer_scores(q, packed, w, dtype="fp8+fp4k", q_scale=qs, k_scale=ks, causal=False)
    b = O.indexer_scores(q, k8, w, dtype="fp8", q_scale=qs, k_scale=ks, causal=False)
    assert np.array_equal(a, b)


def test_entry_pooled_scores_hand_case_and_invariants():
    # pooled reading of the entry footnote (Sec. 2.2): an entry scores as its best visible token
    sc = np.array([[1.0, 5.0, -2.0, 0.5, 9.0, 3.0, 7.0],
                   [4.0, -1.0, 6.0, 2.0, 8.0, 0.0, -3.0]])
    # E = 3, q_pos0 = 3: row 0 sees tokens 0..3, row 1 sees 0..4
    got = O.entry_pool_scores(sc, entry_size=3, q_pos0=3, causal=True)
    assert np.array_equal(got, np.array([[5.0, 0.5, -np.inf], [6.0, 8.0, -np.inf]]))
    # not causal: every token counts, the last entry is partial
    assert np.array_equal(O.entry_pool_scores(sc, entry_size=3, causal=False), np.array([[5.0, 9.0, 7.0], [6.0, 8.0, -3.0]]))
    # E = 1 is the token score itself on the visible prefix
    rng = np.random.default_rng(31)
    r = rng.standard_normal((5, 23))
    one = O.entry_pool_scores(r, entry_size=1, q_pos0=10, causal=True)
    for t in range(5):
        assert np.array_equal(one[t, :11 + t], r[t, :11 + t]) and np.all(np.isneginf(one[t, 11 + t:]))
    # the best entry holds the best visible token; the number of finite entries is the number of entries with a visible token
    E = 4
    pooled = O.entry_pool_scores(r, entry_size=E, q_pos0=10, causal=True)
    for t in range(5):
        prefix = 11 + t
        assert int(np.argmax(pooled[t])) == int(np.argmax(r[t, :prefix])) // E
        assert np.isfinite(pooled[t]).sum() == O.entry_visible_prefix(t, pooled.shape[1], 10, E)
    # brute force: a sorted copy of each entry's visible tokens ends with the pooled value
    for t in range(5):
        for e in range(pooled.shape[1]):
            vis = [r[t, s] for s in range(e * E, min((e + 1) * E, 23)) if s <= 10 + t]
            assert pooled[t, e] == (sorted(vis)[-1] if vis else -np.inf)
