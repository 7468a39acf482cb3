"""GPU parity tests: every library call, through the C ABI, against the CPU oracle on the same seeded inputs.
Sizes span several tiles with ragged tails; edge cases (empty, M=1, zero history, prefix < k, ties) are included.

Tolerances.  Integer outputs (pages, runs, miss sets, selections on exact fp32 scores) are compared exactly.
Indexer scores: the products of bf16 / E4M3 operands are exact in fp32 and the kernels accumulate in fp32, so the
error is a few fp32 roundings of sums of up to D_I*H_I terms: 1e-4 of max(|score|, row rms) is asserted, far inside
the 1e-2 (bf16) / 5e-2 (FP8) acceptance bounds.  Attention: outputs are rounded to bf16 (2^-9 relative) and P is bf16
in tensor-core kernels; bounds are max-abs 2e-2 / mean-abs 2e-3 plus 2e-2 of max|o| and 1e-2 of mean|o|."""
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


# ------------------------------------------------------------------------------------------------ page demand
def _run_page_demand(idx_np, demand_limit, pg, table_np, n_phys, pred_idx_np=None, capacity=None):
    idx = dev(idx_np, "i32")
    table = dev(table_np, "i32")
    pred_bitmap = None
    pred_pages = None
    if pred_idx_np is not None:
        po = B.janus_page_demand(dev(pred_idx_np, "i32"), demand_limit=demand_limit, page_size=pg, page_table=table,
                                 n_phys_pages=n_phys, want_miss=False)
        pred_bitmap = po["bitmap"]
        pred_pages = O.page_demand(pred_idx_np, demand_limit, pg, table_np)["pages"]
        assert Hp.bitmap_to_pages(pred_bitmap, n_phys) == pred_pages
    out = B.janus_page_demand(idx, demand_limit=demand_limit, page_size=pg, page_table=table, n_phys_pages=n_phys,
                              predicted_bitmap=pred_bitmap, capacity=capacity)
    got = Hp.page_lists_from_device(out)
    ref = O.page_demand(idx_np, demand_limit, pg, table_np, predicted_pages=pred_pages)
    return got, ref, out


@pytest.mark.parametrize("n_rows,k,L,pg,n_extra,shuffle", [
    (1, 1, 10, 4, 0, False), (7, 13, 1000, 64, 50, True), (64, 256, 40000, 64, 300, True), (33, 100, 5000, 1, 0, True),
    (16, 64, 3000, 48, 100, True), (5, 3, 63, 64, 0, False),
])
def test_page_demand_matches_oracle(n_rows, k, L, pg, n_extra, shuffle):
    rng = np.random.default_rng(100 + n_rows)
    S = L + n_extra
    n_log = (S + pg - 1) // pg
    n_phys = n_log + 7
    table = (rng.permutation(n_phys)[:n_log] if shuffle else np.arange(n_log)).astype(np.int32)
    idx = rng.integers(-1, S, size=(n_rows, k)).astype(np.int32)
    pidx = rng.integers(-1, L, size=(n_rows, max(1, k // 2))).astype(np.int32)
    got, ref, out = _run_page_demand(idx, L, pg, table, n_phys, pred_idx_np=pidx)
    B.check_dev_status()
    assert got["pages"] == ref["pages"]
    assert got["runs"] == ref["runs"]
    assert got["miss"] == ref["miss"]
    assert got["miss_runs"] == ref["miss_runs"]
    assert Hp.bitmap_to_pages(out["bitmap"], n_phys) == ref["pages"]


def test_page_demand_edge_cases():
    table = np.arange(40, dtype=np.int32)
    # nothing selected
    got, ref, _ = _run_page_demand(np.full((4, 8), -1, np.int32), 1000, 64, table, 40)
    assert got == {"pages": [], "runs": [], "miss": [], "miss_runs": []} and ref["pages"] == []
    # everything selected, identity table: one run; no prediction: miss = demand
    got, ref, _ = _run_page_demand(np.arange(2560, dtype=np.int32).reshape(40, 64), 2560, 64, table, 40)
    assert got["pages"] == list(range(40)) and got["runs"] == [(0, 40)] and got["miss_runs"] == [(0, 40)]
    # new tokens (s >= demand_limit) create no demand; the page straddling the limit counts if a history token in it is selected
    idx = np.array([[100, 130, 127, 128]], dtype=np.int32)
    got, ref, _ = _run_page_demand(idx, 128, 64, table, 40)
    assert got["pages"] == ref["pages"] == [1]
    # a word boundary inside a run, and a run ending at the last page
    idx = (np.array([[30, 31, 32, 33, 39]], dtype=np.int32) * 64)
    got, ref, _ = _run_page_demand(idx, 2560, 64, table, 40)
    assert got["runs"] == ref["runs"] == [(30, 4), (39, 1)]
    B.check_dev_status()


def test_page_demand_large_pool_uses_global_bitmap_and_reports_conditions():
    rng = np.random.default_rng(5)
    n_phys = 300000                       # more pages than the shared-memory bitmap holds
    n_log = 4096
    table = rng.choice(n_phys, size=n_log, replace=False).astype(np.int32)
    idx = rng.integers(0, n_log * 16, size=(64, 128)).astype(np.int32)
    got, ref, _ = _run_page_demand(idx, n_log * 16, 16, table, n_phys)
    assert got["pages"] == ref["pages"] and got["runs"] == ref["runs"]
    B.check_dev_status()
    # capacity smaller than the lists: counts stay true, status says so
    out = B.janus_page_demand(dev(idx, "i32"), demand_limit=n_log * 16, page_size=16, page_table=dev(table, "i32"),
                              n_phys_pages=n_phys, capacity=10)
    assert int(out["counts"][0]) == len(ref["pages"])
    assert out["pages"][:10].cpu().tolist() == ref["pages"][:10]
    with pytest.raises(B.JanusError, match="CAPACITY"):
        B.check_dev_status()
    # an index beyond the page table is skipped and reported
    bad = idx.copy()
    bad[0, 0] = n_log * 16 + 5
    out = B.janus_page_demand(dev(bad, "i32"), demand_limit=n_log * 16 + 100, page_size=16, page_table=dev(table, "i32"),
                              n_phys_pages=n_phys)
    with pytest.raises(B.JanusError, match="INDEX_OUT_OF_RANGE"):
        B.check_dev_status()


def test_page_demand_chunked_lists_long_runs_and_miss_set():
    # a pool large enough for the list kernel that works in 1024-word chunks (32768 pages each): one run of adjacent pages
    # crosses word and chunk boundaries, scattered pages follow, and the miss set is taken against a predicted half
    rng = np.random.default_rng(21)
    pg, n_phys = 16, 110000
    table = np.arange(n_phys, dtype=np.int32)                      # identity: physical adjacency = logical adjacency
    run = np.arange(100, 70000)                                      # pages 100 .. 69999, crosses pages 32768 and 65536
    scattered = rng.choice(np.arange(70010, n_phys), size=3000, replace=False)
    pages_sel = np.concatenate([run, scattered])
    toks = pages_sel * pg + rng.integers(0, pg, size=pages_sel.size)
    pad = (-toks.size) % 128
    idx = np.concatenate([toks, np.full(pad, -1)]).astype(np.int32).reshape(-1, 128)
    rng.shuffle(idx, axis=0)
    pred_pages = np.concatenate([run[::2], scattered[: 1500]])
    pred = np.concatenate([pred_pages * pg, np.full((-pred_pages.size) % 64, -1)]).astype(np.int32).reshape(-1, 64)
    got, ref, out = _run_page_demand(idx, n_phys * pg, pg, table, n_phys, pred_idx_np=pred)
    B.check_dev_status()
    assert got["pages"] == ref["pages"] and len(got["pages"]) == pages_sel.size
    assert got["runs"] == ref["runs"] and got["runs"][0] == (100, 69900)
    assert got["miss"] == ref["miss"]
    assert got["miss_runs"] == ref["miss_runs"]


def test_page_demand_is_deterministic():
    rng = np.random.default_rng(6)
    table = rng.permutation(2112).astype(np.int32)
    idx = dev(rng.integers(0, 2112 * 64, size=(512, 2048)).astype(np.int32), "i32")
    a = B.janus_page_demand(idx, demand_limit=131072, page_size=64, page_table=dev(table, "i32"), n_phys_pages=2112)
    b = B.janus_page_demand(idx, demand_limit=131072, page_size=64, page_table=dev(table, "i32"), n_phys_pages=2112)
    for key in ("bitmap", "counts"):
        assert torch.equal(a[key], b[key])
    n = int(a["counts"][0])
    assert torch.equal(a["pages"][:n], b["pages"][:n])


# ------------------------------------------------------------------------------------------------ top-k
def _check_topk_exact(scores_np, idx_gpu, count_gpu, kth_gpu, k, q_pos0, causal):
    M, n_keys = scores_np.shape
    for t in range(M):
        prefix = O.visible_prefix(t, n_keys, q_pos0, causal)
        row = scores_np[t].astype(np.float64)
        got = idx_gpu[t]
        ok, msg = O.topk_row_agrees(got, row, prefix, k, band_rel=0.0)
        assert ok, f"row {t}: {msg}"
        n = min(k, prefix)
        assert count_gpu[t] == n
        valid = got[got >= 0]
        if n > 0:
            _, tau = O.topk_select(row, prefix, k)
            # exact: everything above the threshold is in, nothing below it is
            assert set(np.nonzero(row[:prefix] > tau)[0]) <= set(valid.tolist()), f"row {t}"
            assert np.all(row[valid] >= tau), f"row {t}"
            assert kth_gpu[t] == np.float32(tau), f"row {t}"
        else:
            assert kth_gpu[t] == -np.inf


def _run_topk(scores_np, k, q_pos0, causal):
    M, n_keys = scores_np.shape
    ld = (n_keys + 31) // 32 * 32
    buf = torch.full((M, ld), float("nan"), dtype=torch.float32, device="cuda")   # poison the padding
    buf[:, :n_keys] = torch.from_numpy(scores_np).cuda()
    idx, count, kth = B.janus_topk(buf, n_keys, k, q_pos0=q_pos0, causal=causal)
    return idx.cpu().numpy(), count.cpu().numpy(), kth.cpu().numpy()


@pytest.mark.parametrize("M,n_keys,k,q_pos0,causal", [
    (5, 37, 8, 32, True), (3, 1000, 1, 0, False), (9, 5000, 256, 4991, True), (4, 20000, 2048, 0, False),
    (6, 70001, 2048, 69995, True), (2, 140003, 2048, 0, False), (3, 13000, 12500, 0, False), (4, 300, 512, 0, False),
    (1, 1, 4, 0, True),
])
def test_topk_gaussian_rows(M, n_keys, k, q_pos0, causal):
    rng = np.random.default_rng(M * 1000 + k)
    sc = (18.0 + 2.5 * rng.standard_normal((M, n_keys))).astype(np.float32)
    idx, count, kth = _run_topk(sc, k, q_pos0, causal)
    _check_topk_exact(sc, idx, count, kth, k, q_pos0, causal)


def test_topk_adversarial_distributions():
    rng = np.random.default_rng(77)
    n, k = 50000, 2048
    rows = [
        np.ones(n),                                               # all equal
        np.arange(n, dtype=np.float64),                           # ascending: the sample underestimates nothing, but ties none
        np.arange(n, dtype=np.float64)[::-1].copy(),              # descending
        np.where(rng.random(n) < 0.5, 3.0, rng.standard_normal(n)),   # half the row is one value
        np.concatenate([np.full(n - 100, -1e30), rng.standard_normal(100)]),  # almost everything tiny: fewer distinct winners than k
        rng.standard_normal(n) * np.repeat(rng.uniform(0.1, 30, n // 500), 500),   # segments of very different scale
        np.where(np.arange(n) % 7 == 0, np.inf, rng.standard_normal(n)),       # infinities
        -np.abs(rng.standard_normal(n)) * 1e-30,                  # denormal-ish negatives
        np.round(rng.standard_normal(n) * 4) / 4,                 # heavy ties everywhere
    ]
    sc = np.stack(rows).astype(np.float32)
    idx, count, kth = _run_topk(sc, k, 0, False)
    _check_topk_exact(sc, idx, count, kth, k, 0, False)


def test_topk_zero_history_and_single_token():
    rng = np.random.default_rng(78)
    sc = rng.standard_normal((6, 6)).astype(np.float32)
    idx, count, kth = _run_topk(sc, 4, 0, True)              # zero history: row t sees t+1 keys
    _check_topk_exact(sc, idx, count, kth, 4, 0, True)
    sc = rng.standard_normal((1, 30000)).astype(np.float32)  # decode-like: a single token
    idx, count, kth = _run_topk(sc, 512, 29999, True)
    _check_topk_exact(sc, idx, count, kth, 512, 29999, True)


# ------------------------------------------------------------------------------------------------ indexer
def _indexer_case(seed, M, n_keys, H, D, dtype, q_pos0, causal, bias=False, per_token_qscale=False):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((M, H, D)).astype(np.float32)
    kk = rng.standard_normal((n_keys, D)).astype(np.float32)
    w = rng.uniform(-0.2, 1.0, (M, H)).astype(np.float32)
    c = {"w": w, "dtype": dtype, "q_scale": None, "k_scale": None, "row_bias": None, "col_bias": None}
    if dtype == "bf16":
        c["q"], c["k"] = W.to_bf16_bits(q), W.to_bf16_bits(kk)
    else:
        c["q"], c["k"] = W.to_e4m3_bits(q * 3), W.to_e4m3_bits(kk * 3)
        c["q_scale"] = np.exp2(rng.uniform(-2, 2, (M, H) if per_token_qscale else (H,))).astype(np.float32)
        c["k_scale"] = np.exp2(rng.uniform(-4, 4, n_keys)).astype(np.float32)
    if bias:
        c["row_bias"] = rng.uniform(0.5, 2.0, M).astype(np.float32)
        c["col_bias"] = rng.uniform(-1.0, 1.0, n_keys).astype(np.float32)
    return c


def _run_indexer(c, q_pos0, causal):
    kind = c["dtype"]
    sc = B.janus_indexer_scores(dev(c["q"], kind), dev(c["k"], kind), dev(c["w"], "f32"), q_scale=dev(c["q_scale"], "f32"),
                                k_scale=dev(c["k_scale"], "f32"), row_bias=dev(c["row_bias"], "f32"), col_bias=dev(c["col_bias"], "f32"),
                                q_pos0=q_pos0, causal=causal)
    n_keys = c["k"].shape[0]
    return sc[:, :n_keys].cpu().numpy()


@pytest.mark.parametrize("M,n_keys,H,D,dtype,q_pos0,causal,bias,ptq", [
    # tensor-core shapes: several key tiles, ragged key and token tails, the diagonal inside a tile
    (37, 128 * 5 + 37, 64, 128, "bf16", 128 * 5, True, False, False),
    (9, 1500, 64, 128, "bf16", 0, False, True, False),
    (37, 128 * 5 + 37, 64, 128, "fp8", 128 * 5, True, True, False),
    (20, 777, 64, 128, "fp8", 0, False, False, True),
    (130, 128 * 3 + 130, 4, 64, "bf16", 128 * 3, True, False, False),
    (70, 900, 16, 128, "bf16", 830, True, True, False),
    (33, 700, 32, 128, "fp8", 667, True, False, False),
    (600, 9000, 8, 64, "bf16", 8400, True, False, False),
    (1, 300, 64, 128, "bf16", 299, True, False, False),            # decode-like: one token
    (16, 16, 64, 128, "bf16", 0, True, False, False),              # zero history
    # general kernel: head counts / dims the tensor-core kernel does not take
    (11, 300, 3, 48, "bf16", 289, True, True, False),
    (5, 200, 5, 32, "fp8", 0, False, False, True),
])
def test_indexer_scores_match_oracle(M, n_keys, H, D, dtype, q_pos0, causal, bias, ptq):
    c = _indexer_case(M * 7 + H, M, n_keys, H, D, dtype, q_pos0, causal, bias, ptq)
    got = _run_indexer(c, q_pos0, causal)
    B.check_dev_status()
    ref = O.indexer_scores(c["q"], c["k"], c["w"], dtype=dtype, q_scale=c["q_scale"], k_scale=c["k_scale"], row_bias=c["row_bias"],
                           col_bias=c["col_bias"], q_pos0=q_pos0, causal=causal)
    Hp.assert_scores_close(got, ref, 1e-4, f"{dtype} H={H} D={D}")


def test_indexer_many_key_chunks_and_token_groups():
    # enough tiles that one token group is split over several CTAs and the ring wraps many times
    M, n_keys, q_pos0 = 40, 128 * 150 + 5, 128 * 150 - 35
    for dtype in ("bf16", "fp8"):
        c = _indexer_case(9, M, n_keys, 64, 128, dtype, q_pos0, True, True, False)
        got = _run_indexer(c, q_pos0, True)
        B.check_dev_status()
        rows = [0, 7, 8, 15, 16, 31, 39]
        ref = O.indexer_scores(c["q"], c["k"], c["w"], dtype=dtype, q_scale=c["q_scale"], k_scale=c["k_scale"], row_bias=c["row_bias"],
                               col_bias=c["col_bias"], q_pos0=q_pos0, causal=True, rows=rows)
        Hp.assert_scores_close(got[rows], ref, 1e-4, dtype)


# ------------------------------------------------------------------------------------------------ sparse attention
def _attention_case(seed, M, S, H_q, n_kv, d_qk, d_v, pg, k, latent, value_scale=1.0):
    rng = np.random.default_rng(seed)
    n_log = (S + pg - 1) // pg
    n_phys = n_log + 3
    table = rng.permutation(n_phys)[:n_log].astype(np.int32)
    Q = W.to_bf16_bits(rng.standard_normal((M, H_q, d_qk)).astype(np.float32) * value_scale)
    kp = W.to_bf16_bits(rng.standard_normal((n_phys, pg, n_kv, d_qk)).astype(np.float32) * value_scale)
    vp = kp if latent else W.to_bf16_bits(rng.standard_normal((n_phys, pg, n_kv, d_v)).astype(np.float32) * value_scale)
    idx = np.full((M, k), -1, dtype=np.int32)
    for t in range(M):
        n = min(k, S)
        n = n if t % 3 else max(1, n - 5)                     # some rows carry padding
        sel = rng.permutation(S)[:n]
        pos = rng.permutation(k)[:n]                           # padding at arbitrary positions
        idx[t, pos] = sel
    return Q, kp, vp, table, idx


def _run_attention(Q, kp, vp, table, idx, pg, scale, d_v):
    qd, kd = dev(Q, "bf16"), dev(kp, "bf16")
    vd = kd if vp is kp else dev(vp, "bf16")
    out, lse = B.janus_sparse_attn_prefill(qd, kd, vd, dev(idx, "i32"), page_table=dev(table, "i32"), page_size=pg,
                                           softmax_scale=scale, d_v=d_v)
    return Hp.bf16_tensor_to_f64(out), lse.cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("M,S,H_q,n_kv,d_qk,d_v,pg,k,latent,scale", [
    (9, 700, 8, 8, 128, 128, 64, 100, False, 1 / np.sqrt(128)),      # multi-head, one query head per kv head
    (5, 300, 16, 4, 64, 64, 16, 37, False, 0.125),                   # grouped heads, ragged tile
    (6, 1000, 128, 1, 576, 512, 64, 300, True, 1 / 24),              # latent layout: value = first 512 dims of the key row
    (3, 200, 128, 1, 576, 512, 64, 64, True, 1 / 24),
    (2, 50, 8, 2, 32, 32, 8, 70, False, 0.3),                        # k larger than the number of keys
])
def test_sparse_attention_matches_oracle(M, S, H_q, n_kv, d_qk, d_v, pg, k, latent, scale):
    Q, kp, vp, table, idx = _attention_case(M + S, M, S, H_q, n_kv, d_qk, d_v, pg, k, latent)
    got, lse = _run_attention(Q, kp, vp, table, idx, pg, scale, d_v)
    B.check_dev_status()
    ref, ref_lse = O.sparse_attention(Q, kp, vp, table, idx, page_size=pg, softmax_scale=scale, d_qk=d_qk, d_v=d_v)
    Hp.assert_attention_close(got, ref, "attention")
    np.testing.assert_allclose(lse, ref_lse, rtol=2e-3, atol=2e-3)


def test_sparse_attention_sharp_softmax_and_special_rows():
    # logits with a standard deviation of several units: the softmax is far from uniform, one key often dominates
    M, S, pg, k = 6, 500, 64, 128
    for latent, H_q, n_kv, d_qk, d_v in ((True, 128, 1, 576, 512), (False, 8, 8, 128, 128)):
        Q, kp, vp, table, idx = _attention_case(5, M, S, H_q, n_kv, d_qk, d_v, pg, k, latent)
        scale = 6.0 / np.sqrt(d_qk)
        idx[1, :] = -1
        idx[1, 7] = 123                                        # a single selected key: output is its value row
        idx[2, :] = -1                                         # nothing selected: zeros, lse = -inf
        got, lse = _run_attention(Q, kp, vp, table, idx, pg, scale, d_v)
        ref, ref_lse = O.sparse_attention(Q, kp, vp, table, idx, page_size=pg, softmax_scale=scale, d_qk=d_qk, d_v=d_v)
        Hp.assert_attention_close(got, ref, "sharp")
        v_row = O.decode_bf16(vp[table[123 // pg], 123 % pg, :, :d_v])
        for h in range(H_q):
            assert np.array_equal(got[1, h], v_row[h * n_kv // H_q])
        assert np.all(got[2] == 0) and np.all(np.isneginf(lse[2]))
        fin = np.isfinite(ref_lse)
        np.testing.assert_allclose(lse[fin], ref_lse[fin], rtol=2e-3, atol=2e-3)
    B.check_dev_status()


def test_sparse_attention_full_selection_equals_dense_causal_attention():
    # k >= prefix: the selection is the whole causal prefix, so the result is ordinary causal attention
    L, M, pg = 150, 20, 16
    S = L + M
    rng = np.random.default_rng(11)
    K = W.to_bf16_bits(rng.standard_normal((S, 2, 64)).astype(np.float32))
    V = W.to_bf16_bits(rng.standard_normal((S, 2, 64)).astype(np.float32))
    Q = W.to_bf16_bits(rng.standard_normal((M, 8, 64)).astype(np.float32))
    n_log = (S + pg - 1) // pg
    table = rng.permutation(n_log).astype(np.int32)
    kp = np.zeros((n_log, pg, 2, 64), np.uint16)
    vp = np.zeros((n_log, pg, 2, 64), np.uint16)
    for s in range(S):
        kp[table[s // pg], s % pg] = K[s]
        vp[table[s // pg], s % pg] = V[s]
    sc = rng.standard_normal((M, S)).astype(np.float32)
    idx, _, _ = _run_topk(sc, 256, L, True)                      # k = 256 > S: every visible key, -1 padded
    got, _ = _run_attention(Q, kp, vp, table, idx, pg, 0.125, 64)
    dense = O.dense_causal_attention(O.decode_bf16(Q), O.decode_bf16(K), O.decode_bf16(V), softmax_scale=0.125, q_pos0=L)
    Hp.assert_attention_close(got, dense, "dense-equivalence")


# ------------------------------------------------------------------------------------------------ the whole chain
@pytest.mark.parametrize("cfg,L,M,k", [(1, 1000, 70, 64), (2, 3000, 40, 256), (3, 3000, 40, 256), (5, 6000, 48, 256)])
def test_chain_on_reduced_configs(cfg, L, M, k):
    shp = W.config_shape(cfg, L=L, M=M, k=k)
    sess = W.make_session(shp, seed=0)
    d = Hp.upload_session(sess)
    sc = B.janus_indexer_scores(d["q_idx"], d["k_idx"], d["w"], q_scale=d["q_scale"], k_scale=d["k_scale"], row_bias=d["row_bias"],
                                col_bias=d["col_bias"], q_pos0=shp.L, causal=True)
    idx, count, kth = B.janus_topk(sc, shp.S, shp.k, q_pos0=shp.L, causal=True)
    pd = B.janus_page_demand(idx, demand_limit=shp.L, page_size=shp.page_size, page_table=d["page_table"],
                             n_phys_pages=sess["n_phys_pages"])
    out, lse = B.janus_sparse_attn_prefill(d["Q"], d["k_pool"], d["v_pool"], idx, page_table=d["page_table"], page_size=shp.page_size,
                                           softmax_scale=shp.softmax_scale, d_v=shp.d_v)
    B.check_dev_status()
    rows = np.arange(M)
    ref_sc = Hp.oracle_scores_rows(sess, rows)
    Hp.assert_scores_close(sc[:, :shp.S].cpu().numpy(), ref_sc, 1e-4 if cfg != 5 else 2e-4, f"config {cfg}")
    idx_np = idx.cpu().numpy()
    for t in range(M):
        ok, msg = O.topk_row_agrees(idx_np[t], ref_sc[t], shp.L + t + 1, shp.k)
        assert ok, f"config {cfg} row {t}: {msg}"
    got = Hp.page_lists_from_device(pd)
    ref = O.page_demand(idx_np, shp.L, shp.page_size, sess["page_table"])
    assert got["pages"] == ref["pages"] and got["runs"] == ref["runs"] and got["miss"] == ref["pages"]
    ref_o, _ = O.sparse_attention(sess["Q"], sess["k_pool"], sess["v_pool"], sess["page_table"], idx_np, page_size=shp.page_size,
                                  softmax_scale=shp.softmax_scale, d_qk=shp.d_qk, d_v=shp.d_v)
    Hp.assert_attention_close(Hp.bf16_tensor_to_f64(out), ref_o, f"config {cfg}")
