"""Decode step over a batch of sessions (Sec. 2.2, "Decode phase": an append prefill with a single appended token per
session) through the C ABI: janus_indexer_scores_batch -> janus_topk_batch -> janus_page_demand_batch ->
janus_sparse_attn_decode, each checked against the oracle session by session.  Sessions have ragged history lengths
(one shorter than k, one shorter than a key tile), their own page tables into one global KV pool, and concatenated
indexer keys."""
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


def make_batch(seed, lengths, dtype, H=64, D=128, page=64):
    """Session b: L_b cached tokens plus the new one.  Keys are concatenated with rows padded to a multiple of 4."""
    rng = np.random.default_rng(seed)
    nb = len(lengths)
    key_off = [0]
    for L in lengths:
        key_off.append(key_off[-1] + (L + 1 + 3) // 4 * 4)
    total = key_off[-1]
    kf = rng.standard_normal((total, D)).astype(np.float32)
    qf = rng.standard_normal((nb, H, D)).astype(np.float32)
    b = {"lengths": lengths, "key_off": np.array(key_off, np.int64), "w": (rng.uniform(0, 1, (nb, H)) / 8).astype(np.float32), "dtype": dtype,
         "q_scale": None, "k_scale": None}
    if dtype == "bf16":
        b["q"], b["k"] = W.to_bf16_bits(qf), W.to_bf16_bits(kf)
    else:
        b["q"], b["k"] = W.to_e4m3_bits(2 * qf), W.to_e4m3_bits(2 * kf)
        b["q_scale"] = np.exp2(rng.uniform(-2, 2, (nb, H))).astype(np.float32)
        b["k_scale"] = np.exp2(rng.uniform(-1, 1, total)).astype(np.float32)
    # page tables: session b needs ceil((L_b + 1) / page) pages, drawn without replacement from one global pool
    n_pages = [(L + 1 + page - 1) // page for L in lengths]
    n_phys = sum(n_pages) + 37
    perm = rng.permutation(n_phys)
    tab_off = np.concatenate([[0], np.cumsum(n_pages)]).astype(np.int64)
    b["tables"] = perm[:tab_off[-1]].astype(np.int32)
    b["tab_off"], b["n_phys"], b["page"] = tab_off, n_phys, page
    return b


def session_keys(b, i):
    a = int(b["key_off"][i])
    return slice(a, a + b["lengths"][i] + 1)


@pytest.mark.parametrize("dtype", ["bf16", "fp8"])
def test_decode_batch_matches_oracle_session_by_session(dtype):
    lengths = [5000, 12345, 300, 20000, 40, 7777, 129]
    k, page, d_qk, d_v, H_q = 128, 64, 576, 512, 128
    b = make_batch(11, lengths, dtype, page=page)
    nb = len(lengths)
    rng = np.random.default_rng(5)
    q_attn = W.to_bf16_bits((rng.standard_normal((nb, H_q, d_qk)) / 4).astype(np.float32))
    pool = W.to_bf16_bits((rng.standard_normal((b["n_phys"], page, 1, d_qk)) / 4).astype(np.float32))
    scale = 1.0 / np.sqrt(d_qk)

    dev = lambda x, kind: B.to_device(x, kind)
    key_off = torch.from_numpy(b["key_off"]).cuda()
    tab_off = torch.from_numpy(b["tab_off"]).cuda()
    limits = torch.tensor(lengths, dtype=torch.int64, device="cuda")
    kd = dev(b["k"], dtype)

    # ---- indexer
    # key_offsets[b+1] - key_offsets[b] includes the padding rows: they are scored like keys (their bits are whatever the
    # caller put there) and left out of the selection through row_lengths
    scores = B.janus_indexer_scores_batch(dev(b["q"], dtype), kd, dev(b["w"], "f32"), key_off, max(lengths) + 4,
                                          q_scale=dev(b["q_scale"], "f32"), k_scale=dev(b["k_scale"], "f32"))
    row_len = torch.tensor([L + 1 for L in lengths], dtype=torch.int64, device="cuda")
    idx, cnt, kth = B.janus_topk_batch(scores, key_off, k, row_lengths=row_len)
    pd = B.janus_page_demand_batch(idx, demand_limits=limits, page_size=page, page_tables=dev(b["tables"], "i32"), table_offsets=tab_off,
                                   n_phys_pages=b["n_phys"])
    out, lse = B.janus_sparse_attn_decode(dev(q_attn, "bf16"), dev(pool, "bf16"), dev(pool, "bf16"), idx, page_tables=dev(b["tables"], "i32"),
                                          table_offsets=tab_off, page_size=page, softmax_scale=scale, d_v=d_v)
    B.check_dev_status()
    scores_h, idx_h, cnt_h = scores.cpu().numpy(), idx.cpu().numpy(), cnt.cpu().numpy()
    out_h, lse_h = Hp.bf16_tensor_to_f64(out), lse.cpu().numpy().astype(np.float64)

    all_pages = set()
    for i, L in enumerate(lengths):
        ks = session_keys(b, i)
        ref = O.indexer_scores(b["q"][i:i + 1], b["k"][ks], b["w"][i:i + 1], dtype=dtype,
                               q_scale=None if b["q_scale"] is None else b["q_scale"][i:i + 1],
                               k_scale=None if b["k_scale"] is None else b["k_scale"][ks], q_pos0=L, causal=True)
        Hp.assert_scores_close(scores_h[ks][None, :], ref, 1e-4 if dtype == "bf16" else 1e-4, f"session {i} scores")
        # selection over the session's L + 1 keys
        n_sel = min(k, L + 1)
        assert cnt_h[i] == n_sel and idx_h[i].max() <= L
        ok, msg = O.topk_row_agrees(idx_h[i], ref[0], L + 1, k)
        assert ok, f"session {i}: {msg}"
        # pages of the selected history tokens through the session's own table
        table = b["tables"][b["tab_off"][i]:b["tab_off"][i + 1]]
        all_pages |= set(O.page_demand(idx_h[i:i + 1], L, page, table)["pages"])
        # attention of the one query row over its selection
        ref_o, ref_lse = O.sparse_attention(q_attn[i:i + 1], pool, pool, table, idx_h[i:i + 1], page_size=page, softmax_scale=scale,
                                            d_qk=d_qk, d_v=d_v)
        Hp.assert_attention_close(out_h[i:i + 1], ref_o, f"session {i} attention")
        np.testing.assert_allclose(lse_h[i:i + 1], ref_lse, rtol=2e-3, atol=2e-3)
    got = Hp.page_lists_from_device(pd)
    assert got["pages"] == sorted(all_pages)
    assert got["runs"] == [tuple(r) for r in O.maximal_runs(sorted(all_pages))]
    assert got["miss"] == sorted(all_pages)          # nothing declared resident


def test_decode_indexer_with_fp4_keys():
    # indexer keys stored as FP4 E2M1, two per byte (Sec. 5.1), FP8 queries: the same ragged batch call with another key format
    lengths = [9000, 129, 20001, 40, 3333]
    rng = np.random.default_rng(17)
    nb, H, D = len(lengths), 64, 128
    key_off = [0]
    for L in lengths:
        key_off.append(key_off[-1] + (L + 1 + 3) // 4 * 4)
    total = key_off[-1]
    codes = rng.integers(0, 16, size=(total, D)).astype(np.uint8)
    packed = (codes[:, 0::2] | (codes[:, 1::2] << 4)).astype(np.uint8)          # element 2i in the low nibble of byte i
    q = W.to_e4m3_bits(2 * rng.standard_normal((nb, H, D)).astype(np.float32))
    w = (rng.uniform(0, 1, (nb, H)) / 8).astype(np.float32)
    q_scale = np.exp2(rng.uniform(-2, 2, (nb, H))).astype(np.float32)
    k_scale = np.exp2(rng.uniform(-1, 1, total)).astype(np.float32)
    off = torch.tensor(key_off, dtype=torch.int64, device="cuda")
    scores = B.janus_indexer_scores_batch(B.to_device(q, "fp8"), torch.from_numpy(packed).cuda(), B.to_device(w, "f32"), off, max(lengths) + 4,
                                          q_scale=B.to_device(q_scale, "f32"), k_scale=B.to_device(k_scale, "f32"), keys_fp4=True)
    B.check_dev_status()
    got = scores.cpu().numpy()
    for i, L in enumerate(lengths):
        ks = slice(key_off[i], key_off[i] + L + 1)
        ref = O.indexer_scores(q[i:i + 1], packed[ks], w[i:i + 1], dtype="fp8+fp4k", q_scale=q_scale[i:i + 1], k_scale=k_scale[ks],
                               q_pos0=L, causal=True)
        Hp.assert_scores_close(got[ks][None, :], ref, 1e-4, f"session {i} scores (fp4 keys)")


def test_prefill_indexer_and_selection_with_fp4_keys():
    # append prefill over a key cache stored as FP4 E2M1 (Sec. 5.1): scores against the oracle on sampled rows, and the
    # one-call indexer + top-k (which takes this key format through a score matrix in its workspace)
    M, L, H, D, k = 70, 20011, 64, 128, 256
    rng = np.random.default_rng(23)
    S = L + M
    codes = rng.integers(0, 16, size=(S, D)).astype(np.uint8)
    packed = (codes[:, 0::2] | (codes[:, 1::2] << 4)).astype(np.uint8)
    q = W.to_e4m3_bits(2 * rng.standard_normal((M, H, D)).astype(np.float32))
    w = (rng.uniform(0, 1, (M, H)) / 8).astype(np.float32)
    q_scale = np.exp2(rng.uniform(-2, 2, (M, H))).astype(np.float32)
    k_scale = np.exp2(rng.uniform(-1, 1, S)).astype(np.float32)
    qd, kd, wd = B.to_device(q, "fp8"), torch.from_numpy(packed).cuda(), B.to_device(w, "f32")
    args = dict(q_scale=B.to_device(q_scale, "f32"), k_scale=B.to_device(k_scale, "f32"), q_pos0=L, causal=True, keys_fp4=True)
    scores = B.janus_indexer_scores(qd, kd, wd, **args)
    idx, cnt, kth = B.janus_indexer_topk(qd, kd, wd, k, **args)
    B.check_dev_status()
    got, idx_h = scores.cpu().numpy(), idx.cpu().numpy()
    assert np.array_equal(cnt.cpu().numpy(), np.full(M, k))
    for t in W.sample_rows(M, 5):
        t = int(t)
        ref = O.indexer_scores(q[t:t + 1], packed, w[t:t + 1], dtype="fp8+fp4k", q_scale=q_scale[t:t + 1], k_scale=k_scale, q_pos0=L + t,
                               causal=True)
        Hp.assert_scores_close(got[t:t + 1, :L + t + 1], ref[:, :L + t + 1], 1e-4, f"row {t} scores (fp4 keys)")
        assert np.all(np.isneginf(got[t, L + t + 1:S]))
        ok, msg = O.topk_row_agrees(idx_h[t], ref[0], L + t + 1, k)
        assert ok, f"row {t}: {msg}"
    # a shape outside the tensor-core kernel has no 4-bit path
    lib = B.load()
    sc = torch.empty((3, 64), dtype=torch.float32, device="cuda")
    rc = lib.janus_indexer_scores(qd.data_ptr(), 5 * D, kd.data_ptr(), D, wd.data_ptr(), args["q_scale"].data_ptr(), 5, args["k_scale"].data_ptr(),
                                  None, None, 3, 5, D, 64, 0, 1, 2, sc.data_ptr(), 64, None, 0, None, None)
    assert rc == 2                                            # JANUS_ERR_UNSUPPORTED


def _status_word():
    """Reads and clears the device status word (the tests below expect it to be set)."""
    st = B.dev_status_tensor()
    v = int(st.item())
    st.zero_()
    return v


def test_batch_entries_report_and_skip_bad_offsets():
    """Offsets and page ids that come from device memory are never trusted (the library's rule: device-visible conditions are
    reported in the status word and skipped, nothing traps): a misaligned or negative score-row offset, a session that
    leaves the key array, a negative page-table offset and a negative physical page id each set
    JANUS_DEV_INDEX_OUT_OF_RANGE, leave the other rows' results as they are, and the next ordinary call passes."""
    lengths = [900, 400, 2500, 131]
    k, page, d_qk, d_v, H_q = 64, 64, 576, 512, 128
    b = make_batch(23, lengths, "fp8", page=page)
    nb = len(lengths)
    dev = lambda x, kind: B.to_device(x, kind)
    key_off = torch.from_numpy(b["key_off"]).cuda()
    kd, qd, wd = dev(b["k"], "fp8"), dev(b["q"], "fp8"), dev(b["w"], "f32")
    qs, ks = dev(b["q_scale"], "f32"), dev(b["k_scale"], "f32")
    total = b["k"].shape[0]
    good = B.janus_indexer_scores_batch(qd, kd, wd, key_off, max(lengths) + 4, q_scale=qs, k_scale=ks)
    B.check_dev_status()
    row_len = torch.tensor([L + 1 for L in lengths], dtype=torch.int64, device="cuda")
    idx_good, cnt_good, _ = B.janus_topk_batch(good, key_off, k, row_lengths=row_len)
    B.check_dev_status()

    # ---- janus_topk_batch: row 1 starts off a 16-byte boundary, row 3 before the array
    bad_off = b["key_off"].copy()
    bad_off[1] += 2
    bad_off[3] = -8
    idx, cnt, kth = B.janus_topk_batch(good, torch.from_numpy(bad_off).cuda(), k, row_lengths=row_len)
    assert _status_word() == 101
    idx_h, cnt_h = idx.cpu().numpy(), cnt.cpu().numpy()
    assert (idx_h[1] == -1).all() and (idx_h[3] == -1).all() and cnt_h[1] == 0 and cnt_h[3] == 0
    assert np.isneginf(kth.cpu().numpy()[[1, 3]]).all()
    for i in (0, 2):
        assert set(idx_h[i].tolist()) == set(idx_good[i].cpu().numpy().tolist()) and cnt_h[i] == int(cnt_good[i])
    # a negative length
    bad_len = row_len.clone()
    bad_len[2] = -5
    idx, cnt, _ = B.janus_topk_batch(good, key_off, k, row_lengths=bad_len)
    assert _status_word() == 101 and int(cnt[2]) == 0 and (idx[2] == -1).all()

    # ---- janus_indexer_scores_batch: the last session claims rows beyond the key array, session 1 starts before it
    canary = torch.full((total + 4096,), 7.5, dtype=torch.float32, device="cuda")
    over = b["key_off"].copy()
    over[-1] = total + 3000
    sc = B.janus_indexer_scores_batch(qd, kd, wd, torch.from_numpy(over).cuda(), max(lengths) + 4, q_scale=qs, k_scale=ks, scores=canary[:total])
    assert _status_word() == 101
    assert (canary[total:] == 7.5).all()                       # nothing was written past the score array
    a0, a3 = int(b["key_off"][0]), int(b["key_off"][3])
    assert torch.equal(sc[a0:a0 + lengths[0] + 1], good[a0:a0 + lengths[0] + 1])
    assert torch.equal(sc[a3:total], good[a3:total])           # the part of the cut session that lies inside the array
    neg = b["key_off"].copy()
    neg[1] = -4
    sc = B.janus_indexer_scores_batch(qd, kd, wd, torch.from_numpy(neg).cuda(), max(lengths) + 4, q_scale=qs, k_scale=ks)
    assert _status_word() == 101
    a2 = int(b["key_off"][2])
    assert torch.equal(sc[a2:a2 + lengths[2] + 1], good[a2:a2 + lengths[2] + 1])

    # ---- janus_page_demand_batch: a negative page-table offset empties that row's table
    tab_off = torch.from_numpy(b["tab_off"]).cuda()
    limits = torch.tensor(lengths, dtype=torch.int64, device="cuda")
    tables = dev(b["tables"], "i32")
    neg_tab = b["tab_off"].copy()
    neg_tab[2] = -3
    pd = B.janus_page_demand_batch(idx_good, demand_limits=limits, page_size=page, page_tables=tables, table_offsets=torch.from_numpy(neg_tab).cuda(),
                                   n_phys_pages=b["n_phys"])
    assert _status_word() == 101
    idx_gh = idx_good.cpu().numpy()
    want = set()
    for i, L in enumerate(lengths):
        if i in (1, 2):      # row 1's table now ends at a negative offset (length < 0), row 2's starts at one: both are empty
            continue
        want |= set(O.page_demand(idx_gh[i:i + 1], L, page, b["tables"][b["tab_off"][i]:b["tab_off"][i + 1]])["pages"])
    assert Hp.page_lists_from_device(pd)["pages"] == sorted(want)

    # ---- janus_sparse_attn_decode: a negative physical page id is skipped like a padding slot
    rng = np.random.default_rng(9)
    q_attn = W.to_bf16_bits((rng.standard_normal((nb, H_q, d_qk)) / 4).astype(np.float32))
    pool = W.to_bf16_bits((rng.standard_normal((b["n_phys"], page, 1, d_qk)) / 4).astype(np.float32))
    bad_tables = b["tables"].copy()
    lp_bad = 3                                                   # session 0, logical page 3
    bad_tables[b["tab_off"][0] + lp_bad] = -1
    pool_d = dev(pool, "bf16")
    scale = 1.0 / np.sqrt(d_qk)
    out, _ = B.janus_sparse_attn_decode(dev(q_attn, "bf16"), pool_d, pool_d, idx_good, page_tables=dev(bad_tables, "i32"), table_offsets=tab_off,
                                        page_size=page, softmax_scale=scale, d_v=d_v)
    hit = (idx_gh[0] >= 0) & (idx_gh[0] // page == lp_bad)
    st = _status_word()
    assert st == (101 if hit.any() else 0)
    idx_ref = idx_gh[0:1].copy()
    idx_ref[0, hit] = -1                                         # the oracle on the selection without the skipped tokens
    ref_o, _ = O.sparse_attention(q_attn[0:1], pool, pool, b["tables"][b["tab_off"][0]:b["tab_off"][1]], idx_ref, page_size=page,
                                  softmax_scale=scale, d_qk=d_qk, d_v=d_v)
    Hp.assert_attention_close(Hp.bf16_tensor_to_f64(out)[0:1], ref_o, "attention with a negative page id")

    # an ordinary call afterwards is clean
    again = B.janus_indexer_scores_batch(qd, kd, wd, key_off, max(lengths) + 4, q_scale=qs, k_scale=ks)
    B.check_dev_status()
    assert torch.equal(again, good)
