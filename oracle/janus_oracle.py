"""CPU oracle for the append-prefill hot path of a top-k sparse-attention layer.

TEST INFRASTRUCTURE ONLY.  This is a plain, slow, fp64 restatement of what the four
library calls compute, written from the paper's definitions.  Only the tests, the smoke
check and the benchmark's CPU-baseline leg may use it; the product path never does, and
this module shares no code with (and does not import) the CUDA path.

Notation: L history tokens, M new tokens, S = L + M keys, 0-based positions (the paper
uses P for the history, L for the appended query and 1-based index sets, Table 1).

Steps and the passages they restate:
  indexer_scores   Eq. 1 (Sec. 2.2): relevance of every preceding token for each new token.
                   The paper leaves the scoring function to the model reports; the reading
                   used is  score[t,s] = sum_h w[t,h] * relu(<q[t,h,:], k[s,:]>)  with one
                   shared indexer key per token, causal over history + earlier new tokens,
                   the token itself included.
  topk_select      Eq. 1: the k best-scoring visible tokens per new token.
  page_demand      Sec. 2.2 (union of selections), Sec. 4.2 (corrective reads = exact minus
                   predicted), Sec. 4.3 (address-ordered unique blocks, maximal runs).
  sparse_attention Sec. 2.2: attention of each new token over only its selected KV rows.
  recall_precision Sec. 4.2: |pred ∩ exact| / |exact| and |pred ∩ exact| / |pred|.

Parity pins: every function here is pinned by CPU tests against closed forms, brute force,
library routines on special cases and hand-computed cases (no function is "parity unpinned").
"""
from __future__ import annotations

import numpy as np

NEG_INF = -np.inf


# ----------------------------------------------------------------------------
# storage formats -> fp64 (exact)
# ----------------------------------------------------------------------------
def decode_bf16(bits) -> np.ndarray:
    """bf16 bit patterns (uint16) -> float64.  bf16 is the upper half of an IEEE binary32."""
    b = np.asarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def _e4m3_table() -> np.ndarray:
    """All 256 values of OCP FP8 E4M3 ("fn": no infinities; S.1111.111 is NaN):
    1 sign, 4 exponent (bias 7), 3 mantissa bits; exponent 0 is subnormal."""
    t = np.empty(256, dtype=np.float64)
    for code in range(256):
        sign = -1.0 if code & 0x80 else 1.0
        e = (code >> 3) & 0xF
        m = code & 0x7
        if e == 0xF and m == 0x7:
            v = np.nan
        elif e == 0:
            v = sign * (m / 8.0) * 2.0 ** (-6)
        else:
            v = sign * (1.0 + m / 8.0) * 2.0 ** (e - 7)
        t[code] = v
    return t


_E4M3 = _e4m3_table()


def decode_e4m3(codes) -> np.ndarray:
    """FP8 E4M3 bytes (uint8) -> float64."""
    return _E4M3[np.asarray(codes, dtype=np.uint8)]


def decode_e2m1(packed) -> np.ndarray:
    """FP4 E2M1 keys (Sec. 5.1: indexer keys of one model family are stored in FP4), two per byte, element 2i in the low
    nibble of byte i -> float64 [..., 2 * bytes].  OCP E2M1: 1 sign, 2 exponent (bias 1), 1 mantissa bit; exponent 0 is
    subnormal (0 or 0.5); no infinities or NaNs: the magnitudes are 0, 0.5, 1, 1.5, 2, 3, 4, 6."""
    b = np.asarray(packed, dtype=np.uint8)
    codes = np.stack([b & 0xF, b >> 4], axis=-1).reshape(*b.shape[:-1], b.shape[-1] * 2)
    sign = np.where(codes & 0x8, -1.0, 1.0)
    e = ((codes >> 1) & 0x3).astype(np.float64)
    m = (codes & 0x1).astype(np.float64)
    mag = np.where(e == 0, 0.5 * m, (1.0 + 0.5 * m) * 2.0 ** (e - 1.0))
    return sign * mag


def decode(x, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return decode_bf16(x)
    if dtype == "fp8":
        return decode_e4m3(x)
    if dtype == "fp4":
        return decode_e2m1(x)
    if dtype == "f64":
        return np.asarray(x, dtype=np.float64)
    raise ValueError(dtype)


def visible_prefix(t: int, n_keys: int, q_pos0: int, causal: bool) -> int:
    """Number of keys row t may see: keys 0..q_pos0+t inclusive when causal, else all."""
    return min(n_keys, q_pos0 + t + 1) if causal else n_keys


# ----------------------------------------------------------------------------
# indexer (Eq. 1, scoring part)
# ----------------------------------------------------------------------------
def indexer_scores(q, k, w, *, dtype: str = "bf16", q_scale=None, k_scale=None,
                   row_bias=None, col_bias=None, recency=None,
                   q_pos0: int = 0, causal: bool = True, rows=None) -> np.ndarray:
    """score[t,s] = sum_h w[t,h] * max(0, <qd[t,h,:], kd[s,:]>) (+ bias), -inf where masked.

    q [M,H,D], k [n_keys,D] in storage format ``dtype``; w [M,H] fp32.
    FP8: qd = decode(q) * q_scale[h] (or q_scale[t,h]), kd = decode(k) * k_scale[s].
    Bias (optional): either the rank-1 product row_bias[t]*col_bias[s], or
    ``recency=(amp, tau)`` evaluated directly as amp*exp(-(q_pos0+t-s)/tau).
    ``rows`` selects query rows (default all); returns float64 [len(rows), n_keys]."""
    # dtype "fp8+fp4k": FP8 queries, FP4 (E2M1, packed two per byte) keys with the same per-key scale convention
    qd = decode(q, "fp8" if dtype == "fp8+fp4k" else dtype)
    kd = decode(k, "fp4" if dtype == "fp8+fp4k" else dtype)
    M, H, D = qd.shape
    n_keys = kd.shape[0]
    w = np.asarray(w, dtype=np.float64)
    if q_scale is not None:
        qs = np.asarray(q_scale, dtype=np.float64)
        qd = qd * (qs[None, :, None] if qs.ndim == 1 else qs[:, :, None])
    if k_scale is not None:
        kd = kd * np.asarray(k_scale, dtype=np.float64)[:, None]
    rows = np.arange(M) if rows is None else np.asarray(rows, dtype=np.int64)
    out = np.full((len(rows), n_keys), NEG_INF, dtype=np.float64)
    s_all = np.arange(n_keys, dtype=np.float64)
    for i, t in enumerate(rows):
        t = int(t)
        n = visible_prefix(t, n_keys, q_pos0, causal)
        if n <= 0:
            continue
        dots = kd[:n] @ qd[t].T                    # [n, H] per-head dot products
        sc = np.maximum(dots, 0.0) @ w[t]           # ReLU, then the weighted head sum
        if recency is not None:
            amp, tau = recency
            sc = sc + amp * np.exp(-((q_pos0 + t) - s_all[:n]) / tau)
        elif row_bias is not None:
            sc = sc + float(row_bias[t]) * np.asarray(col_bias[:n], dtype=np.float64)
        out[i, :n] = sc
    return out


# ----------------------------------------------------------------------------
# top-k (Eq. 1, selection part)
# ----------------------------------------------------------------------------
def topk_select(score_row, prefix: int, k: int):
    """The min(k, prefix) best of score_row[:prefix]; ties go to the lower index.
    Returns (indices sorted by (score desc, index asc), threshold = last selected score)."""
    n = min(k, prefix)
    if n <= 0:
        return np.empty(0, dtype=np.int64), NEG_INF
    sc = np.asarray(score_row[:prefix], dtype=np.float64)
    order = np.lexsort((np.arange(prefix), -sc))   # primary: score descending; secondary: index ascending
    sel = order[:n]
    return sel.astype(np.int64), float(sc[sel[-1]])


def topk(scores, k: int, *, q_pos0: int = 0, causal: bool = True, rows=None) -> np.ndarray:
    """Row-wise top-k of a score block; rows[i] is the query position of scores[i].
    Returns int64 [n_rows, k] padded with -1."""
    scores = np.asarray(scores)
    n_rows, n_keys = scores.shape
    rows = np.arange(n_rows) if rows is None else np.asarray(rows)
    out = np.full((n_rows, k), -1, dtype=np.int64)
    for i, t in enumerate(rows):
        sel, _ = topk_select(scores[i], visible_prefix(int(t), n_keys, q_pos0, causal), k)
        out[i, :len(sel)] = sel
    return out


# ----------------------------------------------------------------------------
# entry granularity (footnote of Sec. 2.2: selection and attention per entry = a region of E consecutive tokens)
# ----------------------------------------------------------------------------
# The paper does not define how an entry is scored or masked.  Reading used here: the indexer has one key per entry, so
# entry scores come from the same indexer run over entry keys; the query at position pos may select every entry that holds
# at least one token at or before pos (entries 0 .. pos // E), and attends to the tokens of the selected entries that are at
# or before pos.
def entry_visible_prefix(t: int, n_entries: int, q_pos0: int, entry_size: int) -> int:
    """Number of entries the query row t (position q_pos0 + t) may select."""
    return max(0, min(n_entries, (q_pos0 + t) // entry_size + 1))


def entry_pool_scores(scores, *, entry_size: int, q_pos0: int = 0, causal: bool = True) -> np.ndarray:
    """Second reading of the entry-granularity footnote of Sec. 2.2 (the paper defines neither): the indexer scores tokens as
    usual and an entry's score is the maximum over the tokens of the entry that the row may see,
        entry_score[t, e] = max { score[t, s] : e*E <= s < (e+1)*E, s <= q_pos0 + t },
    -inf for an entry without a visible token.  scores [n_rows, n_keys]; returns float64 [n_rows, ceil(n_keys / E)]."""
    scores = np.asarray(scores, dtype=np.float64)
    n_rows, n_keys = scores.shape
    n_entries = (n_keys + entry_size - 1) // entry_size
    out = np.full((n_rows, n_entries), NEG_INF, dtype=np.float64)
    for t in range(n_rows):
        prefix = visible_prefix(t, n_keys, q_pos0, causal)
        for e in range(n_entries):
            a, b = e * entry_size, min((e + 1) * entry_size, prefix)
            if b > a:
                out[t, e] = scores[t, a:b].max()
    return out


def entry_topk(entry_scores, k_e: int, *, q_pos0: int, entry_size: int) -> np.ndarray:
    """Row-wise top-k_e over entries.  Returns int64 [n_rows, k_e] padded with -1."""
    entry_scores = np.asarray(entry_scores)
    n_rows, n_entries = entry_scores.shape
    out = np.full((n_rows, k_e), -1, dtype=np.int64)
    for t in range(n_rows):
        sel, _ = topk_select(entry_scores[t], entry_visible_prefix(t, n_entries, q_pos0, entry_size), k_e)
        out[t, :len(sel)] = sel
    return out


def entry_expand(entry_idx, *, q_pos0: int, entry_size: int) -> np.ndarray:
    """Token selection of entry selections: slot e*E + j of row t holds token entry_idx[t, e]*E + j if that token is at or
    before position q_pos0 + t, else -1.  Returns int64 [n_rows, k_e * E]."""
    entry_idx = np.asarray(entry_idx)
    n_rows, k_e = entry_idx.shape
    out = np.full((n_rows, k_e * entry_size), -1, dtype=np.int64)
    for t in range(n_rows):
        pos = q_pos0 + t
        for e in range(k_e):
            ent = int(entry_idx[t, e])
            if ent < 0:
                continue
            for j in range(entry_size):
                tok = ent * entry_size + j
                if tok <= pos:
                    out[t, e * entry_size + j] = tok
    return out


def topk_row_agrees(got_idx, score_row, prefix: int, k: int, band_rel: float = 1e-3):
    """Acceptance rule for one row of a selection computed elsewhere.

    With tau the oracle's k-th score and band = max(band_rel*|tau|, 1e-6*max|score|):
      (i)   exactly min(k,prefix) distinct valid indices in [0,prefix), the rest -1;
      (ii)  every index whose oracle score exceeds tau+band is present;
      (iii) every returned index has oracle score >= tau-band.
    Returns (ok, message)."""
    got = np.asarray(got_idx).astype(np.int64)
    valid = got[got >= 0]
    n = min(k, prefix)
    if len(valid) != n:
        return False, f"{len(valid)} valid indices, expected {n}"
    if n == 0:
        return True, ""
    if len(np.unique(valid)) != n:
        return False, "duplicate indices"
    if valid.max() >= prefix:
        return False, f"index {valid.max()} outside the visible prefix {prefix}"
    sc = np.asarray(score_row[:prefix], dtype=np.float64)
    _, tau = topk_select(sc, prefix, k)
    band = max(band_rel * abs(tau), 1e-6 * float(np.max(np.abs(sc))))
    must = np.nonzero(sc > tau + band)[0]
    missing = np.setdiff1d(must, valid)
    if len(missing):
        return False, f"{len(missing)} indices clearly above the threshold are missing (e.g. {missing[:4]})"
    low = valid[sc[valid] < tau - band]
    if len(low):
        return False, f"{len(low)} returned indices are clearly below the threshold (e.g. {low[:4]})"
    return True, ""


# ----------------------------------------------------------------------------
# page demand: union, runs, miss set (Sec. 2.2, 4.2, 4.3)
# ----------------------------------------------------------------------------
def maximal_runs(sorted_unique_ids):
    """Maximal runs (start, length) of consecutive integers in an ascending list of unique ids."""
    runs = []
    for p in sorted_unique_ids:
        p = int(p)
        if runs and runs[-1][0] + runs[-1][1] == p:
            runs[-1][1] += 1
        else:
            runs.append([p, 1])
    return [(a, b) for a, b in runs]


def page_demand(idx, demand_limit: int, page_size: int, page_table, predicted_pages=None):
    """Pages that hold a selected history token.

    A = { page_table[s // page_size] : s in idx, 0 <= s < demand_limit }.
    Returns dict(pages=sorted(A), runs=maximal runs of A, miss=sorted(A - predicted),
    miss_runs=maximal runs of the miss set)."""
    table = np.asarray(page_table)
    flat = np.asarray(idx).reshape(-1)
    tokens = np.unique(flat[(flat >= 0) & (flat < demand_limit)])   # distinct selected history tokens (library sort)
    demand = set()
    for s in tokens:
        demand.add(int(table[int(s) // page_size]))
    pages = sorted(demand)
    pred = set(int(p) for p in predicted_pages) if predicted_pages is not None else set()
    miss = sorted(demand - pred)
    return {"pages": pages, "runs": maximal_runs(pages), "miss": miss, "miss_runs": maximal_runs(miss)}


def recall_precision(predicted, exact):
    """Recall |pred ∩ exact|/|exact| and precision |pred ∩ exact|/|pred| (Sec. 4.2)."""
    p, e = set(int(x) for x in predicted), set(int(x) for x in exact)
    inter = len(p & e)
    return (inter / len(e) if e else 1.0), (inter / len(p) if p else 1.0)


# ----------------------------------------------------------------------------
# sparse attention over the selected rows (Sec. 2.2)
# ----------------------------------------------------------------------------
def sparse_attention(Q, k_pool, v_pool, page_table, idx, *, page_size: int, softmax_scale: float,
                     d_qk: int, d_v: int, rows=None):
    """o[t,h] = sum_{s in idx[t]} softmax_s(scale * <Q[t,h,:d_qk], K_s[:d_qk]>) * V_s[:d_v].

    Q [M,H_q,d_qk] bf16 bits; pools [n_phys_pages, page_size, n_kv_heads, >=d] bf16 bits;
    token s lives at pool[page_table[s // page_size], s % page_size, h_kv], query head h reads
    kv head h * n_kv_heads // H_q.  idx[i] is the selection of query row rows[i]; -1 skipped.
    Returns (out float64 [n_rows,H_q,d_v], lse float64 [n_rows,H_q]); an empty selection gives
    zeros and lse = -inf."""
    Qd = decode_bf16(Q)
    M, H_q, _ = Qd.shape
    n_kv = k_pool.shape[2]
    table = np.asarray(page_table)
    rows = np.arange(M) if rows is None else np.asarray(rows, dtype=np.int64)
    idx = np.asarray(idx)
    out = np.zeros((len(rows), H_q, d_v), dtype=np.float64)
    lse = np.full((len(rows), H_q), NEG_INF, dtype=np.float64)
    for i, t in enumerate(rows):
        sel = idx[i][idx[i] >= 0].astype(np.int64)
        if len(sel) == 0:
            continue
        pg = table[sel // page_size]
        off = sel % page_size
        hk_loaded = -1
        for h in range(H_q):
            hk = h * n_kv // H_q
            if hk != hk_loaded:                                   # rows of this kv head, decoded once
                K = decode_bf16(k_pool[pg, off, hk, :d_qk])      # [n_sel, d_qk]
                V = decode_bf16(v_pool[pg, off, hk, :d_v])       # [n_sel, d_v]
                hk_loaded = hk
            logit = softmax_scale * (K @ Qd[int(t), h, :d_qk])
            m = logit.max()
            p = np.exp(logit - m)
            z = p.sum()
            out[i, h] = (p @ V) / z
            lse[i, h] = m + np.log(z)
    return out, lse


def dense_causal_attention(Q, K, V, *, softmax_scale: float, q_pos0: int):
    """Plain causal attention with contiguous (unpaged) keys, for cross-checks:
    query row t sees keys 0..q_pos0+t.  Q [M,H,d_qk], K [S,H_kv,d_qk], V [S,H_kv,d_v] float64."""
    M, H, _ = Q.shape
    S, H_kv, d_v = V.shape
    out = np.zeros((M, H, d_v))
    for t in range(M):
        n = min(S, q_pos0 + t + 1)
        for h in range(H):
            hk = h * H_kv // H
            logit = softmax_scale * (K[:n, hk] @ Q[t, h])
            p = np.exp(logit - logit.max())
            out[t, h] = (p / p.sum()) @ V[:n, hk]
    return out
