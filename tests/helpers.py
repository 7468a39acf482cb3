"""Shared helpers for the GPU parity tests: upload a generated session, run the library chain, compare."""
from __future__ import annotations

import numpy as np
import torch

from oracle import janus_oracle as O
from paper_2609_36938_b200 import binding as B


def upload_session(sess, device="cuda"):
    shp = sess["shape"]
    kind = shp.idx_dtype
    d = {
        "q_idx": B.to_device(sess["q_idx"], kind, device),
        "k_idx": B.to_device(sess["k_idx"], kind, device),
        "w": B.to_device(sess["w"], "f32", device),
        "q_scale": B.to_device(sess["q_scale"], "f32", device),
        "k_scale": B.to_device(sess["k_scale"], "f32", device),
        "row_bias": B.to_device(sess["row_bias"], "f32", device),
        "col_bias": B.to_device(sess["col_bias"], "f32", device),
        "page_table": B.to_device(sess["page_table"], "i32", device),
    }
    if "q_pred" in sess:
        d["q_pred"] = B.to_device(sess["q_pred"], kind, device)
    if "Q" in sess:
        d["Q"] = B.to_device(sess["Q"], "bf16", device)
        d["k_pool"] = B.to_device(sess["k_pool"], "bf16", device)
        d["v_pool"] = d["k_pool"] if sess["v_pool"] is sess["k_pool"] else B.to_device(sess["v_pool"], "bf16", device)
    return d


def bf16_tensor_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float64).cpu().numpy()


def bf16_tensor_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().view(torch.int16).numpy().view(np.uint16)


def oracle_scores_rows(sess, rows, *, predicted=False):
    """Oracle indexer scores for the given query rows (exact pass, or the predicted pass over history keys only)."""
    shp = sess["shape"]
    if predicted:
        return O.indexer_scores(sess["q_pred"], sess["k_idx"][:shp.L], sess["w"], dtype=shp.idx_dtype, q_scale=sess["q_scale"],
                                k_scale=None if sess["k_scale"] is None else sess["k_scale"][:shp.L], q_pos0=shp.L, causal=False, rows=rows)
    return O.indexer_scores(sess["q_idx"], sess["k_idx"], sess["w"], dtype=shp.idx_dtype, q_scale=sess["q_scale"], k_scale=sess["k_scale"],
                            recency=sess["recency"], q_pos0=shp.L, causal=True, rows=rows)


def assert_scores_close(got_rows: np.ndarray, ref_rows: np.ndarray, rel: float, what: str = ""):
    """|got - ref| <= rel * max(|ref|, rms(ref row)) on visible entries; masked entries exactly -inf on both sides."""
    assert got_rows.shape == ref_rows.shape
    for i in range(ref_rows.shape[0]):
        ref, got = ref_rows[i], got_rows[i].astype(np.float64)
        vis = np.isfinite(ref)
        assert np.array_equal(np.isneginf(got), ~vis), f"{what}: mask pattern differs in row {i}"
        if not vis.any():
            continue
        rms = np.sqrt(np.mean(ref[vis] ** 2))
        tol = rel * np.maximum(np.abs(ref[vis]), rms)
        err = np.abs(got[vis] - ref[vis])
        bad = err > tol
        assert not bad.any(), f"{what}: row {i}: {bad.sum()} entries off, worst {err.max():.3e} (tol {tol[np.argmax(err)]:.3e})"


def assert_attention_close(got: np.ndarray, ref: np.ndarray, what: str = ""):
    """Absolute bounds (max-abs 2e-2, mean-abs 2e-3) plus bounds relative to the output scale."""
    err = np.abs(got - ref)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3, f"{what}: abs err max {err.max():.3e} mean {err.mean():.3e}"
    scale_max, scale_mean = np.abs(ref).max(), np.abs(ref).mean()
    assert err.max() <= 2e-2 * scale_max + 1e-30, f"{what}: max err {err.max():.3e} vs 2e-2*max|o| {2e-2 * scale_max:.3e}"
    assert err.mean() <= 1e-2 * scale_mean + 1e-30, f"{what}: mean err {err.mean():.3e} vs 1e-2*mean|o| {1e-2 * scale_mean:.3e}"


def page_lists_from_device(out, want_miss=True):
    counts = out["counts"].cpu().numpy()
    n_pages, n_runs, n_miss, n_miss_runs = [int(c) for c in counts]
    res = {
        "pages": out["pages"][:n_pages].cpu().numpy().tolist(),
        "runs": [tuple(r) for r in out["runs"][:n_runs].cpu().numpy().tolist()],
    }
    if want_miss:
        res["miss"] = out["miss_pages"][:n_miss].cpu().numpy().tolist()
        res["miss_runs"] = [tuple(r) for r in out["miss_runs"][:n_miss_runs].cpu().numpy().tolist()]
    return res


def bitmap_to_pages(bitmap: torch.Tensor, n_phys_pages: int):
    words = bitmap.cpu().numpy().view(np.uint32)
    bits = np.unpackbits(words.view(np.uint8), bitorder="little")[:n_phys_pages]
    return np.nonzero(bits)[0].tolist()
