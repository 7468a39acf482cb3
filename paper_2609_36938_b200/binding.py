"""ctypes binding of libjanus.so: same names as the C entry points, argument marshalling only.

Tensors are torch CUDA tensors (torch provides device memory and the stream, nothing else); every
step runs in the library's kernels.  There is no CPU fallback: if the library is missing or the call
fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, Optional, Tuple

import torch

_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG_DIR, "libjanus.so")

JANUS_OK = 0
ERR_NAMES = {1: "JANUS_ERR_INVALID_ARG", 2: "JANUS_ERR_UNSUPPORTED", 3: "JANUS_ERR_WORKSPACE_TOO_SMALL", 4: "JANUS_ERR_CUDA"}
DEV_NAMES = {101: "JANUS_DEV_INDEX_OUT_OF_RANGE", 102: "JANUS_DEV_CAPACITY_EXCEEDED", 103: "JANUS_DEV_WAIT_TIMEOUT"}
DTYPE_BF16, DTYPE_FP8_E4M3, DTYPE_FP8_Q_FP4_K = 0, 1, 2
MBAR_MAX_POLLS = 1 << 16      # the kernels' limit on polls of one in-kernel wait (csrc/sm100_ptx.cuh)

# every symbol include/janus.h declares
EXPORTS = [
    "janus_version", "janus_last_cuda_error",
    "janus_indexer_scores_workspace_size", "janus_indexer_scores",
    "janus_topk_workspace_size", "janus_topk",
    "janus_indexer_topk_workspace_size", "janus_indexer_topk", "janus_indexer_topk_static", "janus_indexer_topk_fallback_counter_offset",
    "janus_page_demand_workspace_size", "janus_page_demand", "janus_page_union",
    "janus_sparse_attn_prefill_workspace_size", "janus_sparse_attn_prefill",
    "janus_indexer_scores_batch", "janus_topk_batch", "janus_page_demand_batch", "janus_sparse_attn_decode",
    "janus_topk_entries", "janus_entry_expand", "janus_entry_pool_scores",
    "janus_selftest_bounded_wait", "janus_fp8_mma_probe",
]


class JanusError(RuntimeError):
    pass


_lib = None


def load() -> ctypes.CDLL:
    """Loads libjanus.so (built in-tree by paper_2609_36938_b200.build).  Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise JanusError(f"{LIB_PATH} not found: build it first (python -m paper_2609_36938_b200.build); there is no fallback path")
    lib = ctypes.CDLL(LIB_PATH)
    c_i, c_i64, c_p, c_f, c_sz = ctypes.c_int, ctypes.c_int64, ctypes.c_void_p, ctypes.c_float, ctypes.c_size_t
    lib.janus_version.restype = c_i
    lib.janus_last_cuda_error.restype = c_i
    lib.janus_indexer_scores_workspace_size.restype = c_sz
    lib.janus_indexer_scores_workspace_size.argtypes = [c_i, c_i, c_i, c_i64, c_i]
    lib.janus_indexer_scores.restype = c_i
    lib.janus_indexer_scores.argtypes = [c_p, c_i64, c_p, c_i64, c_p, c_p, c_i64, c_p, c_p, c_p, c_i, c_i, c_i, c_i64, c_i64, c_i, c_i,
                                         c_p, c_i64, c_p, c_sz, c_p, c_p]
    lib.janus_topk_workspace_size.restype = c_sz
    lib.janus_topk_workspace_size.argtypes = [c_i, c_i64, c_i]
    lib.janus_topk.restype = c_i
    lib.janus_topk.argtypes = [c_p, c_i64, c_i, c_i64, c_i64, c_i, c_i, c_p, c_p, c_p, c_p, c_sz, c_p, c_p]
    lib.janus_indexer_topk_workspace_size.restype = c_sz
    lib.janus_indexer_topk_workspace_size.argtypes = [c_i, c_i, c_i, c_i64, c_i64, c_i, c_i, c_i]
    lib.janus_indexer_topk_fallback_counter_offset.restype = c_i64
    lib.janus_indexer_topk_fallback_counter_offset.argtypes = [c_i, c_i, c_i, c_i64, c_i64, c_i, c_i, c_i]
    lib.janus_indexer_topk.restype = c_i
    lib.janus_indexer_topk.argtypes = [c_p, c_i64, c_p, c_i64, c_p, c_p, c_i64, c_p, c_p, c_p, c_i, c_i, c_i, c_i64, c_i64, c_i, c_i, c_i,
                                       c_p, c_p, c_p, c_p, c_sz, c_p, c_p]
    lib.janus_indexer_topk_static.restype = c_i
    lib.janus_indexer_topk_static.argtypes = [c_p, c_i64, c_p, c_i64, c_p, c_p, c_i64, c_p, c_p, c_p, c_i, c_i, c_i, c_i64, c_i64, c_i, c_i, c_i,
                                              c_p, c_p, c_p, c_p, c_p]
    lib.janus_page_demand_workspace_size.restype = c_sz
    lib.janus_page_demand_workspace_size.argtypes = [c_i64, c_i, c_i64]
    lib.janus_page_demand.restype = c_i
    lib.janus_page_demand.argtypes = [c_p, c_i64, c_i, c_i64, c_i, c_p, c_i64, c_i64, c_p, c_p, c_p, c_p, c_p, c_p, c_p, c_p, c_p, c_p,
                                      c_i64, c_p, c_sz, c_p, c_p]
    lib.janus_page_union.restype = c_i
    lib.janus_page_union.argtypes = [c_p, c_p, c_i64, c_p]
    lib.janus_sparse_attn_prefill_workspace_size.restype = c_sz
    lib.janus_sparse_attn_prefill_workspace_size.argtypes = [c_i, c_i, c_i, c_i, c_i]
    lib.janus_sparse_attn_prefill.restype = c_i
    lib.janus_sparse_attn_prefill.argtypes = [c_p, c_i, c_i, c_i, c_p, c_p, c_i64, c_i64, c_i64, c_i, c_i, c_p, c_i, c_i, c_p, c_i64,
                                              c_f, c_p, c_p, c_p, c_sz, c_p, c_p]
    lib.janus_indexer_scores_batch.restype = c_i
    lib.janus_indexer_scores_batch.argtypes = [c_p, c_p, c_i64, c_p, c_p, c_i64, c_p, c_p, c_p, c_i, c_i, c_i, c_p, c_i64, c_i64, c_i, c_p, c_p, c_p]
    lib.janus_topk_batch.restype = c_i
    lib.janus_topk_batch.argtypes = [c_p, c_p, c_p, c_i, c_i, c_p, c_p, c_p, c_p, c_p]
    lib.janus_page_demand_batch.restype = c_i
    lib.janus_page_demand_batch.argtypes = [c_p, c_i64, c_i, c_p, c_i, c_p, c_p, c_i64, c_p, c_p, c_p, c_p, c_p, c_p, c_p, c_p, c_p, c_p, c_i64,
                                            c_p, c_p]
    lib.janus_sparse_attn_decode.restype = c_i
    lib.janus_sparse_attn_decode.argtypes = [c_p, c_i, c_i, c_i, c_p, c_p, c_i64, c_i64, c_i64, c_i, c_i, c_p, c_i, c_i, c_p, c_p, c_f, c_p, c_p,
                                             c_p, c_p]
    lib.janus_topk_entries.restype = c_i
    lib.janus_topk_entries.argtypes = [c_p, c_i64, c_i, c_i64, c_i64, c_i, c_i, c_p, c_p, c_p, c_p, c_p]
    lib.janus_entry_pool_scores.restype = c_i
    lib.janus_entry_pool_scores.argtypes = [c_p, c_i64, c_i, c_i64, c_i64, c_i, c_i, c_p, c_i64, c_p]
    lib.janus_entry_expand.restype = c_i
    lib.janus_entry_expand.argtypes = [c_p, c_i, c_i, c_i, c_i64, c_p, c_p]
    lib.janus_selftest_bounded_wait.restype = c_i
    lib.janus_selftest_bounded_wait.argtypes = [c_i, c_p, c_p, c_p]
    lib.janus_fp8_mma_probe.restype = c_i
    lib.janus_fp8_mma_probe.argtypes = [c_i, c_i, ctypes.POINTER(ctypes.c_double), c_p, c_p]
    _lib = lib
    return lib


def _check(rc: int, what: str) -> None:
    if rc != JANUS_OK:
        extra = f" (cudaError {load().janus_last_cuda_error()})" if rc == 4 else ""
        raise JanusError(f"{what} failed: {ERR_NAMES.get(rc, rc)}{extra}")


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise JanusError("expected a CUDA tensor (the library takes device pointers)")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


_status: Dict[int, torch.Tensor] = {}


def dev_status_tensor() -> torch.Tensor:
    """The device status word the binding passes to every call on the current device."""
    d = torch.cuda.current_device()
    if d not in _status:
        _status[d] = torch.zeros(1, dtype=torch.int32, device=f"cuda:{d}")
    return _status[d]


def check_dev_status(reset: bool = True) -> None:
    """Synchronises and raises if a kernel reported a device-side condition."""
    st = dev_status_tensor()
    v = int(st.item())
    if reset and v != 0:
        st.zero_()
    if v != 0:
        raise JanusError(f"device status {DEV_NAMES.get(v, v)}")


def janus_version() -> int:
    return int(load().janus_version())


def _idx_dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return DTYPE_BF16
    if t.dtype in (torch.uint8, torch.float8_e4m3fn):
        return DTYPE_FP8_E4M3
    raise JanusError(f"indexer operands must be bfloat16 or E4M3 bytes, got {t.dtype}")


def _idx_dtypes(q_idx: torch.Tensor, k_idx: torch.Tensor, keys_fp4: bool):
    """(dtype code, key row stride in elements) of a query / key pair."""
    dtype = _idx_dtype_code(q_idx)
    if keys_fp4:
        if dtype != DTYPE_FP8_E4M3 or k_idx.dtype != torch.uint8:
            raise JanusError("FP4 keys are uint8 (two per byte) and go with E4M3 queries")
        return DTYPE_FP8_Q_FP4_K, k_idx.stride(0) * 2
    if _idx_dtype_code(k_idx) != dtype:
        raise JanusError("q_idx and k_idx must share a dtype")
    return dtype, k_idx.stride(0)


def janus_indexer_scores(q_idx: torch.Tensor, k_idx: torch.Tensor, w: torch.Tensor, *, q_scale: Optional[torch.Tensor] = None,
                         k_scale: Optional[torch.Tensor] = None, row_bias: Optional[torch.Tensor] = None,
                         col_bias: Optional[torch.Tensor] = None, q_pos0: int = 0, causal: bool = True,
                         scores: Optional[torch.Tensor] = None, keys_fp4: bool = False) -> torch.Tensor:
    """scores[t,s] = sum_h w[t,h] relu(<q_idx[t,h], k_idx[s]>) (+ row_bias[t] col_bias[s]); -inf where masked.
    q_idx [M,H,D], k_idx [n_keys,D] (bf16 or E4M3 bytes), w [M,H] fp32.  Returns [M, ld] fp32, ld >= n_keys.
    keys_fp4: k_idx is uint8 [n_keys, D/2], FP4 E2M1 packed two per byte (queries FP8)."""
    lib = load()
    M, H, D = q_idx.shape
    n_keys = k_idx.shape[0]
    dtype, k_stride = _idx_dtypes(q_idx, k_idx, keys_fp4)
    if scores is None:
        ld = (n_keys + 31) // 32 * 32
        scores = torch.empty((M, ld), dtype=torch.float32, device=q_idx.device)
    qs_stride = 0
    if q_scale is not None and q_scale.dim() == 2:
        qs_stride = H
    rc = lib.janus_indexer_scores(_ptr(q_idx), q_idx.stride(0), _ptr(k_idx), k_stride, _ptr(w), _ptr(q_scale), qs_stride,
                                  _ptr(k_scale), _ptr(row_bias), _ptr(col_bias), M, H, D, n_keys, int(q_pos0), int(bool(causal)), dtype,
                                  _ptr(scores), scores.stride(0), None, 0, _ptr(dev_status_tensor()), _stream())
    _check(rc, "janus_indexer_scores")
    return scores


def janus_topk(scores: torch.Tensor, n_keys: int, k: int, *, q_pos0: int = 0, causal: bool = True, want_count: bool = True,
               want_kth: bool = True, idx: Optional[torch.Tensor] = None):
    """Per-row top-k over the visible prefix.  Returns (idx [M,k] int32 with -1 padding, count [M] | None, kth [M] | None).
    ``idx``: an [M,k] int32 buffer to write into."""
    lib = load()
    M = scores.shape[0]
    if idx is None:
        idx = torch.empty((M, k), dtype=torch.int32, device=scores.device)
    count = torch.empty((M,), dtype=torch.int32, device=scores.device) if want_count else None
    kth = torch.empty((M,), dtype=torch.float32, device=scores.device) if want_kth else None
    rc = lib.janus_topk(_ptr(scores), scores.stride(0), M, int(n_keys), int(q_pos0), int(bool(causal)), int(k), _ptr(idx), _ptr(count),
                        _ptr(kth), None, 0, _ptr(dev_status_tensor()), _stream())
    _check(rc, "janus_topk")
    return idx, count, kth


def janus_indexer_topk(q_idx: torch.Tensor, k_idx: torch.Tensor, w: torch.Tensor, k: int, *, q_scale: Optional[torch.Tensor] = None,
                       k_scale: Optional[torch.Tensor] = None, row_bias: Optional[torch.Tensor] = None,
                       col_bias: Optional[torch.Tensor] = None, q_pos0: int = 0, causal: bool = True, want_count: bool = True,
                       want_kth: bool = True, workspace: Optional[torch.Tensor] = None, idx: Optional[torch.Tensor] = None,
                       keys_fp4: bool = False):
    """Indexer scores and per-row top-k in one call, without the score matrix.  Returns (idx [M,k], count | None, kth | None).
    `workspace` (uint8 CUDA tensor) is allocated if not given or too small; pass one to reuse it across calls; `idx` likewise.
    keys_fp4: k_idx is uint8 [n_keys, D/2], FP4 E2M1 packed two per byte (queries FP8); this format goes through a score
    matrix inside the workspace."""
    lib = load()
    M, H, D = q_idx.shape
    n_keys = k_idx.shape[0]
    dtype, k_stride = _idx_dtypes(q_idx, k_idx, keys_fp4)
    need = int(lib.janus_indexer_topk_workspace_size(M, H, D, n_keys, int(q_pos0), int(bool(causal)), dtype, int(k)))
    if workspace is None or workspace.numel() < need:
        workspace = torch.empty((max(need, 16),), dtype=torch.uint8, device=q_idx.device)
    if idx is None:
        idx = torch.empty((M, k), dtype=torch.int32, device=q_idx.device)
    elif idx.shape != (M, k) or idx.dtype != torch.int32 or not idx.is_contiguous():
        raise JanusError("idx must be a contiguous [M, k] int32 tensor")
    count = torch.empty((M,), dtype=torch.int32, device=q_idx.device) if want_count else None
    kth = torch.empty((M,), dtype=torch.float32, device=q_idx.device) if want_kth else None
    qs_stride = H if (q_scale is not None and q_scale.dim() == 2) else 0
    rc = lib.janus_indexer_topk(_ptr(q_idx), q_idx.stride(0), _ptr(k_idx), k_stride, _ptr(w), _ptr(q_scale), qs_stride, _ptr(k_scale),
                                _ptr(row_bias), _ptr(col_bias), M, H, D, n_keys, int(q_pos0), int(bool(causal)), dtype, int(k), _ptr(idx),
                                _ptr(count), _ptr(kth), _ptr(workspace), workspace.numel(), _ptr(dev_status_tensor()), _stream())
    _check(rc, "janus_indexer_topk")
    return idx, count, kth


STATIC_SCRATCH_BYTES = 64 << 20


def janus_indexer_topk_static(q_idx: torch.Tensor, k_idx: torch.Tensor, w: torch.Tensor, k: int, idx: torch.Tensor, *,
                              count: Optional[torch.Tensor] = None, kth: Optional[torch.Tensor] = None,
                              q_scale: Optional[torch.Tensor] = None, k_scale: Optional[torch.Tensor] = None,
                              row_bias: Optional[torch.Tensor] = None, col_bias: Optional[torch.Tensor] = None, q_pos0: int = 0,
                              causal: bool = True) -> None:
    """janus_indexer_topk on the scratch array built into the library.  Allocates nothing: the caller passes the outputs
    (`idx` [M, k] int32, optionally `count` [M] int32 and `kth` [M] fp32).  Raises if the problem needs more scratch than
    STATIC_SCRATCH_BYTES.  Calls on one device share the array: keep them ordered on the device."""
    lib = load()
    M, H, D = q_idx.shape
    n_keys = k_idx.shape[0]
    dtype = _idx_dtype_code(q_idx)
    if _idx_dtype_code(k_idx) != dtype:
        raise JanusError("q_idx and k_idx must share a dtype")
    if idx.shape != (M, k) or idx.dtype != torch.int32 or not idx.is_contiguous():
        raise JanusError("idx must be a contiguous [M, k] int32 tensor")
    qs_stride = H if (q_scale is not None and q_scale.dim() == 2) else 0
    rc = lib.janus_indexer_topk_static(_ptr(q_idx), q_idx.stride(0), _ptr(k_idx), k_idx.stride(0), _ptr(w), _ptr(q_scale), qs_stride,
                                       _ptr(k_scale), _ptr(row_bias), _ptr(col_bias), M, H, D, n_keys, int(q_pos0), int(bool(causal)), dtype,
                                       int(k), _ptr(idx), _ptr(count), _ptr(kth), _ptr(dev_status_tensor()), _stream())
    _check(rc, "janus_indexer_topk_static")


def page_demand_buffers(n_phys_pages: int, capacity: Optional[int] = None, want_miss: bool = True, device="cuda") -> Dict[str, torch.Tensor]:
    """Output buffers of janus_page_demand / janus_page_demand_batch for a pool of `n_phys_pages` pages.  Allocate once and
    pass as ``out=`` to keep allocations (and the fill of the count words) out of a serving loop."""
    cap = int(capacity) if capacity is not None else int(n_phys_pages)
    n_words = (int(n_phys_pages) + 31) // 32
    out = {
        "bitmap": torch.empty((n_words,), dtype=torch.int32, device=device),
        "pages": torch.empty((max(cap, 1),), dtype=torch.int32, device=device),
        "runs": torch.empty((max(cap, 1), 2), dtype=torch.int32, device=device),
        "counts": torch.zeros((4,), dtype=torch.int32, device=device),   # n_pages, n_runs, n_miss, n_miss_runs (each written by the call that asks for it)
    }
    if want_miss:
        out["miss_pages"] = torch.empty((max(cap, 1),), dtype=torch.int32, device=device)
        out["miss_runs"] = torch.empty((max(cap, 1), 2), dtype=torch.int32, device=device)
    return out


def _page_demand_out_args(out: Dict[str, torch.Tensor], want_miss: bool):
    cp = out["counts"].data_ptr()
    miss_args = [None, None, None, None]
    if want_miss:
        miss_args = [_ptr(out["miss_pages"]), cp + 8, _ptr(out["miss_runs"]), cp + 12]
    return cp, miss_args


def janus_page_demand(idx: torch.Tensor, *, demand_limit: int, page_size: int, page_table: torch.Tensor, n_phys_pages: int,
                      predicted_bitmap: Optional[torch.Tensor] = None, capacity: Optional[int] = None, want_miss: bool = True,
                      out: Optional[Dict[str, torch.Tensor]] = None):
    """Union of selected history tokens as a physical-page bitmap, ascending page list, maximal runs and the miss set
    against ``predicted_bitmap``.  Returns a dict of device tensors; the counts stay on the device (no host sync).
    ``out``: buffers from page_demand_buffers() to write into (nothing is allocated or filled by this call then)."""
    lib = load()
    n_rows, k = idx.shape
    if out is None:
        out = page_demand_buffers(n_phys_pages, capacity, want_miss, idx.device)
    else:
        want_miss = want_miss and "miss_pages" in out
    cap = out["pages"].numel() if capacity is None else int(capacity)
    cp, miss_args = _page_demand_out_args(out, want_miss)
    rc = lib.janus_page_demand(_ptr(idx), n_rows, k, int(demand_limit), int(page_size), _ptr(page_table), page_table.numel(),
                               int(n_phys_pages), _ptr(predicted_bitmap), _ptr(out["bitmap"]), _ptr(out["pages"]), cp,
                               _ptr(out["runs"]), cp + 4, *miss_args, cap, None, 0, _ptr(dev_status_tensor()), _stream())
    _check(rc, "janus_page_demand")
    return out


def janus_page_union(dst: torch.Tensor, src: torch.Tensor, n_phys_pages: int) -> torch.Tensor:
    """dst |= src for two page bitmaps written by janus_page_demand (union of per-shard predicted sets, Sec. 4.2)."""
    _check(load().janus_page_union(_ptr(dst), _ptr(src), int(n_phys_pages), _stream()), "janus_page_union")
    return dst


def janus_sparse_attn_prefill(q: torch.Tensor, k_pool: torch.Tensor, v_pool: torch.Tensor, idx: torch.Tensor, *,
                              page_table: torch.Tensor, page_size: int, softmax_scale: float, d_v: int,
                              want_lse: bool = True, out: Optional[torch.Tensor] = None):
    """Attention of each new token over its selected rows only.  q [M,H_q,d_qk] bf16; pools
    [n_phys_pages, page_size, n_kv_heads, d] bf16 (v_pool may be k_pool itself: value = first d_v dims of the key row);
    idx [M,k] int32.  Returns (out [M,H_q,d_v] bf16, lse [M,H_q] fp32 | None)."""
    lib = load()
    M, H_q, d_qk = q.shape
    n_kv = k_pool.shape[2]
    if out is None:
        out = torch.empty((M, H_q, d_v), dtype=torch.bfloat16, device=q.device)
    lse = torch.empty((M, H_q), dtype=torch.float32, device=q.device) if want_lse else None
    if v_pool.data_ptr() != k_pool.data_ptr() and v_pool.stride() != k_pool.stride():
        raise JanusError("k_pool and v_pool must share strides")
    rc = lib.janus_sparse_attn_prefill(_ptr(q), M, H_q, d_qk, _ptr(k_pool), _ptr(v_pool), k_pool.stride(0), k_pool.stride(1),
                                       k_pool.stride(2), n_kv, int(d_v), _ptr(idx), idx.shape[1], int(page_size), _ptr(page_table),
                                       page_table.numel(), float(softmax_scale), _ptr(out), _ptr(lse), None, 0,
                                       _ptr(dev_status_tensor()), _stream())
    _check(rc, "janus_sparse_attn_prefill")
    return out, lse


# ---- entry granularity ---------------------------------------------------------------------------------------------
def janus_topk_entries(scores: torch.Tensor, n_entries: int, k: int, *, q_pos0: int, entry_size: int, want_count: bool = True,
                       want_kth: bool = True):
    """Top-k over entries of `entry_size` tokens: row t may select entries 0 .. (q_pos0 + t) // entry_size."""
    lib = load()
    M = scores.shape[0]
    idx = torch.empty((M, k), dtype=torch.int32, device=scores.device)
    count = torch.empty((M,), dtype=torch.int32, device=scores.device) if want_count else None
    kth = torch.empty((M,), dtype=torch.float32, device=scores.device) if want_kth else None
    rc = lib.janus_topk_entries(_ptr(scores), scores.stride(0), M, int(n_entries), int(q_pos0), int(entry_size), int(k), _ptr(idx),
                                _ptr(count), _ptr(kth), _ptr(dev_status_tensor()), _stream())
    _check(rc, "janus_topk_entries")
    return idx, count, kth


def janus_entry_pool_scores(scores: torch.Tensor, n_keys: int, *, entry_size: int, q_pos0: int = 0, causal: bool = True) -> torch.Tensor:
    """Entry scores as the maximum over each entry's visible token scores.  Returns [M, ld] fp32, ld = n_entries rounded up to 4."""
    M = scores.shape[0]
    n_entries = (int(n_keys) + entry_size - 1) // entry_size
    ld = max(4, (n_entries + 3) // 4 * 4)
    out = torch.empty((M, ld), dtype=torch.float32, device=scores.device)
    _check(load().janus_entry_pool_scores(_ptr(scores), scores.stride(0), M, int(n_keys), int(q_pos0), int(bool(causal)), int(entry_size),
                                          _ptr(out), ld, _stream()), "janus_entry_pool_scores")
    return out


def janus_entry_expand(idx_entries: torch.Tensor, *, q_pos0: int, entry_size: int) -> torch.Tensor:
    """Entry selection [M, k_e] -> token selection [M, k_e * entry_size] (tokens after the row's position become -1)."""
    lib = load()
    M, k_e = idx_entries.shape
    out = torch.empty((M, k_e * entry_size), dtype=torch.int32, device=idx_entries.device)
    rc = lib.janus_entry_expand(_ptr(idx_entries), M, k_e, int(entry_size), int(q_pos0), _ptr(out), _stream())
    _check(rc, "janus_entry_expand")
    return out


# ---- decode step over a batch of sessions -------------------------------------------------------------------------
def janus_indexer_scores_batch(q_idx: torch.Tensor, k_idx: torch.Tensor, w: torch.Tensor, key_offsets: torch.Tensor, max_keys: int, *,
                               q_scale: Optional[torch.Tensor] = None, k_scale: Optional[torch.Tensor] = None,
                               row_bias: Optional[torch.Tensor] = None, col_bias: Optional[torch.Tensor] = None,
                               scores: Optional[torch.Tensor] = None, keys_fp4: bool = False) -> torch.Tensor:
    """One query row per session against that session's keys.  q_idx [B,H,D]; k_idx [total_keys, D] (sessions concatenated);
    key_offsets [B+1] int64 on the device.  Returns scores [total_keys] fp32 in the same row numbering as k_idx.
    keys_fp4: k_idx is uint8 [total_keys, D/2], FP4 E2M1 packed two per byte (queries FP8)."""
    lib = load()
    B_, H, D = q_idx.shape
    total = k_idx.shape[0]
    dtype = 2 if keys_fp4 else _idx_dtype_code(q_idx)
    k_stride = k_idx.stride(0) * (2 if keys_fp4 else 1)
    if scores is None:
        scores = torch.empty((total,), dtype=torch.float32, device=q_idx.device)
    qs_stride = H if (q_scale is not None and q_scale.dim() == 2) else 0
    rc = lib.janus_indexer_scores_batch(_ptr(q_idx), _ptr(k_idx), k_stride, _ptr(w), _ptr(q_scale), qs_stride, _ptr(k_scale),
                                        _ptr(row_bias), _ptr(col_bias), B_, H, D, _ptr(key_offsets), total, int(max_keys), dtype,
                                        _ptr(scores), _ptr(dev_status_tensor()), _stream())
    _check(rc, "janus_indexer_scores_batch")
    return scores


def janus_topk_batch(scores: torch.Tensor, row_offsets: torch.Tensor, k: int, *, row_lengths: Optional[torch.Tensor] = None,
                     want_count: bool = True, want_kth: bool = True):
    """Top-k of every ragged row scores[row_offsets[b] : row_offsets[b] + row_lengths[b]] (up to the next offset when
    row_lengths is None).  Returns (idx [B,k], count | None, kth | None)."""
    lib = load()
    B_ = row_offsets.numel() - 1
    idx = torch.empty((B_, k), dtype=torch.int32, device=scores.device)
    count = torch.empty((B_,), dtype=torch.int32, device=scores.device) if want_count else None
    kth = torch.empty((B_,), dtype=torch.float32, device=scores.device) if want_kth else None
    rc = lib.janus_topk_batch(_ptr(scores), _ptr(row_offsets), _ptr(row_lengths), B_, int(k), _ptr(idx), _ptr(count), _ptr(kth), _ptr(dev_status_tensor()),
                              _stream())
    _check(rc, "janus_topk_batch")
    return idx, count, kth


def janus_page_demand_batch(idx: torch.Tensor, *, demand_limits: torch.Tensor, page_size: int, page_tables: torch.Tensor,
                            table_offsets: torch.Tensor, n_phys_pages: int, predicted_bitmap: Optional[torch.Tensor] = None,
                            capacity: Optional[int] = None, want_miss: bool = True, out: Optional[Dict[str, torch.Tensor]] = None):
    """janus_page_demand over rows that each have their own page table and history length (int64 device tensors)."""
    lib = load()
    n_rows, k = idx.shape
    if out is None:
        out = page_demand_buffers(n_phys_pages, capacity, want_miss, idx.device)
    else:
        want_miss = want_miss and "miss_pages" in out
    cap = out["pages"].numel() if capacity is None else int(capacity)
    cp, miss_args = _page_demand_out_args(out, want_miss)
    rc = lib.janus_page_demand_batch(_ptr(idx), n_rows, k, _ptr(demand_limits), int(page_size), _ptr(page_tables), _ptr(table_offsets),
                                     int(n_phys_pages), _ptr(predicted_bitmap), _ptr(out["bitmap"]), _ptr(out["pages"]), cp, _ptr(out["runs"]),
                                     cp + 4, *miss_args, cap, _ptr(dev_status_tensor()), _stream())
    _check(rc, "janus_page_demand_batch")
    return out


def janus_sparse_attn_decode(q: torch.Tensor, k_pool: torch.Tensor, v_pool: torch.Tensor, idx: torch.Tensor, *, page_tables: torch.Tensor,
                             table_offsets: torch.Tensor, page_size: int, softmax_scale: float, d_v: int, want_lse: bool = True,
                             out: Optional[torch.Tensor] = None):
    """janus_sparse_attn_prefill with one query row per session and per-row page tables (table_offsets [B+1] int64)."""
    lib = load()
    B_, H_q, d_qk = q.shape
    n_kv = k_pool.shape[2]
    if out is None:
        out = torch.empty((B_, H_q, d_v), dtype=torch.bfloat16, device=q.device)
    lse = torch.empty((B_, H_q), dtype=torch.float32, device=q.device) if want_lse else None
    rc = lib.janus_sparse_attn_decode(_ptr(q), B_, H_q, d_qk, _ptr(k_pool), _ptr(v_pool), k_pool.stride(0), k_pool.stride(1), k_pool.stride(2),
                                      n_kv, int(d_v), _ptr(idx), idx.shape[1], int(page_size), _ptr(page_tables), _ptr(table_offsets),
                                      float(softmax_scale), _ptr(out), _ptr(lse), _ptr(dev_status_tensor()), _stream())
    _check(rc, "janus_sparse_attn_decode")
    return out, lse


# ---- diagnostics ---------------------------------------------------------------------------------------------------
def janus_selftest_bounded_wait(max_polls: int = 256) -> Tuple[int, float]:
    """Runs the kernels' bounded wait on a barrier nobody arrives on.  Returns (status word afterwards, seconds the wait took);
    the status word is cleared again."""
    st = dev_status_tensor()
    st.zero_()
    ns = torch.zeros(1, dtype=torch.int64, device=st.device)
    _check(load().janus_selftest_bounded_wait(int(max_polls), _ptr(ns), _ptr(st), _stream()), "janus_selftest_bounded_wait")
    v = int(st.item())
    st.zero_()
    return v, float(ns.item()) * 1e-9


def janus_fp8_mma_probe(n_ctas: int, fills_per_cta: int) -> float:
    """Launches the dense FP8 tensor-rate probe on the current stream; returns the launch's flop count."""
    flop = ctypes.c_double(0.0)
    _check(load().janus_fp8_mma_probe(int(n_ctas), int(fills_per_cta), ctypes.byref(flop), _ptr(dev_status_tensor()), _stream()), "janus_fp8_mma_probe")
    return flop.value


# ---- helpers to move generator output (bit patterns) onto the device -------------------------------------------
def to_device(x, kind: str, device="cuda") -> Optional[torch.Tensor]:
    """numpy array -> CUDA tensor.  kind: "bf16" (uint16 bit patterns), "fp8" (uint8 codes), "f32", "i32"."""
    import numpy as np

    if x is None:
        return None
    if kind == "bf16":
        return torch.from_numpy(np.ascontiguousarray(x).view(np.int16)).view(torch.bfloat16).to(device)
    if kind == "fp8":
        return torch.from_numpy(np.ascontiguousarray(x)).to(device)
    if kind == "f32":
        return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(device)
    if kind == "i32":
        return torch.from_numpy(np.ascontiguousarray(x, dtype=np.int32)).to(device)
    raise ValueError(kind)
