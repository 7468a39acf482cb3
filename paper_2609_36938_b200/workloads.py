"""Seeded synthetic append-prefill sessions.

This module only *draws inputs*: random tensors, their rounding to the storage
formats (bf16 / FP8 E4M3 bit patterns), page tables and the shapes of the five
benchmark configurations.  It holds none of the method's arithmetic (no indexer,
no selection, no page logic, no attention) and is the one module that both the
CUDA path's callers and the CPU oracle's callers draw inputs from; it imports
neither of them.

The paper's workloads are agentic traces (history tens to hundreds of thousands
of tokens, appended queries of hundreds to thousands, Table 2); these traces are
not available, so seeded synthetic sessions with the same length ranges stand in
for them.  Every tensor comes from
``numpy.random.Generator(PCG64(SeedSequence([seed, config_id, tensor_id])))``.

Naming: ``L`` history tokens, ``M`` new (appended) tokens, ``S = L + M`` keys
(the paper writes P for the history and L for the appended query, Table 1).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional

import numpy as np

# tensor ids inside one (seed, config) stream
_T_QIDX, _T_KIDX, _T_W, _T_QSCALE, _T_KSCALE, _T_Q, _T_POOL, _T_VPOOL, _T_PERM, _T_NOISE, _T_STRUCT, _T_LEN = range(12)


def _rng(seed: int, config_id: int, tensor_id: int, sub: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, config_id, tensor_id, sub])))


# ----------------------------------------------------------------------------
# storage-format rounding (inputs only)
# ----------------------------------------------------------------------------
def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round-to-nearest-even."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def to_e4m3_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> FP8 E4M3 (OCP e4m3fn) bytes, round-to-nearest-even, saturating at +-448."""
    import torch

    t = torch.from_numpy(np.clip(np.ascontiguousarray(x, dtype=np.float32), -448.0, 448.0))
    return t.to(torch.float8_e4m3fn).view(torch.uint8).numpy().copy()


def _normal_bf16(rng: np.random.Generator, shape, scale: float = 1.0, chunk: int = 1 << 24) -> np.ndarray:
    """bf16 bits of scale * N(0,1), drawn in chunks to bound host memory."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16)
    for a in range(0, n, chunk):
        b = min(n, a + chunk)
        v = rng.standard_normal(b - a, dtype=np.float32)
        if scale != 1.0:
            v *= np.float32(scale)
        out[a:b] = to_bf16_bits(v)
    return out.reshape(shape)


# ----------------------------------------------------------------------------
# configurations
# ----------------------------------------------------------------------------
@dataclasses.dataclass(frozen=True)
class SessionShape:
    """Shape of one append-prefill session for one sparse layer."""

    config_id: int
    L: int                 # history tokens
    M: int                 # new tokens
    H_I: int               # indexer heads
    D_I: int               # indexer head dim
    k: int                 # top-k budget
    idx_dtype: str         # "bf16" | "fp8"
    attn: str              # "mha" | "latent"
    H_q: int               # attention query heads
    d_qk: int
    d_v: int
    n_kv_heads: int
    page_size: int = 64
    table: str = "identity"   # "identity" | "shuffled" | "fragmented"
    w_scale: float = 1.0
    structure: str = "iid"    # "iid" | "clustered"
    predicted: Optional[str] = None  # None | "noise0.3" | "cos0.8"

    @property
    def S(self) -> int:
        return self.L + self.M

    @property
    def n_logical_pages(self) -> int:
        return (self.S + self.page_size - 1) // self.page_size

    @property
    def softmax_scale(self) -> float:
        return 1.0 / math.sqrt(self.d_qk)


def config_shape(config_id: int, L: Optional[int] = None, M: Optional[int] = None, k: Optional[int] = None) -> SessionShape:
    """The five benchmark configurations (1-based).  ``L``/``M``/``k`` override the size for reduced test cases."""
    if config_id == 1:
        s = SessionShape(1, 4096, 256, 4, 64, 256, "bf16", "mha", 8, 128, 128, 8, table="identity",
                         w_scale=1.0, predicted="noise0.3")
    elif config_id == 2:
        s = SessionShape(2, 32768, 2048, 64, 128, 2048, "bf16", "latent", 128, 576, 512, 1, table="shuffled",
                         w_scale=1.0 / 8)
    elif config_id == 3:
        s = SessionShape(3, 131072, 4096, 64, 128, 2048, "fp8", "latent", 128, 576, 512, 1, table="shuffled",
                         w_scale=1.0 / 8)
    elif config_id == 4:
        # one session of the ragged batch; sizes are drawn by batch_shapes()
        s = SessionShape(4, 110592, 4352, 64, 128, 2048, "bf16", "latent", 128, 576, 512, 1, table="fragmented",
                         w_scale=1.0 / 8, predicted="cos0.8")
    elif config_id == 5:
        s = SessionShape(5, 262144, 8192, 64, 128, 2048, "fp8", "latent", 128, 576, 512, 1, table="shuffled",
                         w_scale=1.0 / 8, structure="clustered")
    else:
        raise ValueError(f"unknown config {config_id}")
    repl = {}
    if L is not None:
        repl["L"] = int(L)
    if M is not None:
        repl["M"] = int(M)
    if k is not None:
        repl["k"] = int(k)
    return dataclasses.replace(s, **repl) if repl else s


def batch_shapes(seed: int = 0, n_sessions: int = 8, L_range=(16384, 204800), M_range=(512, 8192)) -> List[SessionShape]:
    """Config 4: ragged batch, L ~ U{16K..200K}, M ~ U{512..8192} (not rounded to pages)."""
    rng = _rng(seed, 4, _T_LEN)
    base = config_shape(4)
    out = []
    for _ in range(n_sessions):
        L = int(rng.integers(L_range[0], L_range[1] + 1))
        M = int(rng.integers(M_range[0], M_range[1] + 1))
        out.append(dataclasses.replace(base, L=L, M=M))
    return out


# ----------------------------------------------------------------------------
# page tables
# ----------------------------------------------------------------------------
def make_page_table(shape: SessionShape, seed: int = 0) -> np.ndarray:
    n = shape.n_logical_pages
    if shape.table == "identity":
        return np.arange(n, dtype=np.int32)
    if shape.table == "shuffled":
        return _rng(seed, shape.config_id, _T_PERM).permutation(n).astype(np.int32)
    raise ValueError("fragmented tables are built for a whole batch: fragmented_page_tables()")


def fragmented_page_tables(shapes: List[SessionShape], seed: int = 0):
    """Shared physical pool for a batch: an allocator hands out chunks of 1..8 consecutive
    physical pages round-robin over the sessions until each has its ceil(S/page) pages.
    Returns (list of per-session page tables, n_phys_pages)."""
    rng = _rng(seed, 4, _T_PERM)
    need = [s.n_logical_pages for s in shapes]
    tables = [np.empty(n, dtype=np.int32) for n in need]
    have = [0] * len(shapes)
    nxt = 0
    while any(h < n for h, n in zip(have, need)):
        for b in range(len(shapes)):
            if have[b] >= need[b]:
                continue
            c = min(int(rng.integers(1, 9)), need[b] - have[b])
            tables[b][have[b]:have[b] + c] = np.arange(nxt, nxt + c, dtype=np.int32)
            have[b] += c
            nxt += c
    return tables, nxt


# ----------------------------------------------------------------------------
# one session
# ----------------------------------------------------------------------------
def _indexer_iid(shape: SessionShape, seed: int):
    cid = shape.config_id
    M, S, H, D = shape.M, shape.S, shape.H_I, shape.D_I
    q = _rng(seed, cid, _T_QIDX).standard_normal((M, H, D), dtype=np.float32)
    kk = _rng(seed, cid, _T_KIDX).standard_normal((S, D), dtype=np.float32)
    return q, kk


def _indexer_clustered(shape: SessionShape, seed: int):
    """Config 5 structure: 32 topical clusters laid out in segments, 4 large-norm sink keys,
    queries that lean toward the centroid of a cluster (switching every 256 new tokens)."""
    cid = shape.config_id
    M, L, S, H, D = shape.M, shape.L, shape.S, shape.H_I, shape.D_I
    rs = _rng(seed, cid, _T_STRUCT)
    C = rs.standard_normal((32, D), dtype=np.float32)
    seg_cluster = np.empty(S, dtype=np.int32)
    pos = 0
    while pos < S:
        ln = int(rs.integers(256, 4097))
        seg_cluster[pos:pos + ln] = int(rs.integers(0, 32))
        pos += ln
    kk = C[seg_cluster] + np.float32(0.5) * _rng(seed, cid, _T_KIDX).standard_normal((S, D), dtype=np.float32)
    n_sink = min(4, S)
    kk[:n_sink] = np.float32(8.0) * _rng(seed, cid, _T_KIDX, 1).standard_normal((n_sink, D), dtype=np.float32)
    g = rs.uniform(0.5, 1.5, size=H).astype(np.float32)
    cq = rs.integers(0, 32, size=(M + 255) // 256)
    cq_tok = np.repeat(cq, 256)[:M]
    q = g[None, :, None] * C[cq_tok][:, None, :] + _rng(seed, cid, _T_QIDX).standard_normal((M, H, D), dtype=np.float32)
    return q.astype(np.float32), kk.astype(np.float32)


def make_session(shape: SessionShape, seed: int = 0, *, with_attention: bool = True,
                 page_table: Optional[np.ndarray] = None, n_phys_pages: Optional[int] = None,
                 pool: Optional[Dict[str, np.ndarray]] = None) -> Dict[str, object]:
    """Draw every input of one session.  Tensors in storage formats are returned as bit patterns
    (uint16 for bf16, uint8 for E4M3); everything else is float32 / int32.

    ``page_table`` / ``n_phys_pages`` / ``pool`` let a batch share one physical pool (config 4)."""
    cid = shape.config_id
    M, L, S, H, D = shape.M, shape.L, shape.S, shape.H_I, shape.D_I
    out: Dict[str, object] = {"shape": shape}

    if shape.structure == "clustered":
        q, kk = _indexer_clustered(shape, seed)
    else:
        q, kk = _indexer_iid(shape, seed)
    w = (_rng(seed, cid, _T_W).uniform(0.0, 1.0, size=(M, H)) * shape.w_scale).astype(np.float32)
    out["w"] = w

    q_pred = None
    if shape.predicted == "noise0.3":
        q_pred = q + np.float32(0.3) * _rng(seed, cid, _T_NOISE).standard_normal(q.shape, dtype=np.float32)
    elif shape.predicted == "cos0.8":
        q_pred = np.float32(0.8) * q + np.float32(0.6) * _rng(seed, cid, _T_NOISE).standard_normal(q.shape, dtype=np.float32)

    if shape.idx_dtype == "bf16":
        out["q_idx"] = to_bf16_bits(q)
        out["k_idx"] = to_bf16_bits(kk)
        out["q_scale"] = None
        out["k_scale"] = None
        if q_pred is not None:
            out["q_pred"] = to_bf16_bits(q_pred)
    else:
        if shape.structure == "clustered":
            # calibrated scales so the structure survives quantisation
            k_scale = (np.maximum(np.abs(kk).max(axis=1), 1e-12) / 448.0).astype(np.float32)
            q_scale = (np.maximum(np.abs(q).max(axis=(0, 2)), 1e-12) / 448.0).astype(np.float32)
            out["k_idx"] = to_e4m3_bits(kk / k_scale[:, None])
            out["q_idx"] = to_e4m3_bits(q / q_scale[None, :, None])
        else:
            # bytes are e4m3(N(0,1)); scales drawn log-uniformly and applied on top
            k_scale = np.exp2(_rng(seed, cid, _T_KSCALE).uniform(-4.0, 4.0, size=S)).astype(np.float32)
            q_scale = np.exp2(_rng(seed, cid, _T_QSCALE).uniform(-2.0, 2.0, size=H)).astype(np.float32)
            out["k_idx"] = to_e4m3_bits(kk)
            out["q_idx"] = to_e4m3_bits(q)
        out["k_scale"] = k_scale
        out["q_scale"] = q_scale
        if q_pred is not None:
            out["q_pred"] = to_e4m3_bits(q_pred / q_scale[None, :, None]) if shape.structure == "clustered" else to_e4m3_bits(q_pred)
    del q, kk

    if shape.structure == "clustered":
        # recency term 2*exp(-(L+t-s)/4096) handed to the library as a rank-1 product
        out["recency"] = (2.0, 4096.0)
        t = np.arange(M, dtype=np.float64)
        s = np.arange(S, dtype=np.float64)
        out["row_bias"] = (2.0 * np.exp(-(L + t) / 4096.0)).astype(np.float32)
        out["col_bias"] = np.exp(s / 4096.0).astype(np.float32)
    else:
        out["recency"] = None
        out["row_bias"] = None
        out["col_bias"] = None

    if page_table is None:
        page_table = make_page_table(shape, seed)
        n_phys_pages = shape.n_logical_pages
    out["page_table"] = np.ascontiguousarray(page_table, dtype=np.int32)
    out["n_phys_pages"] = int(n_phys_pages)

    if with_attention:
        pg = shape.page_size
        if shape.attn == "latent":
            vs = 1.0 / 24.0
            out["Q"] = _normal_bf16(_rng(seed, cid, _T_Q), (M, shape.H_q, shape.d_qk), vs)
            if pool is None:
                kp = _normal_bf16(_rng(seed, cid, _T_POOL), (n_phys_pages, pg, 1, shape.d_qk), vs)
                pool = {"k_pool": kp, "v_pool": kp}
        else:
            vs = 1.0 / math.sqrt(shape.d_qk)
            out["Q"] = _normal_bf16(_rng(seed, cid, _T_Q), (M, shape.H_q, shape.d_qk), vs)
            if pool is None:
                pool = {
                    "k_pool": _normal_bf16(_rng(seed, cid, _T_POOL), (n_phys_pages, pg, shape.n_kv_heads, shape.d_qk), vs),
                    "v_pool": _normal_bf16(_rng(seed, cid, _T_VPOOL), (n_phys_pages, pg, shape.n_kv_heads, shape.d_v), vs),
                }
        out["k_pool"] = pool["k_pool"]
        out["v_pool"] = pool["v_pool"]
    return out


def make_batch(seed: int = 0, shapes: Optional[List[SessionShape]] = None, *, with_attention: bool = True):
    """Config 4: sessions sharing one fragmented physical pool."""
    shapes = shapes if shapes is not None else batch_shapes(seed)
    tables, n_phys = fragmented_page_tables(shapes, seed)
    pool = None
    if with_attention:
        s0 = shapes[0]
        kp = _normal_bf16(_rng(seed, 4, _T_POOL), (n_phys, s0.page_size, 1, s0.d_qk), 1.0 / 24.0)
        pool = {"k_pool": kp, "v_pool": kp}
    sessions = []
    for b, (shp, tab) in enumerate(zip(shapes, tables)):
        sessions.append(make_session(shp, seed * 1000 + b + 1, with_attention=with_attention,
                                     page_table=tab, n_phys_pages=n_phys, pool=pool))
    return sessions


def sample_rows(M: int, n: int) -> np.ndarray:
    """First, last and uniformly spread query rows (sorted, unique)."""
    if n >= M:
        return np.arange(M, dtype=np.int64)
    return np.unique(np.round(np.linspace(0, M - 1, n)).astype(np.int64))
