"""Lookahead prediction passes built from the library calls (argument plumbing only; all arithmetic runs in the kernels).

predicted_pages          Eq. 2: the layer's own indexer on lookahead queries over the history keys -> top-k -> page set.
sharded_predicted_pages  Eq. 3 (synchronisation-free parallel prediction): the history is cut into N disjoint, page-aligned
                         shards; each shard selects its own top-(k/N) and builds its own page set (on N GPUs these run
                         independently and each GPU prefetches its own pages; here the shards run one after another on one
                         GPU); the per-shard sets are united when the exact pass needs them.
"""
from __future__ import annotations

from typing import List, Optional, Tuple

import torch

from . import binding as B


def predicted_pages(q_pred, k_idx, w, *, L: int, k: int, page_size: int, page_table, n_phys_pages: int,
                    q_scale=None, k_scale=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Returns (bitmap of predicted physical pages, predicted indices [M,k])."""
    sc = B.janus_indexer_scores(q_pred, k_idx[:L], w, q_scale=q_scale, k_scale=None if k_scale is None else k_scale[:L],
                                q_pos0=L, causal=False)
    idx, _, _ = B.janus_topk(sc, L, k, q_pos0=L, causal=False, want_count=False, want_kth=False)
    pd = B.janus_page_demand(idx, demand_limit=L, page_size=page_size, page_table=page_table, n_phys_pages=n_phys_pages, want_miss=False)
    return pd["bitmap"], idx


def shard_bounds(L: int, n_shards: int, page_size: int) -> List[Tuple[int, int]]:
    """Disjoint, page-aligned [begin, end) token ranges covering [0, L)."""
    n_pages = (L + page_size - 1) // page_size
    out = []
    for n in range(n_shards):
        a = (n * n_pages // n_shards) * page_size
        b = min(L, ((n + 1) * n_pages // n_shards) * page_size)
        if b > a:
            out.append((a, b))
    return out


def sharded_predicted_pages(q_pred, k_idx, w, *, L: int, k: int, n_shards: int, page_size: int, page_table, n_phys_pages: int,
                            q_scale=None, k_scale=None):
    """Returns (union bitmap, list of per-shard bitmaps, list of per-shard local indices [M, k/N])."""
    k_shard = max(1, k // n_shards)
    union: Optional[torch.Tensor] = None
    bitmaps, indices = [], []
    for a, b in shard_bounds(L, n_shards, page_size):
        sc = B.janus_indexer_scores(q_pred, k_idx[a:b], w, q_scale=q_scale, k_scale=None if k_scale is None else k_scale[a:b],
                                    q_pos0=L, causal=False)
        idx, _, _ = B.janus_topk(sc, b - a, k_shard, q_pos0=L, causal=False, want_count=False, want_kth=False)
        # indices are local to the shard; the shard starts on a page boundary, so its pages are a slice of the page table
        pd = B.janus_page_demand(idx, demand_limit=b - a, page_size=page_size, page_table=page_table[a // page_size:],
                                 n_phys_pages=n_phys_pages, want_miss=False)
        bitmaps.append(pd["bitmap"])
        indices.append(idx)
        union = pd["bitmap"].clone() if union is None else B.janus_page_union(union, pd["bitmap"], n_phys_pages)
    return union, bitmaps, indices
