"""Reporting metrics of the page-demand step, computed from the library's device outputs (Sec. 4.2: recall and precision of
the predicted union against the exact one; Sec. 4.3: how the demand coalesces into runs).

Nothing here is on the timed path: the functions read the counts, bitmaps and run lists the kernels wrote and turn them
into the figures the benchmark prints.  Set sizes come from the kernels' own outputs:
|exact ∩ predicted| = |exact| - |miss|, because the miss set is exact minus predicted.
"""
from __future__ import annotations

from typing import Dict, Optional

import torch

from . import binding as B

_POP8 = None


def popcount(bitmap: torch.Tensor) -> int:
    """Number of set bits of a page bitmap (int32 words, as janus_page_demand writes it)."""
    global _POP8
    if _POP8 is None or _POP8.device != bitmap.device:
        _POP8 = torch.tensor([bin(i).count("1") for i in range(256)], dtype=torch.int64, device=bitmap.device)
    return int(_POP8[bitmap.contiguous().view(torch.uint8).long()].sum().item())


def run_length_histogram(pd: Dict[str, torch.Tensor], which: str = "runs", count_index: int = 1) -> Dict[int, int]:
    """{run length: number of runs} of a run list written by janus_page_demand ('runs' or 'miss_runs')."""
    n = int(pd["counts"][count_index].item())
    if n == 0:
        return {}
    lens = pd[which][:n, 1].long()
    vals, cnts = torch.unique(lens, return_counts=True)
    return {int(v): int(c) for v, c in zip(vals.tolist(), cnts.tolist())}


def demand_report(pd: Dict[str, torch.Tensor], predicted_bitmap: Optional[torch.Tensor]) -> Dict[str, object]:
    """Recall, precision, miss-set size and run statistics of one janus_page_demand result against the predicted set it was
    given.  Without a predicted set everything is a miss: recall 0, precision reported as None."""
    n_pages, n_runs, n_miss, n_miss_runs = (int(x) for x in pd["counts"].tolist())
    rep: Dict[str, object] = {"n_demand": n_pages, "n_runs": n_runs, "mean_run_length": (n_pages / n_runs) if n_runs else 0.0,
                              "n_miss": n_miss, "n_miss_runs": n_miss_runs}
    if predicted_bitmap is None:
        rep.update({"n_predicted": 0, "recall": 0.0 if n_pages else 1.0, "precision": None})
        return rep
    n_pred = popcount(predicted_bitmap)
    inter = n_pages - n_miss
    rep.update({"n_predicted": n_pred, "recall": inter / n_pages if n_pages else 1.0, "precision": inter / n_pred if n_pred else 1.0})
    return rep


def token_granularity_report(idx: torch.Tensor, pred_idx: Optional[torch.Tensor], L: int) -> Dict[str, object]:
    """The same report at token granularity: page size 1 and an identity table over the L history tokens, so the 'pages' are
    the selected history tokens themselves (the union of selections of Sec. 2.2) and the runs are runs of adjacent tokens."""
    ident = torch.arange(L, dtype=torch.int32, device=idx.device)
    pred_bitmap = None
    if pred_idx is not None:
        pred_bitmap = B.janus_page_demand(pred_idx, demand_limit=L, page_size=1, page_table=ident, n_phys_pages=L, want_miss=False)["bitmap"]
    pd = B.janus_page_demand(idx, demand_limit=L, page_size=1, page_table=ident, n_phys_pages=L, predicted_bitmap=pred_bitmap)
    return demand_report(pd, pred_bitmap)
