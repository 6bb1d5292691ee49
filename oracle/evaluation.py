"""fp64 CPU oracle of the evaluation path -- TEST INFRASTRUCTURE ONLY (same rules as ``ials.py``).

Paper passages followed (arXiv 2112.02194): Sec. 5, the evaluation protocol (the embedding of a held-out source row
comes from its kept links through Eq. 4 with the trained column table fixed; its nearest neighbours by inner product
are compared with its held-out links); Sec. 4.6 (Top-K: the best k items of a user); Table 2 (Recall@20, Recall@50).

Everything here is the plain definition: all scores, a full sort, set intersections.

Readings (the paper states none of these):
* order of equal scores: ascending id;
* Recall@K of a query = |first K retrieved ids that are ground truth| / |ground truth|; the reported number is the mean
  over the queries that have ground truth;
* whether the kept links may be retrieved: the caller's choice (``exclude``).
"""
from __future__ import annotations

import numpy as np

from . import ials


def fold_in(rowptr, colidx, values, H, alpha, lam, storage="f64"):
    """Eq. 4 for new rows against the fixed column table H: (stored, raw) solutions, one row per new row."""
    return ials.half_step(rowptr, colidx, values, H, alpha, lam, storage, return_raw=True)


def scores(Q, H):
    """All inner products <q, h_i>, fp64."""
    return np.asarray(Q, dtype=np.float64) @ np.asarray(H, dtype=np.float64).T


def topk(Q, H, k, exclude=None):
    """ids [m, k] (int64, -1 where fewer than k items qualify) and scores [m, k] (fp64, -inf there): every item scored,
    the row fully sorted by (score descending, id ascending)."""
    S = scores(Q, H)
    m, n = S.shape
    ids = np.full((m, k), -1, dtype=np.int64)
    sc = np.full((m, k), -np.inf)
    all_ids = np.arange(n)
    for q in range(m):
        keep = np.ones(n, dtype=bool)
        if exclude is not None:
            ptr, idx = exclude
            keep[np.asarray(idx[ptr[q]:ptr[q + 1]], dtype=np.int64)] = False
        cand = all_ids[keep]
        order = np.lexsort((cand, -S[q, cand]))      # last key first: score descending, then id ascending
        top = cand[order[:k]]
        ids[q, :top.size] = top
        sc[q, :top.size] = S[q, top]
    return ids, sc


def recall_at_k(ids, k, truth_ptr, truth_idx):
    """(mean over the queries with ground truth, number of those queries)"""
    total, counted = 0.0, 0
    for q in range(ids.shape[0]):
        truth = set(int(t) for t in truth_idx[truth_ptr[q]:truth_ptr[q + 1]])
        if not truth:
            continue
        hits = sum(1 for i in ids[q, :k] if int(i) in truth)
        total += hits / len(truth)
        counted += 1
    return (total / counted if counted else 0.0), counted
