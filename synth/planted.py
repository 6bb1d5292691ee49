"""Seeded planted-structure link matrix and the evaluation split of the paper's Sec. 5 (stand-in for the WebGraph
train/test files, which are not available offline).  Holds none of the method's arithmetic.

Recipe: `n_groups` groups; every row belongs to one group (row id mod n_groups), every group owns a pool of `pool`
columns (disjoint, consecutive ids, shuffled by a seeded permutation of the columns).  A row of degree k draws
round(p_in k) distinct columns from its group's pool and the rest uniformly from all columns, so the matrix is a noisy
block matrix of rank about n_groups.  Degrees are uniform in [deg_lo, deg_hi].

Split ("strong generalisation"): a seeded 10 % of the rows are test rows and are taken out of the training matrix;
of every test row's links a seeded 25 % (at least one) are held out as ground truth, the rest are what the row's
embedding is computed from.
"""
from __future__ import annotations

import numpy as np


def planted_links(n_rows, n_cols, n_groups, pool, deg_lo, deg_hi, p_in, seed):
    """CSR (rowptr int64, colidx int32, ascending and distinct inside a row)."""
    assert n_groups * pool <= n_cols and deg_hi <= pool
    rng = np.random.Generator(np.random.PCG64(seed))
    perm = rng.permutation(n_cols)
    deg = rng.integers(deg_lo, deg_hi + 1, n_rows)
    rowptr = np.zeros(n_rows + 1, dtype=np.int64)
    cols = []
    for u in range(n_rows):
        g = u % n_groups
        k = int(deg[u])
        k_in = int(round(p_in * k))
        own = perm[g * pool + rng.choice(pool, size=k_in, replace=False)]
        rest = rng.choice(n_cols, size=k - k_in, replace=False)
        c = np.unique(np.concatenate([own, rest]))
        cols.append(c.astype(np.int32))
        rowptr[u + 1] = rowptr[u] + c.size
    return rowptr, np.concatenate(cols)


def split_rows(rowptr, colidx, test_fraction, holdout_fraction, seed):
    """Returns dict(train=(rowptr, colidx), test_rows, kept=(rowptr, colidx), truth=(rowptr, colidx)): the training matrix
    keeps every row id (test rows become empty rows), the two test CSRs have one row per test row, in test_rows order."""
    n = rowptr.size - 1
    rng = np.random.Generator(np.random.PCG64(seed))
    is_test = np.zeros(n, dtype=bool)
    is_test[rng.choice(n, size=max(1, int(round(test_fraction * n))), replace=False)] = True
    test_rows = np.nonzero(is_test)[0]
    tr_ptr = np.zeros(n + 1, dtype=np.int64)
    tr_cols = []
    for u in range(n):
        if not is_test[u]:
            tr_cols.append(colidx[rowptr[u]:rowptr[u + 1]])
        tr_ptr[u + 1] = tr_ptr[u] + (0 if is_test[u] else rowptr[u + 1] - rowptr[u])
    kp, kc, tp, tc = [0], [], [0], []
    for u in test_rows:
        c = colidx[rowptr[u]:rowptr[u + 1]]
        n_hold = min(c.size, max(1, int(round(holdout_fraction * c.size)))) if c.size else 0
        held = np.zeros(c.size, dtype=bool)
        if n_hold:
            held[rng.choice(c.size, size=n_hold, replace=False)] = True
        kc.append(c[~held]); kp.append(kp[-1] + int((~held).sum()))
        tc.append(c[held]); tp.append(tp[-1] + int(held.sum()))
    cat = lambda parts: np.concatenate(parts).astype(np.int32) if parts else np.zeros(0, dtype=np.int32)
    return dict(train=(tr_ptr, cat(tr_cols)), test_rows=test_rows,
                kept=(np.asarray(kp, dtype=np.int64), cat(kc)), truth=(np.asarray(tp, dtype=np.int64), cat(tc)))
