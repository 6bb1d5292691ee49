"""ctypes front end of the fp64 CPU oracle (``ials_oracle.c``) -- TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the CPU-baseline leg of the benchmark may import this module.
It shares nothing with the CUDA library: its own C file, its own shared object.

Paper passages followed (arXiv 2112.02194): Eq. 3 (objective), Eq. 4 (row update),
Algorithm 1 (order of operations), Sec. 4.4 (bf16 tables, wider solve).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ials_oracle.c")
_LIB = os.path.join(_HERE, "libials_oracle.so")

F64, F32, BF16 = 0, 1, 2
STORAGE = {"f64": F64, "f32": F32, "bf16": BF16}

N_CLASSES = 12
SPLIT = 8192


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O3 without fast-math: IEEE arithmetic in source order; OpenMP over rows only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O3", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.alxo_round_storage.restype = ctypes.c_double
        _lib.alxo_round_storage.argtypes = [ctypes.c_double, ctypes.c_int]
        _lib.alxo_degree_class.restype = ctypes.c_int32
        _lib.alxo_degree_class.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int32]
        _lib.alxo_chunks.restype = ctypes.c_int64
        _lib.alxo_half_step_rows.restype = ctypes.c_int
        _lib.alxo_cg.restype = ctypes.c_int
        _lib.alxo_half_step_rows_cg.restype = ctypes.c_int
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def round_storage(x, storage: str):
    """Round an fp64 array to the values representable in the storage type (ties to even)."""
    out = _f64(x).copy()
    lib().alxo_round_array(_p(out), ctypes.c_int64(out.size), ctypes.c_int(STORAGE[storage]))
    return out


def gramian(X):
    X = _f64(X)
    N, d = X.shape
    G = np.empty((d, d), dtype=np.float64)
    lib().alxo_gramian(_p(X), ctypes.c_int64(N), ctypes.c_int(d), _p(G))
    return G


def gramian_stream(block_fn, N, d, block_rows=250_000):
    """Gramian of a table too large to hold in fp64: ``block_fn(row_begin, row_count)`` returns that block of
    rows as fp64 (already rounded to the storage type); blocks are added in order."""
    G = np.zeros((d, d), dtype=np.float64)
    for r0 in range(0, N, block_rows):
        G += gramian(block_fn(r0, min(block_rows, N - r0)))
    return G


def half_step(rowptr, colidx, values, X_fixed, alpha, lam, storage="f64", row_ids=None, G=None,
              return_raw=False, counters=None):
    """Eq. 4 for every row (or the rows in ``row_ids``) of the solved side.

    ``rowptr``/``colidx`` index the solved side's rows and point into ``X_fixed`` (N x d, fp64
    holding values already rounded to the storage type).  Returns the new rows rounded to
    ``storage`` (and the unrounded solution when ``return_raw``).
    """
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int64)
    colidx = np.ascontiguousarray(colidx, dtype=np.int32)
    vals = None if values is None else _f64(values)
    X = _f64(X_fixed)
    N, d = X.shape
    n = rowptr.size - 1
    if G is None:
        G = gramian(X)
    G = _f64(G)
    ids = None if row_ids is None else np.ascontiguousarray(row_ids, dtype=np.int64)
    count = n if ids is None else ids.size
    Y = np.empty((count, d), dtype=np.float64)
    Yraw = np.empty((count, d), dtype=np.float64) if return_raw else None
    cnt = np.zeros(3, dtype=np.int64) if counters is None else counters
    lib().alxo_half_step_rows(
        ctypes.c_int64(n), ctypes.c_int64(N), ctypes.c_int(d), _p(rowptr), _p(colidx), _p(vals), _p(X),
        _p(G), ctypes.c_double(alpha), ctypes.c_double(lam), ctypes.c_int(STORAGE[storage]), _p(ids),
        ctypes.c_int64(count), _p(Y), _p(Yraw), _p(cnt))
    if cnt[2]:
        raise FloatingPointError("oracle: normal matrix not positive definite")
    return (Y, Yraw) if return_raw else Y


def cg(A, b, tol=1e-5, max_iter=64, return_iterates=False):
    """Conjugate gradients on A x = b (Sec. 4.5; textbook form, x_0 = 0, stop at |r_k| <= tol |b| or max_iter)."""
    A, b = _f64(A), _f64(b)
    d = b.size
    x = np.empty(d)
    its = np.empty((max_iter, d)) if return_iterates else None
    work = np.empty(3 * d)
    k = lib().alxo_cg(ctypes.c_int(d), _p(A), _p(b), ctypes.c_double(tol), ctypes.c_int(max_iter), _p(x), _p(its),
                      _p(work))
    return (x, k, its[:k]) if return_iterates else (x, k)


def half_step_cg(rowptr, colidx, values, X_fixed, alpha, lam, storage="f64", row_ids=None, G=None, tol=1e-5,
                 max_iter=64):
    """Eq. 4 with the solve by conjugate gradients; returns (rows rounded to storage, unrounded, steps per row)."""
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int64)
    colidx = np.ascontiguousarray(colidx, dtype=np.int32)
    vals = None if values is None else _f64(values)
    X = _f64(X_fixed)
    N, d = X.shape
    n = rowptr.size - 1
    G = _f64(gramian(X) if G is None else G)
    ids = None if row_ids is None else np.ascontiguousarray(row_ids, dtype=np.int64)
    count = n if ids is None else ids.size
    Y = np.empty((count, d))
    Yraw = np.empty((count, d))
    iters = np.empty(count, dtype=np.int32)
    lib().alxo_half_step_rows_cg(
        ctypes.c_int64(n), ctypes.c_int64(N), ctypes.c_int(d), _p(rowptr), _p(colidx), _p(vals), _p(X), _p(G),
        ctypes.c_double(alpha), ctypes.c_double(lam), ctypes.c_int(STORAGE[storage]), _p(ids), ctypes.c_int64(count),
        ctypes.c_double(tol), ctypes.c_int(max_iter), _p(Y), _p(Yraw), _p(iters))
    return Y, Yraw, iters


def row_system(rowptr, colidx, values, X_fixed, G, alpha, lam, u):
    """A_u and b_u of Eq. 4 for one row, in fp64 (for residual checks)."""
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int64)
    colidx = np.ascontiguousarray(colidx, dtype=np.int32)
    vals = None if values is None else _f64(values)
    X = _f64(X_fixed)
    d = X.shape[1]
    A = np.empty((d, d))
    b = np.empty(d)
    lib().alxo_row_system(ctypes.c_int(d), ctypes.c_int64(int(rowptr[u])), ctypes.c_int64(int(rowptr[u + 1])),
                          _p(colidx), _p(vals), _p(X), _p(_f64(G)), ctypes.c_double(alpha),
                          ctypes.c_double(lam), _p(A), _p(b))
    return A, b


def loss(rowptr, colidx, values, W, H, alpha, lam, explicit=False):
    """Eq. 3; returns (total, (observed, all-pairs, regulariser)).

    ``explicit`` sums the all-pairs term over every (u, i); otherwise it goes through the Gramians.
    """
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int64)
    colidx = np.ascontiguousarray(colidx, dtype=np.int32)
    vals = None if values is None else _f64(values)
    W, H = _f64(W), _f64(H)
    comp = np.empty(3)
    fn = lib().alxo_loss if explicit else lib().alxo_loss_gramian
    fn(ctypes.c_int64(W.shape[0]), ctypes.c_int64(H.shape[0]), ctypes.c_int(W.shape[1]), _p(rowptr), _p(colidx),
       _p(vals), _p(W), _p(H), ctypes.c_double(alpha), ctypes.c_double(lam), _p(comp))
    return float(comp.sum()), tuple(float(c) for c in comp)


def transpose(n_rows, n_cols, rowptr, colidx, values=None):
    """CSR -> CSC with row ids ascending inside each column (stable counting sort)."""
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int64)
    colidx = np.ascontiguousarray(colidx, dtype=np.int32)
    nnz = int(rowptr[-1])
    colptr = np.empty(n_cols + 1, dtype=np.int64)
    rowidx = np.empty(nnz, dtype=np.int32)
    v = None if values is None else np.ascontiguousarray(values, dtype=np.float32)
    vt = None if values is None else np.empty(nnz, dtype=np.float32)
    lib().alxo_transpose(ctypes.c_int64(n_rows), ctypes.c_int64(n_cols), _p(rowptr), _p(colidx), _p(v),
                         _p(colptr), _p(rowidx), _p(vt))
    return colptr, rowidx, vt


def degree_class(deg, split=SPLIT, n_classes=N_CLASSES):
    return int(lib().alxo_degree_class(int(deg), int(split), int(n_classes)))


def bucket_rows(rowptr, split=SPLIT, n_classes=N_CLASSES):
    """Rows ordered by (degree class, id) and the class offsets into that order."""
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int64)
    n = rowptr.size - 1
    order = np.empty(n, dtype=np.int32)
    offs = np.empty(n_classes + 1, dtype=np.int64)
    lib().alxo_bucket_rows(ctypes.c_int64(n), _p(rowptr), ctypes.c_int64(split), ctypes.c_int32(n_classes),
                           _p(order), _p(offs))
    return order, offs


def chunks(rowptr, split=SPLIT, n_classes=N_CLASSES):
    """Chunk descriptors (row, begin, end, slot) of the rows longer than ``split`` and, per such row, its first slot."""
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int64)
    n = rowptr.size - 1
    args = (ctypes.c_int64(n), _p(rowptr), ctypes.c_int64(split), ctypes.c_int32(n_classes))
    n_chunks = lib().alxo_chunks(*args, None, None)
    deg = np.diff(rowptr)
    n_split_rows = int((deg > split).sum())
    desc = np.empty((n_chunks, 4), dtype=np.int64)
    first = np.empty(n_split_rows + 1, dtype=np.int64)
    lib().alxo_chunks(*args, _p(desc), _p(first))
    return desc, first


def epoch(rowptr, colidx, values, W, H, alpha, lam, storage="f64"):
    """One epoch in Alg. 1's order: rows with H fixed, then columns with the new W fixed."""
    n_rows, n_cols = W.shape[0], H.shape[0]
    W1 = half_step(rowptr, colidx, values, H, alpha, lam, storage)
    colptr, rowidx, vt = transpose(n_rows, n_cols, rowptr, colidx, values)
    H1 = half_step(colptr, rowidx, vt, W1, alpha, lam, storage)
    return W1, H1
