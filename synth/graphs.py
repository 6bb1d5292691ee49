"""Seeded synthetic inputs: sparse observation matrices and initial embedding tables.

This module serves both the CPU oracle and the CUDA library and holds none of the method's
arithmetic.  Everything that depends on the seed is integer hashing, so the numpy code here and
the CUDA twin in ``synth/csrc/synth.cu`` give identical bits, and any single row can be
regenerated alone (used to check sampled rows of graphs that only ever exist on the device).

Recipe (stand-in for the paper's WebGraph link matrices, Table 1: square node x node, long-tailed
degrees; the real data set is not available offline):

* degrees: rank-size Zipf, deg(rank r) = clamp(round(C r^-s), 1, cap), C bisected so that the sum
  is the nominal number of edges; rank -> row id by an affine bijection (a r + b) mod n.
  Computed once on the host in fp64 and passed around as an int32 table.
* columns of a row with k entries are k strata of a column domain, one draw per stratum, hence
  strictly ascending and distinct by construction (realised nnz == nominal nnz):
    - law "quantile": stratum j = [j + floor((N-k) g(j/k)), (j+1) + floor((N-k) g((j+1)/k))),
      g a monotone map of [0,1] stored as a 2^16+1 entry fixed-point table (uniform: g(x) = x;
      Zipf popularity with a cap on the in-degree: g = inverse CDF, column 0 the most popular);
    - law "local": round(0.8 k) entries from a window of +-delta ids around the row's own id
      (shifted to stay inside [0, N)), the rest from the ids outside the window, both uniform strata.
* embeddings: i.i.d. normal with standard deviation sigma via an inverse-CDF table (2^12 cells,
  integer interpolation, tails end at about 3.7 sigma), rounded to the storage type.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from math import gcd

import numpy as np

U64 = np.uint64
_M1 = U64(0xBF58476D1CE4E5B9)
_M2 = U64(0x94D049BB133111EB)
_GOLD = U64(0x9E3779B97F4A7C15)

LAW_QUANTILE = 0
LAW_LOCAL = 1
QT_BITS = 16           # quantile table has 2^16 cells
NT_BITS = 12           # normal table has 2^12 cells
NT_FRAC_BITS = 20
NT_SCALE_BITS = 24     # table values are Phi^-1 * 2^24


def mix64(z):
    """splitmix64 finaliser on uint64 arrays (wraps modulo 2^64)."""
    z = np.asarray(z, dtype=U64)
    with np.errstate(over="ignore"):
        z = (z ^ (z >> U64(30))) * _M1
        z = (z ^ (z >> U64(27))) * _M2
        return z ^ (z >> U64(31))


def hash2(key, a, b):
    """hash of (key, a, b): mix64(mix64(key ^ a) + b * GOLD)."""
    with np.errstate(over="ignore"):
        return mix64(mix64(np.asarray(key, dtype=U64) ^ np.asarray(a, dtype=U64))
                     + np.asarray(b, dtype=U64) * _GOLD)


def stream_key(seed: int, stream: int) -> np.uint64:
    with np.errstate(over="ignore"):
        return mix64(np.array([seed], dtype=U64) + _GOLD * U64(stream + 1))[0]


# ----------------------------------------------------------------------------- degrees

def zipf_degrees(n: int, nnz: int, s: float, cap: int, seed: int) -> np.ndarray:
    """int32[n] degrees following a rank-size law, summing exactly to nnz, scattered over row ids."""
    r = np.arange(1, n + 1, dtype=np.float64)
    base = r ** (-s)

    def total(C):
        return np.clip(np.rint(C * base), 1, cap).sum()

    lo, hi = 0.0, float(cap) * 4
    while total(hi) < nnz:
        hi *= 2
    for _ in range(64):
        mid = 0.5 * (lo + hi)
        if total(mid) < nnz:
            lo = mid
        else:
            hi = mid
    deg = np.clip(np.rint(hi * base), 1, cap).astype(np.int64)
    # trim the rounding surplus from the middle of the ranking so that the sum is exact
    surplus = int(deg.sum() - nnz)
    if surplus > 0:
        idx = np.nonzero((deg > 1) & (deg < cap))[0]
        if idx.size < surplus:
            idx = np.nonzero(deg > 1)[0]
        take = idx[:surplus]
        deg[take] -= 1
    elif surplus < 0:
        idx = np.nonzero(deg < cap)[0][: -surplus]
        deg[idx] += 1
    assert int(deg.sum()) == nnz
    a, b = affine_bijection(n, seed)
    rows = (np.arange(n, dtype=np.int64) * a + b) % n
    out = np.empty(n, dtype=np.int32)
    out[rows] = deg.astype(np.int32)
    return out


def affine_bijection(n: int, seed: int):
    """(a, b) with gcd(a, n) = 1: r -> (a r + b) mod n permutes [0, n)."""
    h = int(mix64(np.array([seed], dtype=U64))[0])
    a = int(n * 0.6180339887) | 1
    while gcd(a, n) != 1:
        a += 2
    a %= n
    if a == 0:
        a = 1
    assert a * n < 2 ** 63
    return a, h % n


# ----------------------------------------------------------------------------- column laws

def uniform_quantile_table() -> np.ndarray:
    T = 1 << QT_BITS
    return (np.arange(T + 1, dtype=np.uint64) << np.uint64(32 - QT_BITS)).astype(np.uint64)


def zipf_quantile_table(n_cols: int, s: float, max_share: float) -> np.ndarray:
    """Fixed-point (2^32 = 1.0) inverse CDF of a popularity law p(c) ~ min((c+1)^-s, level) over columns.

    ``max_share`` bounds the probability of the most popular column (cap on in-degree / nnz).
    """
    c = np.arange(1, n_cols + 1, dtype=np.float64)
    w = c ** (-s)
    # find the clipping level so that the largest normalised weight is max_share
    lo, hi = 0.0, 1.0
    for _ in range(100):
        mid = 0.5 * (lo + hi)
        wc = np.minimum(w, mid)
        if wc[0] / wc.sum() > max_share:
            hi = mid
        else:
            lo = mid
    wc = np.minimum(w, lo if lo > 0 else hi)
    cdf = np.cumsum(wc)
    cdf /= cdf[-1]
    T = 1 << QT_BITS
    q = np.searchsorted(cdf, np.arange(T + 1, dtype=np.float64) / T, side="left").astype(np.float64)
    q = np.minimum(q, n_cols) / n_cols
    q[0], q[-1] = 0.0, 1.0
    q = np.maximum.accumulate(q)
    return np.minimum(np.floor(q * 2.0 ** 32), 2.0 ** 32).astype(np.uint64)


@dataclass
class GraphSpec:
    """Everything the edge generator needs besides the degree table; integers only."""
    n_rows: int
    n_cols: int
    seed: int
    law: int = LAW_QUANTILE
    qtable: np.ndarray = field(default_factory=uniform_quantile_table)  # uint64[2^16 + 1]
    delta: int = 0          # law "local": half window
    local_num: int = 4      # law "local": local share = local_num / local_den
    local_den: int = 5


def _g_fixed(qtable, j, k):
    """g(j / k) in 2^32 fixed point by integer interpolation of the quantile table."""
    j = j.astype(U64)
    k = k.astype(U64)
    pos = (j << U64(32)) // k                       # in [0, 2^32]
    idx = pos >> U64(32 - QT_BITS)
    frac = pos & U64((1 << (32 - QT_BITS)) - 1)
    idx = np.minimum(idx, U64((1 << QT_BITS)))
    nxt = np.minimum(idx + U64(1), U64(1 << QT_BITS))
    q0 = qtable[idx.astype(np.int64)]
    q1 = qtable[nxt.astype(np.int64)]
    return q0 + (((q1 - q0) * frac) >> U64(32 - QT_BITS))


def _quantile_bound(spec, j, k):
    """B_j = j + floor((N - k) g(j/k))."""
    N = U64(spec.n_cols)
    g = _g_fixed(spec.qtable, j, k)
    return j.astype(U64) + (((N - k.astype(U64)) * g) >> U64(32))


def _uniform_bound(j, k, M):
    """floor(j M / k) as uint64 arrays."""
    return (j.astype(U64) * M.astype(U64)) // np.maximum(k.astype(U64), U64(1))


def row_columns_flat(spec: GraphSpec, rows: np.ndarray, deg: np.ndarray):
    """Columns of the given rows, concatenated.  rows: int64[m]; deg: int32/int64[m] (their degrees).

    Returns (ptr int64[m+1], cols int32[sum deg]).
    """
    rows = np.asarray(rows, dtype=np.int64)
    deg = np.asarray(deg, dtype=np.int64)
    ptr = np.zeros(rows.size + 1, dtype=np.int64)
    np.cumsum(deg, out=ptr[1:])
    total = int(ptr[-1])
    if total == 0:
        return ptr, np.empty(0, dtype=np.int32)
    rid = np.repeat(np.arange(rows.size, dtype=np.int64), deg)
    u = rows[rid].astype(U64)
    k = deg[rid].astype(U64)
    j = (np.arange(total, dtype=np.int64) - ptr[rid]).astype(U64)
    key = stream_key(spec.seed, 1)
    if spec.law == LAW_QUANTILE:
        lo = _quantile_bound(spec, j, k)
        hi = _quantile_bound(spec, j + U64(1), k)
        cols = lo + hash2(key, u, j) % (hi - lo)
        return ptr, cols.astype(np.int32)
    # law "local"
    N = spec.n_cols
    wsz = 2 * spec.delta + 1
    assert wsz < N
    ku = deg.astype(np.int64)
    kloc_r = np.minimum((ku * spec.local_num + spec.local_den // 2) // spec.local_den, wsz)
    kfar_r = ku - kloc_r
    M = N - wsz
    assert int(kfar_r.max(initial=0)) <= M
    wlo_r = np.clip(rows - spec.delta, 0, N - wsz)
    # number of far draws that land below the window
    jj = np.minimum(kfar_r, ((wlo_r + 1) * kfar_r - 1) // M) + 1      # strata starting at or below wlo
    js = jj - 1                                                        # the stratum that may straddle wlo
    has = (kfar_r > 0) & (js < kfar_r)
    jsU, kfU = js.astype(U64), np.maximum(kfar_r, 1).astype(U64)
    MU = np.full(rows.size, M, dtype=U64)
    f0 = _uniform_bound(jsU, kfU, MU)
    f1 = _uniform_bound(jsU + U64(1), kfU, MU)
    ts = f0 + hash2(key, rows.astype(U64), jsU + U64(1 << 40)) % np.maximum(f1 - f0, U64(1))
    cbelow_r = np.where(kfar_r > 0, js + (has & (ts.astype(np.int64) < wlo_r)), 0)
    cbelow = cbelow_r[rid].astype(U64)
    kloc = kloc_r[rid].astype(U64)
    kfar = kfar_r[rid].astype(U64)
    wlo = wlo_r[rid].astype(U64)
    is_loc = (j >= cbelow) & (j < cbelow + kloc)
    # local draws
    jl = np.where(is_loc, j - cbelow, U64(0))
    W = np.full(total, wsz, dtype=U64)
    l0 = _uniform_bound(jl, np.maximum(kloc, U64(1)), W)
    l1 = _uniform_bound(jl + U64(1), np.maximum(kloc, U64(1)), W)
    loc = wlo + l0 + hash2(key, u, jl) % np.maximum(l1 - l0, U64(1))
    # far draws
    jf = np.where(is_loc, U64(0), np.where(j < cbelow, j, j - kloc))
    MM = np.full(total, M, dtype=U64)
    g0 = _uniform_bound(jf, np.maximum(kfar, U64(1)), MM)
    g1 = _uniform_bound(jf + U64(1), np.maximum(kfar, U64(1)), MM)
    t = g0 + hash2(key, u, jf + U64(1 << 40)) % np.maximum(g1 - g0, U64(1))
    far = np.where(t < wlo, t, t + U64(wsz))
    cols = np.where(is_loc, loc, far)
    return ptr, cols.astype(np.int32)


def build_csr(spec: GraphSpec, deg: np.ndarray, rows_per_block: int = 1 << 16):
    """Whole graph on the host: (rowptr int64[n+1], colidx int32[nnz])."""
    n = spec.n_rows
    rowptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(deg.astype(np.int64), out=rowptr[1:])
    colidx = np.empty(int(rowptr[-1]), dtype=np.int32)
    for r0 in range(0, n, rows_per_block):
        r1 = min(n, r0 + rows_per_block)
        _, cols = row_columns_flat(spec, np.arange(r0, r1, dtype=np.int64), deg[r0:r1])
        colidx[rowptr[r0]:rowptr[r1]] = cols
    return rowptr, colidx


def uniform_cells_csr(n_rows: int, n_cols: int, nnz: int, seed: int):
    """Exactly nnz distinct cells chosen uniformly at random (small matrices only)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    cells = np.sort(rng.choice(n_rows * n_cols, size=nnz, replace=False))
    r = cells // n_cols
    rowptr = np.zeros(n_rows + 1, dtype=np.int64)
    np.cumsum(np.bincount(r, minlength=n_rows), out=rowptr[1:])
    return rowptr, (cells % n_cols).astype(np.int32)


# ----------------------------------------------------------------------------- embeddings

def normal_table() -> np.ndarray:
    """int64[2^12 + 1]: Phi^-1 at the cell edges of (0, 1), times 2^24; ends clipped to finite values."""
    from scipy.special import ndtri
    T = 1 << NT_BITS
    p = np.arange(T + 1, dtype=np.float64) / T
    p[0], p[-1] = 0.5 / T / 16, 1 - 0.5 / T / 16
    return np.rint(ndtri(p) * 2.0 ** NT_SCALE_BITS).astype(np.int64)


def normal_fixed(seed: int, stream: int, start: int, count: int, table: np.ndarray, index=None) -> np.ndarray:
    """int64[count]: standard normal draws times 2^24 for element indices start .. start+count-1
    (or for the explicit element indices in ``index``)."""
    key = stream_key(seed, stream)
    if index is None:
        idx = np.arange(start, start + count, dtype=np.int64).astype(U64)
    else:
        idx = np.asarray(index, dtype=np.int64).astype(U64)
    h = hash2(key, idx, U64(0))
    cell = (h >> U64(64 - NT_BITS)).astype(np.int64)
    frac = ((h >> U64(64 - NT_BITS - NT_FRAC_BITS)) & U64((1 << NT_FRAC_BITS) - 1)).astype(np.int64)
    t0 = table[cell]
    t1 = table[cell + 1]
    return t0 + (((t1 - t0) * frac) >> NT_FRAC_BITS)


def to_storage_bits(x64: np.ndarray, storage: str) -> np.ndarray:
    """fp64 -> storage type, round to nearest even: float32 array, or uint16 array of bf16 bit patterns."""
    f = x64.astype(np.float32)
    if storage == "f32":
        return f
    b = f.view(np.uint32)
    rounded = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def storage_to_f64(a: np.ndarray, storage: str) -> np.ndarray:
    if storage == "f32":
        return a.astype(np.float64)
    return (a.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def init_embeddings(n: int, d: int, seed: int, stream: int, storage: str, row_begin: int = 0,
                    row_count: int | None = None, sigma: float | None = None) -> np.ndarray:
    """Rows row_begin .. of an n x d table of N(0, sigma^2) draws in the storage type's bit layout.

    sigma defaults to 0.1 / sqrt(d).  Returns float32[rows, d] or uint16[rows, d] (bf16 bits).
    """
    if row_count is None:
        row_count = n - row_begin
    if sigma is None:
        sigma = 0.1 / np.sqrt(d)
    v = normal_fixed(seed, stream, row_begin * d, row_count * d, normal_table())
    x = v.astype(np.float64) * (sigma / 2.0 ** NT_SCALE_BITS)
    return to_storage_bits(x, storage).reshape(row_count, d)


def init_embedding_rows(row_ids, d: int, seed: int, stream: int, storage: str, sigma: float | None = None):
    """The listed rows of the table init_embeddings(n, d, seed, stream, storage) would give, without the rest."""
    row_ids = np.asarray(row_ids, dtype=np.int64)
    if sigma is None:
        sigma = 0.1 / np.sqrt(d)
    index = (row_ids[:, None] * d + np.arange(d, dtype=np.int64)[None, :]).reshape(-1)
    v = normal_fixed(seed, stream, 0, 0, normal_table(), index=index)
    x = v.astype(np.float64) * (sigma / 2.0 ** NT_SCALE_BITS)
    return to_storage_bits(x, storage).reshape(row_ids.size, d)
