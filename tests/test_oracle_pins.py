"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU, no CUDA code).

Each test is chosen so that a plausible slip in the oracle (dropped all-pairs term, regulariser on the
wrong place, transposed index, wrong sign) fails at least one of them.
"""
import json
import os

import numpy as np
import pytest

from oracle import ials

HERE = os.path.dirname(os.path.abspath(__file__))


def random_problem(n_rows, n_cols, d, density, seed, binary=False):
    rng = np.random.default_rng(seed)
    mask = rng.random((n_rows, n_cols)) < density
    mask[0, :] = False                                    # one empty row
    if n_rows > 2:
        mask[1, :] = True                                 # one fully observed row
    rowptr = np.zeros(n_rows + 1, dtype=np.int64)
    rowptr[1:] = np.cumsum(mask.sum(1))
    colidx = np.nonzero(mask)[1].astype(np.int32)
    vals = np.ones(colidx.size) if binary else rng.normal(1.0, 0.7, colidx.size)
    W = rng.normal(0, 0.5, (n_rows, d))
    H = rng.normal(0, 0.5, (n_cols, d))
    return rowptr, colidx, vals, W, H, mask


def dense_Y(rowptr, colidx, vals, n_rows, n_cols):
    Y = np.zeros((n_rows, n_cols))
    for u in range(n_rows):
        for e in range(rowptr[u], rowptr[u + 1]):
            Y[u, colidx[e]] = vals[e]
    return Y


# ---- hand-derived golden values ------------------------------------------------------------

def test_hand_examples():
    with open(os.path.join(HERE, "golden", "hand_examples.json")) as f:
        cases = json.load(f)["cases"]
    for c in cases:
        H = np.array(c["H"])
        rowptr = np.array([0, len(c["obs_cols"])], dtype=np.int64)
        colidx = np.array(c["obs_cols"], dtype=np.int32)
        y = np.array(c["obs_y"])
        w = ials.half_step(rowptr, colidx, y, H, c["alpha"], c["lambda"])
        expect = np.array(c["w_num"], dtype=np.float64) / c["w_den"]
        np.testing.assert_allclose(w[0], expect, rtol=1e-14, atol=0)
        if "loss_num" in c:
            for explicit in (True, False):
                tot, comp = ials.loss(rowptr, colidx, y, w, H, c["alpha"], c["lambda"], explicit=explicit)
                np.testing.assert_allclose(tot, c["loss_num"] / c["loss_den"], rtol=1e-14)
                np.testing.assert_allclose(
                    comp, np.array(c["loss_components_num"]) / c["loss_components_den"], rtol=1e-13)


# ---- brute force: stacked weighted least squares by QR, no normal equations ------------------

@pytest.mark.parametrize("shape", [(8, 6, 3, 0.5, 1), (30, 20, 4, 0.3, 2), (12, 40, 7, 0.2, 3)])
def test_half_step_matches_stacked_least_squares(shape):
    n_rows, n_cols, d, dens, seed = shape
    rowptr, colidx, vals, W, H, mask = random_problem(n_rows, n_cols, d, dens, seed)
    alpha, lam = 0.3, 0.2
    got = ials.half_step(rowptr, colidx, vals, H, alpha, lam)
    for u in range(n_rows):
        cols = colidx[rowptr[u]:rowptr[u + 1]]
        # minimise |H_obs w - y|^2 + alpha |H_all w|^2 + lam |w|^2 as one least-squares problem
        M = np.vstack([H[cols], np.sqrt(alpha) * H, np.sqrt(lam) * np.eye(d)])
        t = np.concatenate([vals[rowptr[u]:rowptr[u + 1]], np.zeros(n_cols), np.zeros(d)])
        ref = np.linalg.lstsq(M, t, rcond=None)[0]
        np.testing.assert_allclose(got[u], ref, rtol=1e-10, atol=1e-12)
    assert np.all(got[0] == 0.0)          # empty row -> exactly zero


def test_column_half_step_is_the_same_update_on_the_transpose():
    rowptr, colidx, vals, W, H, mask = random_problem(9, 7, 3, 0.5, 4)
    vals = vals.astype(np.float32).astype(np.float64)     # the transpose carries labels as fp32
    alpha, lam = 0.1, 0.4
    colptr, rowidx, vt = ials.transpose(9, 7, rowptr, colidx, vals)
    got = ials.half_step(colptr, rowidx, vt, W, alpha, lam)
    Y = dense_Y(rowptr, colidx, vals, 9, 7)
    for i in range(7):
        rows = np.nonzero(mask[:, i])[0]
        M = np.vstack([W[rows], np.sqrt(alpha) * W, np.sqrt(lam) * np.eye(3)])
        t = np.concatenate([Y[rows, i], np.zeros(9), np.zeros(3)])
        ref = np.linalg.lstsq(M, t, rcond=None)[0]
        np.testing.assert_allclose(got[i], ref, rtol=1e-10, atol=1e-12)


# ---- closed forms ----------------------------------------------------------------------------

def test_closed_form_d1():
    rng = np.random.default_rng(5)
    H = rng.normal(size=(11, 1))
    cols = np.array([1, 4, 5, 9], dtype=np.int32)
    y = rng.normal(size=4)
    alpha, lam = 0.37, 0.21
    w = ials.half_step(np.array([0, 4]), cols, y, H, alpha, lam)[0, 0]
    h = H[:, 0]
    expect = (h[cols] * y).sum() / ((h[cols] ** 2).sum() + alpha * (h ** 2).sum() + lam)
    np.testing.assert_allclose(w, expect, rtol=1e-13)


def test_closed_form_single_observation():
    rng = np.random.default_rng(6)
    d = 5
    H = rng.normal(size=(9, d))
    y, lam = 1.7, 0.3
    h = H[3]
    # alpha = 0: Sherman-Morrison on (h h^T + lam I)
    w = ials.half_step(np.array([0, 1]), np.array([3], dtype=np.int32), np.array([y]), H, 0.0, lam)[0]
    np.testing.assert_allclose(w, h * y / (h @ h + lam), rtol=1e-12)
    # alpha > 0: B = alpha G + lam I, w = B^-1 h y / (1 + h^T B^-1 h)
    alpha = 0.25
    B = alpha * H.T @ H + lam * np.eye(d)
    Bih = np.linalg.solve(B, h)
    w = ials.half_step(np.array([0, 1]), np.array([3], dtype=np.int32), np.array([y]), H, alpha, lam)[0]
    np.testing.assert_allclose(w, Bih * y / (1 + h @ Bih), rtol=1e-12)


def test_closed_form_orthogonal_fixed_side():
    # H^T H = c I, the row observes every column with y_i = <w*, h_i>:  w = c / ((1 + alpha) c + lam) w*
    d, c = 4, 3.0
    Q = np.linalg.qr(np.random.default_rng(7).normal(size=(12, d)))[0]   # 12 x 4, orthonormal columns
    H = np.sqrt(c) * Q
    wstar = np.array([0.3, -1.2, 0.5, 2.0])
    y = H @ wstar
    alpha, lam = 0.6, 0.9
    w = ials.half_step(np.array([0, 12]), np.arange(12, dtype=np.int32), y, H, alpha, lam)[0]
    np.testing.assert_allclose(w, c / ((1 + alpha) * c + lam) * wstar, rtol=1e-12)


def test_alpha_zero_is_ridge_regression():
    rowptr, colidx, vals, W, H, mask = random_problem(15, 12, 4, 0.4, 8)
    lam = 0.15
    got = ials.half_step(rowptr, colidx, vals, H, 0.0, lam)
    for u in range(15):
        cols = colidx[rowptr[u]:rowptr[u + 1]]
        Hu = H[cols]
        ref = np.linalg.solve(Hu.T @ Hu + lam * np.eye(4), Hu.T @ vals[rowptr[u]:rowptr[u + 1]])
        np.testing.assert_allclose(got[u], ref, rtol=1e-10, atol=1e-13)


# ---- the update is the exact minimiser: gradient of Eq. 3, all-pairs term summed explicitly -----

def test_push_through_identity_gives_the_same_row():
    """Eq. 4 restated for a row with k < d observations (the form the library uses for short rows):
    (B + H^T H)^-1 H^T y = B^-1 H^T (I_k + H B^-1 H^T)^-1 y with B = alpha G + lambda I.  The oracle solves the
    d x d form; the k x k form written out with numpy must give the same rows."""
    rowptr, colidx, vals, W, H, _ = random_problem(9, 40, 12, 0.12, 31)
    alpha, lam = 0.07, 0.3
    got = ials.half_step(rowptr, colidx, vals, H, alpha, lam)
    B = alpha * (H.T @ H) + lam * np.eye(H.shape[1])
    Binv = np.linalg.inv(B)
    for u in range(9):
        idx = colidx[rowptr[u]:rowptr[u + 1]]
        if idx.size == 0:
            assert np.all(got[u] == 0)
            continue
        Hu, yu = H[idx], vals[rowptr[u]:rowptr[u + 1]]
        Z = Hu @ Binv
        t = np.linalg.solve(np.eye(idx.size) + Z @ Hu.T, yu)
        np.testing.assert_allclose(got[u], Z.T @ t, rtol=1e-10, atol=1e-13)


def test_gradient_of_objective_vanishes_at_the_update():
    n_rows, n_cols, d = 25, 18, 5
    rowptr, colidx, vals, W, H, mask = random_problem(n_rows, n_cols, d, 0.35, 9)
    alpha, lam = 0.2, 0.05
    Wn = ials.half_step(rowptr, colidx, vals, H, alpha, lam)
    Y = dense_Y(rowptr, colidx, vals, n_rows, n_cols)
    for u in range(n_rows):
        g = np.zeros(d)
        bnorm = np.zeros(d)
        for i in range(n_cols):                         # explicit sum over ALL items, no Gramian
            yhat = Wn[u] @ H[i]
            if mask[u, i]:
                g += -2 * (Y[u, i] - yhat) * H[i]
                bnorm += Y[u, i] * H[i]
            g += 2 * alpha * yhat * H[i]
        g += 2 * lam * Wn[u]
        scale = 2 * np.linalg.norm(bnorm)
        if scale == 0:
            assert np.all(Wn[u] == 0)
        else:
            assert np.linalg.norm(g) / scale <= 1e-9


def test_residual_gate_every_row_medium():
    # spec gate on the oracle itself: |A w - b| / |b| <= 1e-9 for every row, d = 64
    from synth import graphs
    deg = graphs.zipf_degrees(400, 12000, 1.1, 300, 3)
    spec = graphs.GraphSpec(400, 400, 5)
    rowptr, colidx = graphs.build_csr(spec, deg)
    H = graphs.storage_to_f64(graphs.init_embeddings(400, 64, 1, 2, "f32"), "f32")
    alpha, lam = 0.001, 0.05
    G = ials.gramian(H)
    Wn, raw = ials.half_step(rowptr, colidx, None, H, alpha, lam, return_raw=True, G=G)
    for u in range(0, 400, 7):
        A, b = ials.row_system(rowptr, colidx, None, H, G, alpha, lam, u)
        assert np.linalg.norm(A @ raw[u] - b) <= 1e-9 * np.linalg.norm(b)
        assert np.allclose(A, A.T) and np.linalg.eigvalsh(A)[0] >= lam * (1 - 1e-9)


# ---- objective ------------------------------------------------------------------------------------

def test_loss_matches_dense_definition_and_gramian_identity():
    n_rows, n_cols, d = 14, 11, 4
    rowptr, colidx, vals, W, H, mask = random_problem(n_rows, n_cols, d, 0.4, 10)
    alpha, lam = 0.3, 0.7
    Y = dense_Y(rowptr, colidx, vals, n_rows, n_cols)
    P = W @ H.T
    obs = ((Y - P) ** 2)[mask].sum()
    imp = alpha * (P ** 2).sum()
    reg = lam * ((W ** 2).sum() + (H ** 2).sum())
    for explicit in (True, False):
        tot, comp = ials.loss(rowptr, colidx, vals, W, H, alpha, lam, explicit=explicit)
        np.testing.assert_allclose(comp, (obs, imp, reg), rtol=1e-12)
        np.testing.assert_allclose(tot, obs + imp + reg, rtol=1e-12)


@pytest.mark.parametrize("storage,slack", [("f64", 1e-12), ("f32", 1e-7), ("bf16", 1e-5)])
def test_objective_non_increasing(storage, slack):
    n_rows, n_cols, d = 60, 45, 6
    rowptr, colidx, vals, W, H, mask = random_problem(n_rows, n_cols, d, 0.2, 11, binary=True)
    alpha, lam = 0.05, 0.1
    W, H = ials.round_storage(W, storage), ials.round_storage(H, storage)
    colptr, rowidx, vt = ials.transpose(n_rows, n_cols, rowptr, colidx, vals)
    prev = ials.loss(rowptr, colidx, vals, W, H, alpha, lam)[0]
    first = prev
    for ep in range(3):
        W = ials.half_step(rowptr, colidx, vals, H, alpha, lam, storage)
        cur = ials.loss(rowptr, colidx, vals, W, H, alpha, lam)[0]
        assert cur <= prev * (1 + slack)
        prev = cur
        H = ials.half_step(colptr, rowidx, vt, W, alpha, lam, storage)
        cur = ials.loss(rowptr, colidx, vals, W, H, alpha, lam)[0]
        assert cur <= prev * (1 + slack)
        prev = cur
    assert prev < 0.9 * first and prev >= 0


def test_epoch_uses_updated_rows_for_the_column_pass():
    rowptr, colidx, vals, W, H, mask = random_problem(10, 8, 3, 0.5, 12)
    vals = vals.astype(np.float32).astype(np.float64)
    W1, H1 = ials.epoch(rowptr, colidx, vals, W, H, 0.1, 0.2)
    colptr, rowidx, vt = ials.transpose(10, 8, rowptr, colidx, vals)
    np.testing.assert_array_equal(W1, ials.half_step(rowptr, colidx, vals, H, 0.1, 0.2))
    np.testing.assert_array_equal(H1, ials.half_step(colptr, rowidx, vt, W1, 0.1, 0.2))
    H_stale = ials.half_step(colptr, rowidx, vt, W, 0.1, 0.2)
    assert np.abs(H_stale - H1).max() > 1e-3


# ---- invariants -----------------------------------------------------------------------------------

def test_permutation_equivariance():
    n_rows, n_cols, d = 20, 16, 4
    rowptr, colidx, vals, W, H, mask = random_problem(n_rows, n_cols, d, 0.3, 13)
    alpha, lam = 0.2, 0.1
    base = ials.half_step(rowptr, colidx, vals, H, alpha, lam)
    rng = np.random.default_rng(14)
    pr, pc = rng.permutation(n_rows), rng.permutation(n_cols)     # new id of old row u is pr[u]
    Y = dense_Y(rowptr, colidx, vals, n_rows, n_cols)
    Y2 = np.zeros_like(Y); M2 = np.zeros_like(mask)
    Y2[np.ix_(pr, pc)] = Y
    M2[np.ix_(pr, pc)] = mask
    H2 = np.zeros_like(H); H2[pc] = H
    rp2 = np.zeros(n_rows + 1, dtype=np.int64); rp2[1:] = np.cumsum(M2.sum(1))
    ci2 = np.nonzero(M2)[1].astype(np.int32)
    v2 = Y2[M2]
    got = ials.half_step(rp2, ci2, v2, H2, alpha, lam)
    np.testing.assert_allclose(got[pr], base, rtol=1e-10, atol=1e-13)


def test_operation_counters_match_cost_model():
    # Sec. 3: an epoch costs O(d^2 |S| + d^3 (|U| + |I|)): one outer product per observation, one solve per row
    rowptr, colidx, vals, W, H, mask = random_problem(17, 13, 3, 0.4, 15)
    cnt = np.zeros(3, dtype=np.int64)
    ials.half_step(rowptr, colidx, vals, H, 0.1, 0.1, counters=cnt)
    assert cnt[0] == colidx.size and cnt[1] == 17 and cnt[2] == 0


def test_row_subset_equals_full():
    rowptr, colidx, vals, W, H, mask = random_problem(17, 13, 3, 0.4, 16)
    full = ials.half_step(rowptr, colidx, vals, H, 0.1, 0.1)
    ids = np.array([16, 0, 5, 5, 1])
    np.testing.assert_array_equal(ials.half_step(rowptr, colidx, vals, H, 0.1, 0.1, row_ids=ids), full[ids])


# ---- storage rounding (Sec. 4.4) ---------------------------------------------------------------------

def test_bf16_rounding_ties_to_even_and_matches_bit_trick():
    r = lambda x: ials.round_storage(np.array([x]), "bf16")[0]
    assert r(1 + 2.0 ** -8) == 1.0                       # tie -> even significand
    assert r(1 + 3 * 2.0 ** -8) == 1 + 2.0 ** -6         # tie -> even significand
    assert r(1 + 2.0 ** -8 + 2.0 ** -30) == 1 + 2.0 ** -7
    assert r(-0.3) == -r(0.3) and r(0.0) == 0.0
    rng = np.random.default_rng(17)
    x = rng.normal(size=20000).astype(np.float32)        # exactly representable in fp32: no double rounding
    b = x.view(np.uint32)
    ref = (((b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)) << np.uint32(16)).view(np.float32)
    np.testing.assert_array_equal(ials.round_storage(x.astype(np.float64), "bf16"), ref.astype(np.float64))
    y = rng.normal(size=1000)
    np.testing.assert_array_equal(ials.round_storage(y, "f32"), y.astype(np.float32).astype(np.float64))


# ---- integer structures ---------------------------------------------------------------------------

def test_transpose_against_independent_sort_and_scipy():
    import scipy.sparse as sp
    from synth import graphs
    deg = graphs.zipf_degrees(500, 9000, 1.0, 200, 21)
    rowptr, colidx = graphs.build_csr(graphs.GraphSpec(500, 380, 22), np.minimum(deg, 380))
    nnz = colidx.size
    vals = np.arange(nnz, dtype=np.float32)
    colptr, rowidx, vt = ials.transpose(500, 380, rowptr, colidx, vals)
    rows = np.repeat(np.arange(500), np.diff(rowptr))
    order = np.lexsort((rows, colidx))                    # by column, then row
    np.testing.assert_array_equal(rowidx, rows[order].astype(np.int32))
    np.testing.assert_array_equal(vt, vals[order])
    np.testing.assert_array_equal(colptr, np.concatenate([[0], np.cumsum(np.bincount(colidx, minlength=380))]))
    m = sp.csr_matrix((vals + 1, colidx, rowptr), shape=(500, 380)).tocsc()
    m.sort_indices()
    np.testing.assert_array_equal(m.indptr, colptr)
    np.testing.assert_array_equal(m.indices, rowidx)
    # transposing twice gives the original back
    rp2, ci2, v2 = ials.transpose(380, 500, colptr, rowidx, vt)
    np.testing.assert_array_equal(rp2, rowptr)
    np.testing.assert_array_equal(ci2, colidx)
    np.testing.assert_array_equal(v2, vals)


def test_degree_class_rule():
    bounds = [(0, 0), (1, 1), (16, 1), (17, 2), (32, 2), (33, 3), (64, 3), (65, 4), (128, 4), (129, 5),
              (4096, 9), (4097, 10), (8192, 10), (8193, 11), (10 ** 6, 11)]
    for deg, c in bounds:
        assert ials.degree_class(deg) == c
    # smaller split (used by tests to exercise split rows on small inputs)
    assert ials.degree_class(100, split=64) == 11 and ials.degree_class(64, split=64) == 3


def test_bucket_and_chunk_invariants():
    rng = np.random.default_rng(23)
    deg = rng.integers(0, 40, size=3000)
    deg[rng.integers(0, 3000, 40)] = rng.integers(100, 1000, 40)
    deg[5] = 0
    rowptr = np.concatenate([[0], np.cumsum(deg)]).astype(np.int64)
    split = 256
    order, offs = ials.bucket_rows(rowptr, split=split)
    assert sorted(order.tolist()) == list(range(3000))               # a permutation
    cls = np.array([ials.degree_class(x, split=split) for x in deg])
    np.testing.assert_array_equal(order, np.lexsort((np.arange(3000), cls)).astype(np.int32))
    for c in range(ials.N_CLASSES):
        seg = order[offs[c]:offs[c + 1]]
        assert np.all(cls[seg] == c) and np.all(np.diff(seg) > 0)
    desc, first = ials.chunks(rowptr, split=split)
    split_rows = np.nonzero(deg > split)[0]
    assert first.size == split_rows.size + 1 and first[-1] == desc.shape[0]
    np.testing.assert_array_equal(desc[:, 3], np.arange(desc.shape[0]))
    for j, u in enumerate(split_rows):
        d = desc[first[j]:first[j + 1]]
        assert np.all(d[:, 0] == u) and d[0, 1] == rowptr[u] and d[-1, 2] == rowptr[u + 1]
        assert np.all(d[1:, 1] == d[:-1, 2]) and np.all(d[:-1, 2] - d[:-1, 1] == split)
        assert 0 < d[-1, 2] - d[-1, 1] <= split


# ---- streamed Gramian (used by the full-size parity tests) ---------------------------------------------

def test_gramian_stream_equals_gramian_on_a_ragged_table():
    rng = np.random.default_rng(5)
    X = rng.normal(0, 0.3, (1003, 7))
    calls = []

    def block(r0, cnt):
        calls.append((r0, cnt))
        return X[r0:r0 + cnt]
    G = ials.gramian_stream(block, 1003, 7, block_rows=250)
    assert calls == [(0, 250), (250, 250), (500, 250), (750, 250), (1000, 3)]     # every row once, ragged tail
    assert np.abs(G - ials.gramian(X)).max() <= 1e-13 * np.abs(G).max()
    assert np.abs(G - X.T @ X).max() <= 1e-12 * np.abs(G).max()
    # a block function that is handed (or honours) wrong ranges must not go unnoticed
    G_bad = ials.gramian_stream(lambda r0, cnt: X[r0:r0 + min(cnt, 249)], 1003, 7, block_rows=250)
    assert np.abs(G_bad - G).max() > 1e-6 * np.abs(G).max()
    # one block (table shorter than the block size) and an exact multiple
    assert np.allclose(ials.gramian_stream(block, 1003, 7, block_rows=5000), G, rtol=0, atol=1e-13 * np.abs(G).max())
    assert np.allclose(ials.gramian_stream(lambda r0, cnt: X[r0:r0 + cnt], 1000, 7, block_rows=250), X[:1000].T @ X[:1000])


# ---- conjugate gradients (Sec. 4.5): pinned by its limit and by the textbook properties of its iterates ----

def _spd(d, eigs, seed):
    rng = np.random.default_rng(seed)
    Q, _ = np.linalg.qr(rng.standard_normal((d, d)))
    return (Q * np.asarray(eigs, dtype=np.float64)) @ Q.T, rng.standard_normal(d)


def test_cg_converges_to_the_direct_solution():
    A, b = _spd(24, np.linspace(0.5, 40.0, 24), 1)
    x, k = ials.cg(A, b, tol=1e-13, max_iter=200)
    assert np.linalg.norm(x - np.linalg.solve(A, b)) <= 1e-11 * np.linalg.norm(x)
    assert k <= 40
    # d = 1: one step gives b / A
    x1, k1 = ials.cg(np.array([[4.0]]), np.array([3.0]), tol=1e-15, max_iter=5)
    assert k1 == 1 and x1[0] == 0.75
    # zero right-hand side: zero steps, zero solution
    x0, k0 = ials.cg(A, np.zeros(24))
    assert k0 == 0 and np.all(x0 == 0)


def test_cg_is_exact_after_as_many_steps_as_distinct_eigenvalues():
    eigs = np.repeat([0.3, 1.0, 2.5, 7.0, 19.0], 6)          # d = 30, five distinct eigenvalues
    A, b = _spd(30, eigs, 2)
    x, k, its = ials.cg(A, b, tol=1e-9, max_iter=30, return_iterates=True)
    assert k == 5
    assert np.linalg.norm(A @ x - b) <= 1e-9 * np.linalg.norm(b)
    assert np.linalg.norm(A @ its[3] - b) > 1e-6 * np.linalg.norm(b)       # and not before


def test_cg_error_decreases_in_the_energy_norm_and_residuals_are_orthogonal():
    A, b = _spd(40, np.geomspace(0.05, 30.0, 40), 3)
    x_star = np.linalg.solve(A, b)
    _, k, its = ials.cg(A, b, tol=1e-10, max_iter=80, return_iterates=True)
    err = [np.sqrt((x_star - x) @ A @ (x_star - x)) for x in [np.zeros(40)] + list(its)]
    assert all(e1 < e0 for e0, e1 in zip(err, err[1:]))
    R = np.array([b - A @ x for x in [np.zeros(40)] + list(its[:12])])
    Rn = R / np.linalg.norm(R, axis=1, keepdims=True)
    off = Rn @ Rn.T - np.eye(len(Rn))
    assert np.abs(off).max() <= 1e-8
    # each iterate minimises the energy norm over the Krylov space: x_2 against brute force over span{b, A b}
    K = np.stack([b, A @ b], axis=1)
    c = np.linalg.solve(K.T @ A @ K, K.T @ b)
    assert np.linalg.norm(K @ c - its[1]) <= 1e-10 * np.linalg.norm(its[1])


def test_half_step_cg_meets_the_tolerance_and_approaches_the_exact_half_step():
    rowptr, colidx, vals, W, H, _ = random_problem(30, 22, 6, 0.3, 11)
    alpha, lam = 0.05, 0.2
    G = ials.gramian(H)
    exact, exact_raw = ials.half_step(rowptr, colidx, vals, H, alpha, lam, G=G, return_raw=True)
    Y, raw, iters = ials.half_step_cg(rowptr, colidx, vals, H, alpha, lam, G=G, tol=1e-5, max_iter=64)
    assert iters[0] == 0 and np.all(raw[0] == 0)                            # the empty row
    for u in range(1, 30):
        A, b = ials.row_system(rowptr, colidx, vals, H, G, alpha, lam, u)
        assert np.linalg.norm(A @ raw[u] - b) <= 1.0001e-5 * np.linalg.norm(b)
        assert 1 <= iters[u] <= 6                                           # at most d steps
    tight, tight_raw, _ = ials.half_step_cg(rowptr, colidx, vals, H, alpha, lam, G=G, tol=1e-13, max_iter=64)
    assert np.linalg.norm(tight_raw - exact_raw) <= 1e-10 * np.linalg.norm(exact_raw)
