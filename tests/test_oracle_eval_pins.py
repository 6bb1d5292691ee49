"""Pins of the evaluation oracle (fold-in, exact Top-K, Recall@K) against hand-worked examples, closed forms and brute
force -- no GPU, no CUDA code."""
import numpy as np

from oracle import evaluation as ev


def test_topk_hand_example_with_ties_exclusion_and_short_rows():
    # integer-valued, so every score is exact.  scores: q0 = [3 1 3 0 3], q1 = [0 2 5 2 0], q2 = [3 3 8 2 3]
    H = np.array([[3, 0], [1, 2], [3, 5], [0, 2], [3, 0]], dtype=np.float64)
    Q = np.array([[1, 0], [0, 1], [1, 1]], dtype=np.float64)
    ids, sc = ev.topk(Q, H, 3)
    np.testing.assert_array_equal(ids, [[0, 2, 4], [2, 1, 3], [2, 0, 1]])      # equal scores: the smaller id first
    np.testing.assert_array_equal(sc, [[3, 3, 3], [5, 2, 2], [8, 3, 3]])
    ptr = np.array([0, 1, 1, 3])
    idx = np.array([0, 0, 2])
    ids, sc = ev.topk(Q, H, 3, exclude=(ptr, idx))
    np.testing.assert_array_equal(ids, [[2, 4, 1], [2, 1, 3], [1, 4, 3]])
    ids, sc = ev.topk(Q, H, 6)
    np.testing.assert_array_equal(ids[0], [0, 2, 4, 1, 3, -1])
    assert sc[0, 5] == -np.inf


def test_topk_matches_brute_force_loops():
    rng = np.random.default_rng(5)
    H = rng.integers(-3, 4, (40, 5)).astype(np.float64)      # small integers: many exact ties
    Q = rng.integers(-3, 4, (7, 5)).astype(np.float64)
    ids, _ = ev.topk(Q, H, 9)
    for q in range(Q.shape[0]):
        scored = []
        for i in range(H.shape[0]):
            s = 0.0
            for f in range(H.shape[1]):
                s += Q[q, f] * H[i, f]
            scored.append((-s, i))
        scored.sort()
        assert [i for _, i in scored[:9]] == list(ids[q])


def test_recall_hand_example():
    ids = np.array([[3, 7, 9], [1, 2, 4], [5, 6, 8]])
    tptr = np.array([0, 2, 2, 5])
    tidx = np.array([7, 11, 5, 8, 20])
    r, n = ev.recall_at_k(ids, 3, tptr, tidx)       # q0: 1 of 2, q1: no ground truth (left out), q2: 2 of 3
    assert n == 2 and abs(r - (0.5 + 2.0 / 3.0) / 2) < 1e-15
    r, n = ev.recall_at_k(ids, 1, tptr, tidx)       # q0: 0 of 2, q2: 1 of 3
    assert n == 2 and abs(r - (1.0 / 3.0) / 2) < 1e-15


def test_fold_in_closed_form_for_a_single_link():
    """H with orthogonal columns of equal norm: H^T H = c I, so alpha0 G + lambda I = beta I and a row with the single
    link (i, y) has the solution y h_i / (beta + |h_i|^2) (Sherman-Morrison)."""
    rng = np.random.default_rng(8)
    n, d, alpha, lam, c = 30, 6, 0.3, 0.2, 2.5
    Qm, _ = np.linalg.qr(rng.normal(size=(n, d)))
    H = Qm * np.sqrt(c)
    rowptr = np.array([0, 1, 2, 2])
    colidx = np.array([4, 17], dtype=np.int32)
    vals = np.array([1.0, -0.7])
    W, _ = ev.fold_in(rowptr, colidx, vals, H, alpha, lam)
    beta = alpha * c + lam
    for r, (i, y) in enumerate([(4, 1.0), (17, -0.7)]):
        np.testing.assert_allclose(W[r], y * H[i] / (beta + H[i] @ H[i]), rtol=1e-12, atol=1e-15)
    np.testing.assert_array_equal(W[2], 0.0)


def test_fold_in_minimises_the_row_objective_by_brute_force():
    """The row objective of Eq. 3 written out over ALL columns (no Gramian): the fold-in solution has a vanishing
    finite-difference gradient and no random neighbour does better."""
    rng = np.random.default_rng(9)
    n, d, alpha, lam = 25, 4, 0.15, 0.05
    H = rng.normal(0, 0.6, (n, d))
    links = np.array([2, 9, 10, 21], dtype=np.int32)
    y = np.array([1.0, 0.5, 2.0, 1.0])
    W, _ = ev.fold_in(np.array([0, 4]), links, y, H, alpha, lam)

    def objective(w):
        f = lam * float(w @ w)
        for i in range(n):
            f += alpha * float(w @ H[i]) ** 2
        for i, yi in zip(links, y):
            f += (yi - float(w @ H[i])) ** 2
        return f

    w = W[0]
    f0 = objective(w)
    for f_ in range(d):
        e = np.zeros(d); e[f_] = 1e-6
        assert abs(objective(w + e) - objective(w - e)) / 2e-6 < 1e-8
    for _ in range(50):
        assert objective(w + rng.normal(0, 1e-2, d)) > f0
