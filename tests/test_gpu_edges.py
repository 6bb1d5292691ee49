"""Edge cases of the half-step through the C ABI: row lengths on both sides of every degree-class and kernel boundary
(1, 16 / 17, 32 / 33, 64 / 65, 512 / 513, 1024 / 1025, above the split threshold), a single row, a single column,
every supported (d, storage) pair, labelled and unlabelled -- one epoch each with the full set of gates against the
oracle (both half-steps: table, per-row maximum, exact zeros, residuals, loss)."""
import numpy as np
import pytest

from tests import problems
from tests.test_gpu_parity import _epoch_checks

pytestmark = pytest.mark.gpu

BOUNDARY_DEGREES = [0, 1, 2, 3, 4, 5, 8, 9, 15, 16, 17, 31, 32, 33, 63, 64, 65, 127, 128, 129, 255, 256, 257, 511, 512, 513,
                    1023, 1024, 1025, 1500, 2047, 2048, 2049, 3000]


def boundary_problem(name, d, storage, n_cols, split, values, seed, repeat=3, extra_rows=200):
    """Rows whose lengths sit on the boundaries (each `repeat` times, capped at n_cols), plus a few hundred ordinary rows so that
    the columns get a spread of lengths too."""
    rng = np.random.Generator(np.random.PCG64(seed))
    deg = [min(k, n_cols) for k in BOUNDARY_DEGREES for _ in range(repeat)]
    deg += list(rng.integers(1, 40, extra_rows))
    deg = np.asarray(deg, dtype=np.int64)
    rng.shuffle(deg)
    n_rows = deg.size
    rowptr = np.zeros(n_rows + 1, dtype=np.int64)
    rowptr[1:] = np.cumsum(deg)
    # popular columns first, so that a few columns are long (they cross the same boundaries on the columns side)
    weights = 1.0 / np.arange(1, n_cols + 1) ** 0.7
    weights /= weights.sum()
    cols = [np.sort(rng.choice(n_cols, int(k), replace=False, p=weights)) if k < n_cols else np.arange(n_cols) for k in deg]
    colidx = np.concatenate(cols).astype(np.int32)
    vals = rng.uniform(0.25, 2.0, colidx.size).astype(np.float32) if values else None
    W0, H0 = problems._tables(n_rows, n_cols, d, seed + 1, storage)
    return problems.Problem(name, n_rows, n_cols, d, 0.05, 0.003, storage, rowptr, colidx, vals, W0, H0, split)


CASES = [
    ("edges_d128_bf16", 128, "bf16", 3100, 0, False),
    ("edges_d128_bf16_labels_split", 128, "bf16", 3100, 1024, True),
    ("edges_d64_f32", 64, "f32", 3100, 0, False),
    ("edges_d64_f32_labels_split", 64, "f32", 3100, 512, True),
    ("edges_d128_f32", 128, "f32", 2100, 256, True),
    ("edges_d64_bf16", 64, "bf16", 2100, 0, False),
    ("edges_d32_f32", 32, "f32", 2100, 128, False),
    ("edges_d16_bf16", 16, "bf16", 1100, 64, True),
]


@pytest.mark.parametrize("name,d,storage,n_cols,split,values", CASES, ids=[c[0] for c in CASES])
def test_rows_on_every_boundary(name, d, storage, n_cols, split, values):
    seed = 7 + 11 * [c[0] for c in CASES].index(name)
    _epoch_checks(boundary_problem(name, d, storage, n_cols, split, values, seed=seed))


@pytest.mark.parametrize("d,storage", [(128, "bf16"), (64, "f32"), (16, "f32")])
def test_single_row_and_single_column_matrices(d, storage):
    rng = np.random.Generator(np.random.PCG64(5))
    # one row that links to 40 of 300 columns
    cols = np.sort(rng.choice(300, 40, replace=False)).astype(np.int32)
    W0, H0 = problems._tables(1, 300, d, 3, storage)
    _epoch_checks(problems.Problem("one_row", 1, 300, d, 0.05, 0.01, storage, np.array([0, 40], dtype=np.int64), cols, None, W0, H0))
    # 300 rows, one column: rows have one entry or none.  Every non-empty row then has the same embedding, so the column's
    # system is dominated by one direction and its solution is sensitive to the last bit of W: the rows half-step is held
    # to the usual gates, the column to its residual and to the exact solve from the GPU's own W.
    from oracle import ials
    from tests.test_gpu_parity import make_ctx, rel_fro
    deg = (rng.random(300) < 0.6).astype(np.int64)
    rowptr = np.zeros(301, dtype=np.int64)
    rowptr[1:] = np.cumsum(deg)
    W0, H0 = problems._tables(300, 1, d, 4, storage)
    p = problems.Problem("one_column", 300, 1, d, 0.05, 0.01, storage, rowptr, np.zeros(int(deg.sum()), dtype=np.int32), None, W0, H0)
    a = make_ctx(p)
    a.half_epoch(0)
    dt = "bf16" if storage == "bf16" else "f32"
    W = p.f64(a.get_embeddings(0, dtype=dt))
    W_ref = ials.half_step(p.rowptr, p.colidx, None, p.f64(p.H0), p.alpha, p.lam, p.storage)
    assert rel_fro(W, W_ref) <= p.emb_tol and np.all(W[deg == 0] == 0.0)
    x32 = a.half_epoch_capture(1, np.zeros(1, dtype=np.int64)).astype(np.float64)
    assert a.get_stats().not_spd == 0
    a.destroy()
    colptr, rowidx, _ = ials.transpose(p.n_rows, p.n_cols, p.rowptr, p.colidx, None)
    G = ials.gramian(W)
    A, b = ials.row_system(colptr, rowidx, None, W, G, p.alpha, p.lam, 0)
    assert np.linalg.norm(A @ x32[0] - b) <= 1e-4 * np.linalg.norm(b)
    exact = np.linalg.solve(A, b)
    # (an fp32 solve is backward stable: its error is bounded by cond(A) d 2^-23, and this matrix -- 180 copies of one outer
    # product on top of lambda I -- has a condition of 10^4 .. 10^5: the residual above is the gate that means something)
    assert np.linalg.norm(x32[0] - exact) <= max(p.emb_tol, d * 1.2e-7 * np.linalg.cond(A)) * np.linalg.norm(exact)


@pytest.mark.parametrize("case", [0, 3], ids=["edges_d128_bf16", "edges_d64_f32_labels_split"])
def test_six_epochs_on_the_boundary_problems_each_match_the_oracle_epoch(case):
    """Several epochs in a row: the solver choice per side, the routing of the rows of 17..32 entries and the start vectors
    all depend on the context's history.  Every epoch is compared with the oracle's epoch from the SAME start tables (the
    GPU's own, read back before the epoch): tables within the tolerance, loss to 1e-4, and the loss must not rise.  (Two
    free-running trajectories drift apart by the storage rounding of every epoch, which says nothing about an epoch.)"""
    from oracle import ials
    from tests.test_gpu_parity import make_ctx, rel_fro
    name, d, storage, n_cols, split, values = CASES[case]
    p = boundary_problem(name, d, storage, n_cols, split, values, seed=7 + 11 * case)
    a = make_ctx(p)
    dt = "bf16" if storage == "bf16" else "f32"
    colptr, rowidx, vt = ials.transpose(p.n_rows, p.n_cols, p.rowptr, p.colidx, p.values)
    v64 = None if p.values is None else p.values.astype(np.float64)
    vt64 = None if vt is None else vt.astype(np.float64)
    prev = a.loss()[0]
    H = p.f64(p.H0)
    for ep in range(6):
        a.half_epoch(0)
        dual_rows = a.get_stats().dual_rows
        a.half_epoch(1)
        W_ref = ials.half_step(p.rowptr, p.colidx, v64, H, p.alpha, p.lam, p.storage)
        H_ref = ials.half_step(colptr, rowidx, vt64, W_ref, p.alpha, p.lam, p.storage)
        W_gpu = p.f64(a.get_embeddings(0, dtype=dt))
        H_gpu = p.f64(a.get_embeddings(1, dtype=dt))
        tot = a.loss()[0]
        ref = ials.loss(p.rowptr, p.colidx, v64, W_ref, H_ref, p.alpha, p.lam)[0]
        st = a.get_stats()
        print(f"{name} epoch {ep + 1}: W {rel_fro(W_gpu, W_ref):.2e} H {rel_fro(H_gpu, H_ref):.2e} loss {abs(tot - ref) / ref:.2e}, "
              f"dual-form rows {dual_rows}, products per row {st.cg_products / max(st.cg_rows, 1):.1f}, Cholesky by policy "
              f"{list(st.cholesky_by_policy)}")
        assert rel_fro(W_gpu, W_ref) <= p.emb_tol and rel_fro(H_gpu, H_ref) <= p.emb_tol
        assert abs(tot - ref) <= 1e-4 * ref
        assert tot <= prev * (1 + 1e-6) and st.not_spd == 0
        prev = tot
        H = H_gpu
    a.destroy()


OPTION_SETS = [
    dict(solver=1), dict(kernels=1), dict(kernels=2), dict(cg_start=1), dict(cg_max_iter=3), dict(cg_max_iter=200),
    dict(cg_tol=1e-7), dict(dual_cond_limit=1.0), dict(dual_cond_limit=1e9), dict(cg_switch_products=1.0),
    dict(solver=1, kernels=2), dict(cg_start=1, dual_cond_limit=1.0, cg_max_iter=5), dict(kernels=2, cg_tol=3e-6, cg_start=1),
]


@pytest.mark.parametrize("case", [1, 3, 6], ids=["edges_d128_bf16_labels_split", "edges_d64_f32_labels_split", "edges_d32_f32"])
@pytest.mark.parametrize("opt", range(len(OPTION_SETS)), ids=[",".join(f"{k}={v}" for k, v in o.items()) for o in OPTION_SETS])
def test_every_option_gives_the_same_epoch(case, opt):
    """The options choose HOW a row is solved (kernel family, solver, start vector, step limit, limits), never WHAT: one
    epoch of a boundary problem under each setting, held to the gates of the storage type and of the residual.  These
    problems have rows with cond(A) of a few thousand, where conjugate gradients stopped at a relative residual leave
    an error of cond(A) times that: the solver's fp32 solution is therefore held to the storage type's tolerance here,
    not to the 1e-3 that the direct solves and the better conditioned suites reach."""
    name, d, storage, n_cols, split, values = CASES[case]
    p = boundary_problem(name, d, storage, n_cols, split, values, seed=7 + 11 * case)
    _epoch_checks(p, raw_gate=(p.emb_tol, 10 * p.emb_tol), **OPTION_SETS[opt])
