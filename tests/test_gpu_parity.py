"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest

from oracle import ials
from tests import problems

pytestmark = pytest.mark.gpu

ROWS, COLS = 0, 1


def make_ctx(p, kernels=0, **kw):
    from paper_2112_02194_b200 import Alx
    a = Alx(p.n_rows, p.n_cols, p.d, p.lam, p.alpha, storage=p.storage, split=p.split, kernels=kernels, **kw)
    a.set_csr(p.rowptr, p.colidx, p.values)
    a.set_embeddings(ROWS, p.W0)
    a.set_embeddings(COLS, p.H0)
    return a


def rel_fro(x, ref):
    return np.linalg.norm(x - ref) / max(np.linalg.norm(ref), 1e-300)


def row_rel(x, ref):
    num = np.linalg.norm(x - ref, axis=1)
    den = np.linalg.norm(ref, axis=1)
    ok = den > 0
    return num[ok] / den[ok]


# maximum of the per-row relative error, as a multiple of the table tolerance (a row is one of up to 10^4: the table
# gate alone would let a few rows be arbitrarily wrong)
ROW_MAX_FACTOR = 10.0


def _check_half_step(p, side, X_gpu, X_ref, X_raw, x32, deg, ptr, idx, vals64, X_fixed, G, raw_gate=(1e-3, 1e-2)):
    """The gates of one half-step: the table (Frobenius), every row (99.9th percentile and maximum of the per-row relative
    error), exact zeros for rows without observations, the residual of the solver's own fp32 solutions."""
    rr = row_rel(X_gpu, X_ref)
    print(f"{p.name} {side}: table {rel_fro(X_gpu, X_ref):.2e}, per row p99.9 {np.quantile(rr, 0.999):.2e} max {rr.max():.2e} "
          f"(tolerance {p.emb_tol:g})")
    assert rel_fro(X_gpu, X_ref) <= p.emb_tol
    assert np.quantile(rr, 0.999) <= 10 * p.emb_tol
    assert rr.max() <= ROW_MAX_FACTOR * p.emb_tol, rr.max()
    assert np.all(X_gpu[deg == 0] == 0.0) and np.all(x32[deg == 0] == 0)
    zero_rhs = ~np.any(X_raw != 0.0, axis=1)          # no observation, or every label 0: the solution is exactly 0
    assert np.all(X_gpu[zero_rhs] == 0.0) and np.all(x32[zero_rhs] == 0)
    # residual gate |A x - b| / |b| <= 1e-4 on the solver's own fp32 solution, A and b rebuilt in fp64: the 40 longest
    # rows and about 150 more spread over the ids
    n = deg.size
    worst = 0.0
    check = np.unique(np.concatenate([np.argsort(deg)[-40:], np.arange(0, n, max(1, n // 150))]))
    for u in check:
        if deg[u] == 0:
            continue
        A, b = ials.row_system(ptr, idx, vals64, X_fixed, G, p.alpha, p.lam, int(u))
        nb = np.linalg.norm(b)
        if nb == 0:
            assert np.all(x32[u] == 0)
            continue
        worst = max(worst, np.linalg.norm(A @ x32[u].astype(np.float64) - b) / nb)
    print(f"{p.name} {side}: worst residual of {check.size} rows {worst:.2e}")
    assert worst <= 1e-4, worst
    # the solver's own fp32 solution against the exact one (before the storage cast): table and worst row.  A row's
    # error is at most cond(A) times its relative residual (gated above), and conjugate gradients stop at 3e-5 for
    # bfloat16 tables: a worst row of 1e-2 sits at the rounding edge there (0.0099 or 0.0105 with the order of the
    # solver's sums), so bfloat16 problems take the storage type's own tolerance, 2e-2, as the worst-row gate.
    xr = row_rel(x32.astype(np.float64), X_raw)
    row_gate = max(raw_gate[1], p.emb_tol) if p.storage == "bf16" else raw_gate[1]
    assert rel_fro(x32.astype(np.float64), X_raw) <= raw_gate[0] and xr.max() <= row_gate, (rel_fro(x32.astype(np.float64), X_raw), xr.max())


SUITE = problems.small_suite()
IDS = ["tiny", "zipf_d64_f32", "local_d128_bf16", "split_d128_bf16", "split_d32_f32_labels", "alpha0_d16_bf16",
       "default_split_d64_bf16", "long_labels_d128_bf16", "split_labels_d128_bf16", "zero_labels_d128_f32",
       "uniform_d32_bf16", "split_labels_d64_f32"]


@pytest.fixture(scope="module", params=list(range(len(SUITE))), ids=IDS)
def prob(request):
    return SUITE[request.param]()


def test_transpose_and_buckets_bit_exact(prob):
    p = prob
    a = make_ctx(p)
    split = p.split or ials.SPLIT
    colptr, rowidx, vt = a.get_transpose(p.nnz, with_values=p.values is not None)
    o_colptr, o_rowidx, o_vt = ials.transpose(p.n_rows, p.n_cols, p.rowptr, p.colidx, p.values)
    np.testing.assert_array_equal(colptr, o_colptr)
    np.testing.assert_array_equal(rowidx, o_rowidx)
    if p.values is not None:
        np.testing.assert_array_equal(vt, o_vt)
    for side, ptr in ((ROWS, p.rowptr), (COLS, o_colptr)):
        order, offs, desc = a.get_buckets(side)
        o_order, o_offs = ials.bucket_rows(ptr, split=split)
        o_desc, _ = ials.chunks(ptr, split=split)
        np.testing.assert_array_equal(order, o_order)
        np.testing.assert_array_equal(offs, o_offs)
        np.testing.assert_array_equal(desc, o_desc)
    a.destroy()


def test_gramian_matches_oracle(prob):
    p = prob
    a = make_ctx(p)
    for side, tab in ((ROWS, p.W0), (COLS, p.H0)):
        G = a.gramian(side)
        ref = ials.gramian(p.f64(tab))
        # 1e-6 for fp32 FMA sums; the tensor-core accumulator truncates (up to 2^-24 per 16-row step, always
        # towards zero, 16 steps per read-out), which adds a bias of up to ~1e-6 on the diagonal
        print(f"{p.name} Gramian of side {side}: max |G - ref| / max |ref| = {np.abs(G - ref).max() / np.abs(ref).max():.2e}, "
              f"diagonal bias {np.mean(np.diag(G - ref)) / np.mean(np.diag(ref)):+.2e}")
        assert np.abs(G - ref).max() <= 2e-6 * np.abs(ref).max()
        np.testing.assert_array_equal(G, G.T)
    a.destroy()


def test_epoch_embeddings_residual_and_loss(prob):
    _epoch_checks(prob)


@pytest.mark.parametrize("name", ["local_d128_bf16", "split_d128_bf16", "zipf_d64_f32", "split_labels_d64_f32"])
def test_fp32_alu_kernels_on_the_tensor_path_problems(name):
    """kernels = 1 forces the FP32-ALU kernels where the tensor-core kernels would run (d = 128 with bfloat16 tables,
    d = 64 with fp32 tables): the same gates against the oracle."""
    _epoch_checks(_problem(name), kernels=1)


def _epoch_checks(p, raw_gate=(1e-3, 1e-2), **ctx_kw):
    a = make_ctx(p, **ctx_kw)
    W0, H0 = p.f64(p.W0), p.f64(p.H0)
    colptr, rowidx, vt = ials.transpose(p.n_rows, p.n_cols, p.rowptr, p.colidx, p.values)
    vals64 = None if p.values is None else p.values.astype(np.float64)
    vt64 = None if vt is None else vt.astype(np.float64)

    # loss at the initial tables: isolates the loss kernels
    tot, comp = a.loss()
    o_tot, o_comp = ials.loss(p.rowptr, p.colidx, vals64, W0, H0, p.alpha, p.lam)
    np.testing.assert_allclose(comp, o_comp, rtol=1e-6, atol=1e-12 * o_tot)

    # --- rows half-step, with the fp32 solutions before rounding captured for every row
    ids = np.arange(p.n_rows, dtype=np.int64)
    x32 = a.half_epoch_capture(ROWS, ids)
    W_gpu = p.f64(a.get_embeddings(ROWS, dtype=p.storage))
    G = ials.gramian(H0)
    W_ref, W_raw = ials.half_step(p.rowptr, p.colidx, vals64, H0, p.alpha, p.lam, p.storage, G=G, return_raw=True)
    deg = np.diff(p.rowptr)
    _check_half_step(p, "rows", W_gpu, W_ref, W_raw, x32, deg, p.rowptr, p.colidx, vals64, H0, G, raw_gate)

    # --- columns half-step on the GPU's own new W (trajectories may differ by storage rounding): the same gates
    cids = np.arange(p.n_cols, dtype=np.int64)
    h32 = a.half_epoch_capture(COLS, cids)
    H_gpu = p.f64(a.get_embeddings(COLS, dtype=p.storage))
    G_W = ials.gramian(W_gpu)
    H_ref_same, H_raw_same = ials.half_step(colptr, rowidx, vt64, W_gpu, p.alpha, p.lam, p.storage, G=G_W, return_raw=True)
    cdeg = np.diff(colptr)
    _check_half_step(p, "columns", H_gpu, H_ref_same, H_raw_same, h32, cdeg, colptr, rowidx, vt64, W_gpu, G_W, raw_gate)
    # and end to end against the oracle's own trajectory
    H_ref = ials.half_step(colptr, rowidx, vt64, W_ref, p.alpha, p.lam, p.storage)
    assert rel_fro(H_gpu, H_ref) <= p.emb_tol

    # loss: kernel on the GPU's tables vs oracle on the same tables; and end to end
    tot, comp = a.loss()
    o_tot, o_comp = ials.loss(p.rowptr, p.colidx, vals64, W_gpu, H_gpu, p.alpha, p.lam)
    assert abs(tot - o_tot) <= 1e-6 * o_tot
    e_tot, _ = ials.loss(p.rowptr, p.colidx, vals64, W_ref, H_ref, p.alpha, p.lam)
    assert abs(tot - e_tot) <= 1e-4 * e_tot
    st = a.get_stats()
    assert st.not_spd == 0 and st.nnz == p.nnz
    a.destroy()


def test_run_to_run_bitwise_determinism(prob):
    p = prob
    outs = []
    for _ in range(2):
        a = make_ctx(p)
        a.epoch()
        outs.append((a.get_embeddings(ROWS, dtype=p.storage).copy(), a.get_embeddings(COLS, dtype=p.storage).copy(),
                     a.loss()[0]))
        a.destroy()
    np.testing.assert_array_equal(outs[0][0], outs[1][0])
    np.testing.assert_array_equal(outs[0][1], outs[1][1])
    assert outs[0][2] == outs[1][2]


def test_three_epochs_loss_tracks_oracle_and_decreases():
    p = SUITE[1]()            # d = 64, fp32: the shape of the "3 epochs with loss tracked" configuration
    a = make_ctx(p)
    W, H = p.f64(p.W0), p.f64(p.H0)
    colptr, rowidx, vt = ials.transpose(p.n_rows, p.n_cols, p.rowptr, p.colidx, None)
    prev = a.loss()[0]
    for ep in range(3):
        a.epoch()
        W = ials.half_step(p.rowptr, p.colidx, None, H, p.alpha, p.lam, p.storage)
        H = ials.half_step(colptr, rowidx, None, W, p.alpha, p.lam, p.storage)
        tot = a.loss()[0]
        ref = ials.loss(p.rowptr, p.colidx, None, W, H, p.alpha, p.lam)[0]
        assert abs(tot - ref) <= 1e-4 * ref
        assert tot <= prev * (1 + 1e-6)
        prev = tot
    a.destroy()


def test_device_pointers_and_ranged_reads():
    import torch
    p = SUITE[2]()
    from paper_2112_02194_b200 import Alx
    a = Alx(p.n_rows, p.n_cols, p.d, p.lam, p.alpha, storage=p.storage)
    dev = torch.device("cuda")
    a.set_csr(torch.from_numpy(p.rowptr).to(dev), torch.from_numpy(p.colidx).to(dev))
    H_t = torch.from_numpy(p.H0.view(np.int16)).to(dev).view(torch.bfloat16)
    a.set_embeddings(COLS, H_t)
    a.set_embeddings(ROWS, p.f64(p.W0).astype(np.float32))     # fp32 source into a bf16 table: converted
    np.testing.assert_array_equal(a.get_embeddings(ROWS, dtype="bf16"), p.W0)
    a.half_epoch(ROWS)
    full = a.get_embeddings(ROWS, dtype="bf16")
    part = a.get_embeddings(ROWS, dtype="bf16", row_begin=100, row_count=37)
    np.testing.assert_array_equal(part, full[100:137])
    out = torch.empty((37, p.d), dtype=torch.float32, device=dev)
    a.get_embeddings(ROWS, row_begin=100, row_count=37, out=out)
    np.testing.assert_array_equal(out.cpu().numpy(), p.f64(part).astype(np.float32))
    b = make_ctx(p)
    b.half_epoch(ROWS)
    np.testing.assert_array_equal(b.get_embeddings(ROWS, dtype="bf16"), full)
    a.destroy(); b.destroy()


@pytest.mark.parametrize("which", [1, 2, 7])
def test_overlapped_host_calls_match_the_separate_calls(which):
    """alx_load_host + alx_epoch_to_host (copies overlapped with kernels on a second stream) give, bit for bit, what
    alx_set_csr + alx_set_embeddings x2 + alx_epoch + alx_get_embeddings x2 give; page-locked buffers, labelled or not."""
    import torch
    p = SUITE[which]()
    dt = "bf16" if p.storage == "bf16" else "f32"
    a = make_ctx(p)
    a.epoch()
    W_ref, H_ref = a.get_embeddings(ROWS, dtype=dt), a.get_embeddings(COLS, dtype=dt)
    a.destroy()
    from paper_2112_02194_b200 import Alx

    def pinned(x):
        t = torch.empty(x.shape, dtype=torch.int16 if x.dtype == np.uint16 else torch.float32, pin_memory=True)
        arr = t.numpy().view(x.dtype)
        arr[...] = x
        return t, arr
    b = Alx(p.n_rows, p.n_cols, p.d, p.lam, p.alpha, storage=p.storage, split=p.split)
    keepW, W0 = pinned(p.W0)
    keepH, H0 = pinned(p.H0)
    keepWo, W_out = pinned(np.zeros_like(p.W0))
    keepHo, H_out = pinned(np.zeros_like(p.H0))
    b.load_host(p.rowptr, p.colidx, p.values, W0, H0)
    b.epoch_to_host(W_out, H_out)
    np.testing.assert_array_equal(W_out, W_ref)
    np.testing.assert_array_equal(H_out, H_ref)
    # and once more on the same context (the second stream and its event are reused).  The context remembers what the
    # conjugate gradients of each side cost last time and may pick Cholesky now: the same solution to within what the
    # solver's stopping rule allows (a tenth of the table tolerance), not the same bits
    b.load_host(p.rowptr, p.colidx, p.values, W0, H0)
    b.epoch_to_host(W_out, H_out)
    for got, ref in ((W_out, W_ref), (H_out, H_ref)):
        assert rel_fro(p.f64(got), p.f64(ref)) <= 0.1 * p.emb_tol
    b.destroy()
    # with one solver throughout, the second round gives the same bits too
    c = Alx(p.n_rows, p.n_cols, p.d, p.lam, p.alpha, storage=p.storage, split=p.split, solver=1)
    outs = []
    for _ in range(2):
        c.load_host(p.rowptr, p.colidx, p.values, W0, H0)
        c.epoch_to_host(W_out, H_out)
        outs.append((W_out.copy(), H_out.copy()))
    np.testing.assert_array_equal(outs[0][0], outs[1][0])
    np.testing.assert_array_equal(outs[0][1], outs[1][1])
    c.destroy()


def test_error_paths_return_status_codes():
    from paper_2112_02194_b200 import Alx, AlxError
    with pytest.raises(AlxError) as e:
        Alx(10, 10, 16, 0.0, 0.1)                       # lambda = 0: minimiser not unique
    assert e.value.status == 7
    with pytest.raises(AlxError) as e:
        Alx(10, 10, 24, 0.1, 0.1)                       # unsupported d
    assert e.value.status == 7
    with pytest.raises(AlxError) as e:
        Alx(0, 10, 16, 0.1, 0.1)
    assert e.value.status == 1
    a = Alx(4, 5, 16, 0.1, 0.1)
    with pytest.raises(AlxError) as e:
        a.half_epoch(ROWS)                              # before the matrix is set
    assert e.value.status == 2
    rowptr = np.array([0, 2, 2, 3, 5], dtype=np.int64)
    good = np.array([0, 3, 1, 2, 4], dtype=np.int32)
    for bad_cols, code in ((np.array([3, 0, 1, 2, 4], dtype=np.int32), 5),      # not ascending
                           (np.array([0, 0, 1, 2, 4], dtype=np.int32), 5),      # duplicate
                           (np.array([0, 5, 1, 2, 4], dtype=np.int32), 5),      # out of range
                           (np.array([0, -1, 1, 2, 4], dtype=np.int32), 5)):
        with pytest.raises(AlxError) as e:
            a.set_csr(rowptr, bad_cols)
        assert e.value.status == code
    with pytest.raises(AlxError) as e:
        a.set_csr(np.array([0, 3, 2, 3, 5], dtype=np.int64), good)             # rowptr not monotone
    assert e.value.status == 5
    a.set_csr(rowptr, good)                                                    # the context is still usable
    with pytest.raises(AlxError) as e:
        a.half_epoch(ROWS)                                                     # fixed table not set
    assert e.value.status == 2
    a.set_embeddings(COLS, np.ones((5, 16), dtype=np.float32))
    a.half_epoch(ROWS)
    w = a.get_embeddings(ROWS)
    assert np.all(w[1] == 0) and np.all(np.isfinite(w))
    with pytest.raises(AlxError):
        a.get_embeddings(ROWS, row_begin=3, row_count=5)
    a.destroy()


def test_empty_matrix_gives_zero_tables():
    from paper_2112_02194_b200 import Alx
    a = Alx(7, 9, 32, 0.1, 0.01)
    a.set_csr(np.zeros(8, dtype=np.int64), np.zeros(0, dtype=np.int32))
    a.set_embeddings(ROWS, np.ones((7, 32), dtype=np.float32))
    a.set_embeddings(COLS, np.ones((9, 32), dtype=np.float32))
    a.epoch()
    assert np.all(a.get_embeddings(ROWS) == 0) and np.all(a.get_embeddings(COLS) == 0)
    assert a.loss()[0] == 0.0
    a.destroy()


def test_device_generators_match_numpy():
    import torch
    from synth import device, graphs
    n = 20000
    deg = graphs.zipf_degrees(n, 500000, 1.1, 6000, 5)
    for spec in (graphs.GraphSpec(n, n, 9, law=graphs.LAW_LOCAL, delta=200),
                 graphs.GraphSpec(n, n, 9, qtable=graphs.zipf_quantile_table(n, 1.1, 0.01)),
                 graphs.GraphSpec(n, n - 777, 10)):
        rowptr, colidx = graphs.build_csr(spec, deg)
        rp_t, ci_t = device.device_csr(spec, deg)
        np.testing.assert_array_equal(rp_t.cpu().numpy(), rowptr)
        np.testing.assert_array_equal(ci_t.cpu().numpy(), colidx)
    for storage in ("f32", "bf16"):
        ref = graphs.init_embeddings(3000, 128, 7, 2, storage)
        t = device.device_embeddings(3000, 128, 7, 2, storage)
        got = t.view(torch.int16).cpu().numpy().view(np.uint16) if storage == "bf16" else t.cpu().numpy()
        np.testing.assert_array_equal(got, ref)


def _problem(name):
    for make in problems.small_suite():
        p = make()
        if p.name == name:
            return p
    raise KeyError(name)


def _class1_rows(p):
    """rows of 1 .. 32 observations: the ones the dual form takes"""
    deg = np.diff(p.rowptr)
    return np.nonzero((deg >= 1) & (deg <= 32))[0].astype(np.int64)


def test_dual_form_for_short_rows_matches_oracle_and_primal_form():
    """Rows with at most 32 observations are solved through the push-through identity (a k x k system); the
    result must satisfy the same residual gate as the primal form and agree with it."""
    p = _problem("local_d128_bf16")
    ids = _class1_rows(p)
    assert ids.size > 100
    H0 = p.f64(p.H0)
    G = ials.gramian(H0)
    sols = {}
    for kernels in (0, 2):
        a = make_ctx(p, kernels=kernels)
        sols[kernels] = a.half_epoch_capture(ROWS, ids).astype(np.float64)
        st = a.get_stats()
        assert st.dual_rows == (ids.size if kernels == 0 else 0)
        assert st.not_spd == 0
        a.destroy()
    _, W_raw = ials.half_step(p.rowptr, p.colidx, None, H0, p.alpha, p.lam, p.storage, row_ids=ids, G=G, return_raw=True)
    for kernels in (0, 2):
        assert rel_fro(sols[kernels], W_raw) <= 1e-4
    worst = 0.0
    for n, u in enumerate(ids):
        A, b = ials.row_system(p.rowptr, p.colidx, None, H0, G, p.alpha, p.lam, int(u))
        worst = max(worst, np.linalg.norm(A @ sols[0][n] - b) / np.linalg.norm(b))
    assert worst <= 1e-4, worst


def test_dual_form_beyond_its_condition_limit_is_polished_or_steps_aside():
    """alpha0 G + lambda I with a condition number of about 4e4: the dual form alone would lose four digits.  With
    conjugate gradients available its solutions are only the start vectors of a conjugate-gradient pass over the same
    rows (which stops at the usual residual); with the Cholesky-only option the d x d solve takes every row.  Either
    way every short row meets the residual gate."""
    from synth import graphs
    p = _problem("local_d128_bf16")
    rng = np.random.Generator(np.random.PCG64(77))
    H0 = 0.05 + 0.002 * rng.standard_normal((p.n_cols, p.d))
    p.H0 = graphs.to_storage_bits(H0, p.storage)
    p.alpha, p.lam = 0.5, 0.01
    ids = _class1_rows(p)
    H0r = p.f64(p.H0)
    G = ials.gramian(H0r)
    assert np.linalg.cond(p.alpha * G + p.lam * np.eye(p.d)) > 1e4
    for kw in (dict(), dict(solver=1)):
        a = make_ctx(p, **kw)
        x32 = a.half_epoch_capture(ROWS, ids).astype(np.float64)
        st = a.get_stats()
        a.destroy()
        assert st.kernel_path[0] == 1 and st.not_spd == 0
        if kw:
            assert st.dual_rows == 0 and st.dual_polished_rows == 0
        else:
            assert st.dual_rows == ids.size and st.dual_polished_rows == ids.size
            # started from the dual solution (rounded to bfloat16), the pass needs a fraction of a solve from scratch
            print(f"polish: {st.dual_polish_products / st.dual_polished_rows:.1f} products per row")
            assert st.dual_polish_products <= 12 * st.dual_polished_rows
        worst = 0.0
        for n in range(0, ids.size, 7):
            A, b = ials.row_system(p.rowptr, p.colidx, None, H0r, G, p.alpha, p.lam, int(ids[n]))
            worst = max(worst, np.linalg.norm(A @ x32[n] - b) / np.linalg.norm(b))
        assert worst <= 1e-4, worst


@pytest.mark.parametrize("name,offset,kmax", [("local_d128_bf16", 0.02, 32), ("zipf_d64_f32", 0.05, 16)])
def test_dual_form_meets_the_residual_gate_close_to_its_condition_limit(name, offset, kmax):
    """||B||_F ||B^-1||_F of about 7300 (d = 128) and 8100 (d = 64), just inside the default limit of 8192 (cond_2(B) about 860
    and 1200): the short rows are solved in the dual form and every one of them meets the residual gate with room to
    spare (the form's error grows with the condition of B, which is what the limit is for)."""
    from synth import graphs
    p = _problem(name)
    rng = np.random.Generator(np.random.PCG64(77))
    H0 = offset + 0.1 / np.sqrt(p.d) * rng.standard_normal((p.n_cols, p.d))
    p.H0 = graphs.to_storage_bits(H0, p.storage)
    p.alpha, p.lam = 0.5, 0.01
    deg = np.diff(p.rowptr)
    ids = np.nonzero((deg > 0) & (deg <= kmax))[0].astype(np.int64)
    a = make_ctx(p)
    x32 = a.half_epoch_capture(ROWS, ids).astype(np.float64)
    st = a.get_stats()
    a.destroy()
    assert st.dual_rows == ids.size and st.not_spd == 0
    H0r = p.f64(p.H0)
    G = ials.gramian(H0r)
    B = p.alpha * G + p.lam * np.eye(p.d)
    fro = np.linalg.norm(B) * np.linalg.norm(np.linalg.inv(B))
    assert 6000 < fro < 8192, fro
    worst = 0.0
    for n in range(ids.size):
        A, b = ials.row_system(p.rowptr, p.colidx, None, H0r, G, p.alpha, p.lam, int(ids[n]))
        worst = max(worst, np.linalg.norm(A @ x32[n] - b) / np.linalg.norm(b))
    print(f"{name}: ||B|| ||B^-1|| = {fro:.0f}, worst residual of {ids.size} dual-form rows {worst:.2e}")
    assert worst <= 5e-5, worst


def _whole_rows(p):
    """rows of 33 .. 1024 observations: the ones the whole-rows tensor-core kernel solves"""
    deg = np.diff(p.rowptr)
    return np.nonzero((deg >= 33) & (deg <= 1024))[0].astype(np.int64)


@pytest.mark.parametrize("name", ["local_d128_bf16", "long_labels_d128_bf16"])
def test_conjugate_gradient_solve_meets_the_gates_and_tracks_the_oracle(name):
    """Sec. 4.5: conjugate gradients (the default solve of the whole-rows tensor-core kernel), started at 0 and
    stopped at |r| <= 3e-5 |b| (the default for bfloat16 tables).  Judged by the residual of the fp32 solution and its distance to the exact row update;
    the number of products is compared with the oracle's textbook iteration (the iterates themselves are unpinned)."""
    p = _problem(name)
    ids = _whole_rows(p)
    assert ids.size > 200
    H0 = p.f64(p.H0)
    G = ials.gramian(H0)
    vals64 = None if p.values is None else p.values.astype(np.float64)
    sols, stats = {}, {}
    # (start at zero, as the oracle's iteration does; the default start, the stored embedding, is covered by every other test)
    for label, kw in (("cg", dict(cg_start=1)), ("chol", dict(solver=1)), ("fallback", dict(cg_max_iter=2, cg_start=1))):
        a = make_ctx(p, **kw)
        sols[label] = a.half_epoch_capture(ROWS, ids).astype(np.float64)
        stats[label] = a.get_stats()
        assert stats[label].not_spd == 0
        a.destroy()
    assert stats["cg"].cg_rows == ids.size and stats["cg"].cg_fallbacks == 0
    assert stats["chol"].cg_rows == 0
    assert stats["fallback"].cg_rows == ids.size and stats["fallback"].cg_fallbacks > 0.9 * ids.size
    _, W_raw = ials.half_step(p.rowptr, p.colidx, vals64, H0, p.alpha, p.lam, p.storage, row_ids=ids, G=G, return_raw=True)
    _, _, o_iters = ials.half_step_cg(p.rowptr, p.colidx, vals64, H0, p.alpha, p.lam, p.storage, row_ids=ids, G=G,
                                     tol=3e-5, max_iter=48)
    # products = steps + 1 (the product of the step at which convergence is seen); fp32 may need a step more or less
    mean_products = stats["cg"].cg_products / stats["cg"].cg_rows
    assert abs(mean_products - (o_iters.mean() + 1)) <= 1.0, (mean_products, o_iters.mean())
    for label in ("cg", "chol", "fallback"):
        assert rel_fro(sols[label], W_raw) <= 1e-4, label
        assert row_rel(sols[label], W_raw).max() <= 1e-3, label
    worst = 0.0
    for n in range(0, ids.size, 3):
        A, b = ials.row_system(p.rowptr, p.colidx, vals64, H0, G, p.alpha, p.lam, int(ids[n]))
        for label in ("cg", "fallback"):
            worst = max(worst, np.linalg.norm(A @ sols[label][n] - b) / np.linalg.norm(b))
    print(f"{name}: worst residual of the conjugate-gradient rows {worst:.2e}, {mean_products:.1f} products per row")
    assert worst <= 1e-4, worst


@pytest.mark.parametrize("name", ["zipf_d64_f32", "split_labels_d64_f32"])
def test_fp32_tables_of_64_features_on_the_tensor_cores(name):
    """d = 64 with fp32 tables: the outer products run on the tensor cores over bfloat16 parts of the fixed table
    (x = x1 + x2 + x3), the 64 x 64 system is folded out of the 128 x 128 sums and solved by conjugate gradients
    (Sec. 4.5) or, on request or when they do not converge, by Cholesky.  Every non-empty row, all three routes and
    the FP32-ALU kernels against the exact row update and the residual gate."""
    p = _problem(name)
    deg = np.diff(p.rowptr)
    ids = np.nonzero(deg > 0)[0].astype(np.int64)
    H0 = p.f64(p.H0)
    G = ials.gramian(H0)
    vals64 = None if p.values is None else p.values.astype(np.float64)
    sols, stats = {}, {}
    # kernels = 2: the 64 x 64 form for every row; kernels = 0 (default): rows of at most 16 observations in the dual form
    for label, kw in (("cg", dict(cg_start=1, kernels=2)), ("chol", dict(solver=1, kernels=2)),
                      ("fallback", dict(cg_max_iter=2, cg_start=1, kernels=2)), ("dual", dict(cg_start=1)),
                      ("alu", dict(kernels=1))):
        a = make_ctx(p, **kw)
        sols[label] = a.half_epoch_capture(ROWS, ids).astype(np.float64)
        stats[label] = a.get_stats()
        assert stats[label].not_spd == 0
        assert stats[label].kernel_path[0] == (0 if label == "alu" else 1)
        a.destroy()
    assert stats["cg"].cg_rows == ids.size and stats["cg"].cg_fallbacks == 0 and stats["cg"].dual_rows == 0
    assert stats["chol"].cg_rows == 0 and stats["alu"].cg_rows == 0
    assert stats["fallback"].cg_rows == ids.size and stats["fallback"].cg_fallbacks > 0.5 * ids.size
    n_short = int(((deg > 0) & (deg <= 16)).sum())
    assert n_short > 500 and stats["dual"].dual_rows == n_short and stats["dual"].cg_rows == ids.size - n_short
    if p.split == 0:
        assert stats["cg"].long_rows[0] > 0      # whole rows of more than 512 observations took the chunks kernel
    _, W_raw = ials.half_step(p.rowptr, p.colidx, vals64, H0, p.alpha, p.lam, p.storage, row_ids=ids, G=G, return_raw=True)
    _, _, o_iters = ials.half_step_cg(p.rowptr, p.colidx, vals64, H0, p.alpha, p.lam, p.storage, row_ids=ids, G=G,
                                     tol=1e-6, max_iter=48)
    mean_products = stats["cg"].cg_products / stats["cg"].cg_rows
    assert abs(mean_products - (o_iters.mean() + 1)) <= 1.0, (mean_products, o_iters.mean())
    nz = np.linalg.norm(W_raw, axis=1) > 0      # (rows whose labels are all 0 have the solution 0)
    for label in sols:
        assert rel_fro(sols[label], W_raw) <= 1e-4, label
        assert row_rel(sols[label][nz], W_raw[nz]).max() <= 1e-3, label
        assert np.all(sols[label][~nz] == 0.0), label
    worst = 0.0
    for n in range(0, ids.size, 5):
        if not nz[n]:
            continue
        A, b = ials.row_system(p.rowptr, p.colidx, vals64, H0, G, p.alpha, p.lam, int(ids[n]))
        for label in ("cg", "chol", "fallback", "dual"):
            worst = max(worst, np.linalg.norm(A @ sols[label][n] - b) / np.linalg.norm(b))
    assert worst <= 1e-4, worst


def test_conjugate_gradients_on_an_ill_conditioned_base_matrix_meet_the_residual_gate():
    """alpha0 G + lambda I with a condition number of about 4e4 (one dominant direction): whichever rows conjugate
    gradients finish within the step limit and whichever go on to the Cholesky launch, every row must meet the
    residual gate."""
    from synth import graphs
    p = _problem("local_d128_bf16")
    rng = np.random.Generator(np.random.PCG64(78))
    H0 = 0.05 + 0.002 * rng.standard_normal((p.n_cols, p.d))
    p.H0 = graphs.to_storage_bits(H0, p.storage)
    p.alpha, p.lam = 0.5, 0.01
    ids = _whole_rows(p)
    a = make_ctx(p)
    x32 = a.half_epoch_capture(ROWS, ids).astype(np.float64)
    st = a.get_stats()
    a.destroy()
    # (the dual form steps aside on this matrix, so the rows of at most 32 observations take the same route)
    assert st.not_spd == 0 and st.cg_rows >= ids.size and 0 <= st.cg_fallbacks <= st.cg_rows
    H0r = p.f64(p.H0)
    G = ials.gramian(H0r)
    worst = 0.0
    for n in range(0, ids.size, 5):
        A, b = ials.row_system(p.rowptr, p.colidx, None, H0r, G, p.alpha, p.lam, int(ids[n]))
        worst = max(worst, np.linalg.norm(A @ x32[n] - b) / np.linalg.norm(b))
    assert worst <= 1e-4, worst


def test_solver_policy_moves_an_expensive_side_to_cholesky():
    """A side whose conjugate-gradient half-epoch spent more products per row than the switch value (28 by default) takes
    Cholesky next time; the choice is made on the device from the counts of the last run.  With the switch at 3 products
    the second rows half-epoch must be Cholesky for every row, meet the gates, and leave the other side alone."""
    p = _problem("local_d128_bf16")
    ids = _whole_rows(p)
    H0 = p.f64(p.H0)
    G = ials.gramian(H0)
    a = make_ctx(p, cg_switch_products=3.0)
    a.half_epoch(ROWS)
    st = a.get_stats()
    assert st.cholesky_by_policy[0] == 0 and st.cg_rows >= ids.size and st.cg_products > 3 * st.cg_rows
    assert st.cg_fallbacks == 0
    a.set_embeddings(COLS, p.H0)
    x32 = a.half_epoch_capture(ROWS, ids).astype(np.float64)
    st = a.get_stats()
    assert st.cholesky_by_policy[0] == 1 and st.cholesky_by_policy[1] == 0 and st.cg_rows == 0 and st.not_spd == 0
    a.destroy()
    _, W_raw = ials.half_step(p.rowptr, p.colidx, None, H0, p.alpha, p.lam, p.storage, row_ids=ids, G=G, return_raw=True)
    assert rel_fro(x32, W_raw) <= 1e-4
    worst = 0.0
    for n in range(0, ids.size, 5):
        A, b = ials.row_system(p.rowptr, p.colidx, None, H0, G, p.alpha, p.lam, int(ids[n]))
        worst = max(worst, np.linalg.norm(A @ x32[n] - b) / np.linalg.norm(b))
    assert worst <= 1e-4, worst
