"""Properties of the seeded input generators (no method arithmetic lives there)."""
import numpy as np
import pytest

from synth import graphs


def check_rows_sorted_unique(rowptr, colidx, n_cols):
    assert colidx.min() >= 0 and colidx.max() < n_cols
    d = np.diff(colidx.astype(np.int64))
    starts = np.zeros(colidx.size, dtype=bool)
    inner = rowptr[1:-1]
    starts[inner[inner < colidx.size]] = True
    assert not np.any((d <= 0) & ~starts[1:])


@pytest.mark.parametrize("law", ["uniform", "zipf", "local"])
def test_rows_strictly_ascending_and_degrees_exact(law):
    n, nnz = 20000, 400000
    deg = graphs.zipf_degrees(n, nnz, 1.1, 5000, 3)
    assert deg.sum() == nnz and deg.min() >= 1 and deg.max() <= 5000
    if law == "uniform":
        spec = graphs.GraphSpec(n, n, 9)
    elif law == "zipf":
        spec = graphs.GraphSpec(n, n, 9, qtable=graphs.zipf_quantile_table(n, 1.1, 3000 / nnz))
    else:
        spec = graphs.GraphSpec(n, n, 9, law=graphs.LAW_LOCAL, delta=200)
    rowptr, colidx = graphs.build_csr(spec, deg)
    assert rowptr[-1] == nnz
    check_rows_sorted_unique(rowptr, colidx, n)
    if law == "local":
        u = np.repeat(np.arange(n), deg)
        small = np.repeat(deg <= 400, deg)
        assert 0.7 < (np.abs(colidx - u) <= 400)[small].mean() <= 1.0
    if law == "zipf":
        indeg = np.bincount(colidx, minlength=n)
        assert indeg[:10].mean() > 50 * np.median(indeg)


def test_single_rows_regenerate_identically():
    n = 5000
    deg = graphs.zipf_degrees(n, 100000, 1.0, 2000, 4)
    for spec in (graphs.GraphSpec(n, n, 5, law=graphs.LAW_LOCAL, delta=100),
                 graphs.GraphSpec(n, n, 5, qtable=graphs.zipf_quantile_table(n, 1.2, 0.01))):
        rowptr, colidx = graphs.build_csr(spec, deg, rows_per_block=777)
        rows = np.array([0, 17, 4999, 2500, int(np.argmax(deg))])
        ptr, cols = graphs.row_columns_flat(spec, rows, deg[rows])
        for k, u in enumerate(rows):
            np.testing.assert_array_equal(cols[ptr[k]:ptr[k + 1]], colidx[rowptr[u]:rowptr[u + 1]])


def test_uniform_cells_exact_count():
    rowptr, colidx = graphs.uniform_cells_csr(2000, 1500, 40000, 1)
    assert rowptr[-1] == 40000 and colidx.size == 40000
    check_rows_sorted_unique(rowptr, colidx, 1500)


def test_embeddings_normal_and_block_consistent():
    full = graphs.init_embeddings(3000, 16, 7, 2, "f32")
    part = graphs.init_embeddings(3000, 16, 7, 2, "f32", row_begin=1000, row_count=50)
    np.testing.assert_array_equal(part, full[1000:1050])
    sigma = 0.1 / 4
    assert abs(full.std() / sigma - 1) < 0.02 and abs(full.mean()) < 3 * sigma / np.sqrt(full.size) * 2
    assert abs((np.abs(full) < sigma).mean() - 0.6827) < 0.01
    b = graphs.init_embeddings(3000, 16, 7, 2, "bf16")
    back = graphs.storage_to_f64(b, "bf16")
    assert np.abs(back - full).max() <= np.abs(full).max() * 2.0 ** -8


def test_planted_links_and_the_evaluation_split():
    """The planted block matrix and the split of the evaluation protocol: seeded (same call, same arrays), rows ascending and
    distinct, most of a row's links inside its group's pool, 10 % test rows taken out of the training matrix, a quarter of
    every test row's links (at least one) held out and the rest kept, nothing lost or invented."""
    from synth import planted
    n, n_cols = 600, 480
    rowptr, colidx = planted.planted_links(n, n_cols, n_groups=12, pool=40, deg_lo=8, deg_hi=20, p_in=0.85, seed=3)
    rowptr2, colidx2 = planted.planted_links(n, n_cols, n_groups=12, pool=40, deg_lo=8, deg_hi=20, p_in=0.85, seed=3)
    np.testing.assert_array_equal(rowptr, rowptr2)
    np.testing.assert_array_equal(colidx, colidx2)
    deg = np.diff(rowptr)
    assert deg.min() >= 7 and deg.max() <= 20 and colidx.min() >= 0 and colidx.max() < n_cols
    for u in range(n):
        c = colidx[rowptr[u]:rowptr[u + 1]]
        assert np.all(np.diff(c) > 0)
    # rows of one group share a pool: two rows of the same group overlap far more than rows of different groups
    sets = [set(colidx[rowptr[u]:rowptr[u + 1]].tolist()) for u in range(48)]
    same = np.mean([len(sets[u] & sets[u + 12]) for u in range(24)])
    other = np.mean([len(sets[u] & sets[u + 1]) for u in range(24)])
    assert same > 3 * max(other, 0.1)
    sp = planted.split_rows(rowptr, colidx, 0.10, 0.25, seed=4)
    test_rows = sp["test_rows"]
    assert test_rows.size == 60
    tr_ptr, tr_idx = sp["train"]
    assert np.all(np.diff(tr_ptr)[test_rows] == 0)
    kept_ptr, kept_idx = sp["kept"]
    truth_ptr, truth_idx = sp["truth"]
    for j, u in enumerate(test_rows):
        kept = kept_idx[kept_ptr[j]:kept_ptr[j + 1]]
        truth = truth_idx[truth_ptr[j]:truth_ptr[j + 1]]
        full = colidx[rowptr[u]:rowptr[u + 1]]
        assert truth.size == max(1, int(round(0.25 * full.size)))
        np.testing.assert_array_equal(np.sort(np.concatenate([kept, truth])), full)
        assert np.all(np.diff(kept) > 0) and np.all(np.diff(truth) > 0)
    train_rows = np.setdiff1d(np.arange(n), test_rows)
    assert int(np.diff(tr_ptr)[train_rows].sum()) == int(deg[train_rows].sum()) == tr_idx.size
