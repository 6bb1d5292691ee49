"""Seeded test problems shared by the parity tests: scaled-down versions of the benchmark configurations."""
from dataclasses import dataclass

import numpy as np

from synth import graphs


@dataclass
class Problem:
    name: str
    n_rows: int
    n_cols: int
    d: int
    lam: float
    alpha: float
    storage: str          # "f32" or "bf16"
    rowptr: np.ndarray
    colidx: np.ndarray
    values: np.ndarray | None
    W0: np.ndarray        # storage bit layout (float32 or uint16)
    H0: np.ndarray
    split: int = 0

    @property
    def nnz(self):
        return int(self.rowptr[-1])

    def f64(self, table):
        return graphs.storage_to_f64(table, self.storage)

    @property
    def emb_tol(self):
        return 1e-3 if self.storage == "f32" else 2e-2


def _tables(n_rows, n_cols, d, seed, storage):
    return (graphs.init_embeddings(n_rows, d, seed, 2, storage), graphs.init_embeddings(n_cols, d, seed, 3, storage))


def tiny():
    """Configuration 1 of the benchmark list: 2000 x 1500, 40 000 uniform cells, d = 16, fp32."""
    rowptr, colidx = graphs.uniform_cells_csr(2000, 1500, 40000, 0xA1C50001)
    W0, H0 = _tables(2000, 1500, 16, 0x1A150001, "f32")
    return Problem("tiny", 2000, 1500, 16, 0.1, 0.01, "f32", rowptr, colidx, None, W0, H0)


def powerlaw(name, n, nnz, s, cap, d, lam, alpha, storage, law, seed, split=0, values=False, n_cols=None,
             empty_rows=0, zero_labels=0.0):
    n_cols = n if n_cols is None else n_cols
    deg = graphs.zipf_degrees(n, nnz, s, min(cap, n_cols // 2), seed)
    if empty_rows:
        deg[np.arange(empty_rows) * 37 % n] = 0
    if law == "local":
        spec = graphs.GraphSpec(n, n_cols, seed + 1, law=graphs.LAW_LOCAL, delta=max(n_cols // 100, 8))
    elif law == "zipf":
        spec = graphs.GraphSpec(n, n_cols, seed + 1, qtable=graphs.zipf_quantile_table(n_cols, s, cap / nnz))
    else:
        spec = graphs.GraphSpec(n, n_cols, seed + 1)
    rowptr, colidx = graphs.build_csr(spec, deg)
    vals = None
    if values:
        rng = np.random.Generator(np.random.PCG64(seed + 2))
        vals = rng.uniform(0.5, 2.0, colidx.size).astype(np.float32)
        if zero_labels:       # y = 0 is a legal observation: it adds x (x) x to the row's matrix and nothing to its right-hand side
            vals[rng.random(colidx.size) < zero_labels] = 0.0
            for u in (5, 17, 33):       # and a few rows whose every label is 0
                vals[rowptr[u]:rowptr[u + 1]] = 0.0
    W0, H0 = _tables(n, n_cols, d, seed + 3, storage)
    return Problem(name, n, n_cols, d, lam, alpha, storage, rowptr, colidx, vals, W0, H0, split)


def small_suite():
    """Problems the oracle finishes in seconds; together they span every degree class, both storage types,
    every supported d, labelled entries (on both kernel paths), empty rows, alpha0 = 0 and rows longer than the split
    threshold."""
    return [
        tiny,
        lambda: powerlaw("zipf_d64_f32", 6000, 180000, 1.2, 3000, 64, 0.05, 0.001, "f32", "zipf", 11, empty_rows=5),
        lambda: powerlaw("local_d128_bf16", 5000, 200000, 1.1, 2400, 128, 0.01, 0.001, "bf16", "local", 12,
                         empty_rows=3),
        lambda: powerlaw("split_d128_bf16", 3000, 150000, 0.9, 1400, 128, 0.01, 0.0005, "bf16", "zipf", 13, split=256),
        lambda: powerlaw("split_d32_f32_labels", 2500, 60000, 1.0, 1000, 32, 0.05, 0.01, "f32", "uniform", 14,
                         split=128, values=True, n_cols=2100),
        lambda: powerlaw("alpha0_d16_bf16", 1500, 30000, 1.0, 600, 16, 0.1, 0.0, "bf16", "uniform", 15, n_cols=1300),
        lambda: powerlaw("default_split_d64_bf16", 1200, 120000, 1.3, 9500, 64, 0.02, 0.001, "bf16", "uniform", 16,
                         n_cols=20000),
        # labelled entries on the tensor-core path: whole rows of more than 1024 observations (their sums come from the
        # chunks kernel), and the same matrix with rows split at 512
        lambda: powerlaw("long_labels_d128_bf16", 1500, 120000, 1.0, 3000, 128, 0.02, 0.001, "bf16", "zipf", 17,
                         values=True, n_cols=8000),
        lambda: powerlaw("split_labels_d128_bf16", 1500, 120000, 1.0, 3000, 128, 0.02, 0.001, "bf16", "zipf", 17,
                         split=512, values=True, n_cols=8000),
        # the remaining (d, storage) pairs: d = 128 with fp32 tables, labels of which a fifth are 0 (some rows hold nothing
        # but zeros: their right-hand side is 0 and so is their solution); d = 32 with bfloat16 tables
        lambda: powerlaw("zero_labels_d128_f32", 1200, 40000, 1.0, 700, 128, 0.02, 0.001, "f32", "zipf", 18,
                         split=256, values=True, n_cols=2500, zero_labels=0.2),
        lambda: powerlaw("uniform_d32_bf16", 2000, 50000, 1.1, 900, 32, 0.05, 0.002, "bf16", "uniform", 19, n_cols=1700,
                         empty_rows=2),
        # fp32 tables of 64 features on the tensor cores (bfloat16 parts, doubled entry lists): labelled entries, rows
        # split at 256 observations, whole rows of more than 512 (their sums come from the chunks kernel)
        lambda: powerlaw("split_labels_d64_f32", 2000, 90000, 1.0, 2500, 64, 0.05, 0.002, "f32", "zipf", 21, split=512,
                         values=True, n_cols=3000, zero_labels=0.1, empty_rows=2),
    ]
