"""Thin Python binding of the C ABI in ``include/alx.h``: argument marshalling only.

Every step of the method runs inside ``libalx_b200.so``.  PyTorch is used here for device memory
(the context's allocator callbacks hand out ``torch.empty`` buffers) and for the CUDA stream.
Importing this module needs the built library; there is no fallback of any kind.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import (CFUNCTYPE, POINTER, Structure, byref, c_char_p, c_double, c_float, c_int, c_int32, c_int64,
                    c_size_t, c_void_p)

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libalx_b200.so")

ALX_OK = 0
ALX_ROWS, ALX_COLS = 0, 1
ALX_F32, ALX_BF16 = 0, 1
ALX_N_CLASSES = 12
ALX_DEFAULT_SPLIT = 8192
STATUS_NAMES = ["ALX_OK", "ALX_ERR_INVALID_ARG", "ALX_ERR_BAD_STATE", "ALX_ERR_OOM", "ALX_ERR_CUDA",
                "ALX_ERR_BAD_CSR", "ALX_ERR_NOT_SPD", "ALX_ERR_UNSUPPORTED"]

ALLOC_FN = CFUNCTYPE(c_void_p, c_size_t, c_void_p)
FREE_FN = CFUNCTYPE(None, c_void_p, c_void_p)


class alx_options(Structure):
    _fields_ = [("n_rows", c_int64), ("n_cols", c_int64), ("d", c_int32), ("lambda_", c_float),
                ("alpha0", c_float), ("storage", c_int32), ("device", c_int32), ("stream", c_void_p),
                ("alloc", ALLOC_FN), ("free", FREE_FN), ("alloc_user", c_void_p), ("split", c_int64),
                ("kernels", c_int32), ("solver", c_int32), ("cg_max_iter", c_int32), ("cg_tol", c_float),
                ("cg_switch_products", c_float), ("cg_start", c_int32), ("dual_cond_limit", c_float)]


class alx_stats(Structure):
    _fields_ = [("nnz", c_int64), ("rows_in_class", (c_int64 * ALX_N_CLASSES) * 2), ("n_chunks", c_int64 * 2),
                ("not_spd", c_int64), ("ms_gramian", c_double), ("ms_rows", c_double),
                ("ms_half_epoch", c_double), ("kernel_launches", c_int64), ("workspace_bytes", c_int64),
                ("kernel_path", c_int32 * 2), ("ms_main_kernel", c_double), ("dual_rows", c_int64),
                ("long_rows", c_int64 * 2), ("long_entries", c_int64 * 2), ("cg_rows", c_int64),
                ("cg_products", c_int64), ("cg_fallbacks", c_int64), ("cholesky_by_policy", c_int32 * 2),
                ("dual_polished_rows", c_int64), ("dual_polish_products", c_int64),
                ("entries_in_class", (c_int64 * ALX_N_CLASSES) * 2)]


EXPORTS = ["alx_create", "alx_create_ex", "alx_destroy", "alx_set_csr", "alx_set_embeddings", "alx_set_embedding_rows",
           "alx_half_epoch", "alx_load_host", "alx_epoch_to_host",
           "alx_epoch", "alx_half_epoch_capture", "alx_loss", "alx_get_embeddings", "alx_get_gramian",
           "alx_gramian", "alx_fp32_peak_tflops", "alx_get_transpose", "alx_get_buckets", "alx_get_stats", "alx_synchronize",
           "alx_last_error", "alx_version", "alx_gramian_noalloc", "alx_gramian_noalloc_max_rows",
           "alx_noalloc_last_error", "alx_fold_in", "alx_topk", "alx_recall_at_k"]

_lib = None


def load_library() -> ctypes.CDLL:
    """Load libalx_b200.so (built in-tree by ``build.py``); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} not found: run `python -m paper_2112_02194_b200.build` first "
                          "(there is no CPU or library fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    P = c_void_p
    lib.alx_create.argtypes = [c_int64, c_int64, c_int32, c_float, c_float, POINTER(P)]
    lib.alx_create_ex.argtypes = [POINTER(alx_options), POINTER(P)]
    lib.alx_destroy.argtypes = [P]
    lib.alx_set_csr.argtypes = [P, P, P, P, c_int64, c_int]
    lib.alx_set_embeddings.argtypes = [P, c_int, P, c_int, c_int]
    lib.alx_set_embedding_rows.argtypes = [P, c_int, c_int64, c_int64, P, c_int, c_int]
    lib.alx_half_epoch.argtypes = [P, c_int]
    lib.alx_epoch.argtypes = [P]
    lib.alx_load_host.argtypes = [P, P, P, P, c_int64, P, P]
    lib.alx_epoch_to_host.argtypes = [P, P, P]
    lib.alx_half_epoch_capture.argtypes = [P, c_int, P, c_int64, P]
    lib.alx_loss.argtypes = [P, POINTER(c_double), POINTER(c_double)]
    lib.alx_get_embeddings.argtypes = [P, c_int, P, c_int, c_int64, c_int64, c_int]
    lib.alx_get_gramian.argtypes = [P, c_int, P]
    lib.alx_gramian.argtypes = [P, c_int, P]
    lib.alx_get_transpose.argtypes = [P, P, P, P]
    lib.alx_get_buckets.argtypes = [P, c_int, P, P, P, POINTER(c_int64)]
    lib.alx_get_stats.argtypes = [P, POINTER(alx_stats)]
    lib.alx_synchronize.argtypes = [P]
    lib.alx_fold_in.argtypes = [P, P, P, P, c_int64, c_int64, c_int, P]
    lib.alx_topk.argtypes = [P, c_int, P, c_int64, c_int32, P, P, c_int, P, P]
    lib.alx_recall_at_k.argtypes = [P, P, c_int64, c_int32, c_int32, P, P, c_int, POINTER(c_double), POINTER(c_int64)]
    lib.alx_fp32_peak_tflops.argtypes = [P, POINTER(c_double)]
    lib.alx_last_error.argtypes = [P]
    lib.alx_last_error.restype = c_char_p
    lib.alx_version.restype = c_char_p
    lib.alx_gramian_noalloc.argtypes = [P, c_int, c_int64, c_int32, P, P]
    lib.alx_gramian_noalloc_max_rows.argtypes = [c_int32]
    lib.alx_gramian_noalloc_max_rows.restype = c_int64
    lib.alx_noalloc_last_error.restype = c_char_p
    for name in EXPORTS:
        if name not in ("alx_last_error", "alx_version", "alx_gramian_noalloc_max_rows", "alx_noalloc_last_error"):
            getattr(lib, name).restype = c_int
    _lib = lib
    return lib


class AlxError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else status}: {message}")
        self.status = status


def _np_ptr(a):
    return None if a is None else a.ctypes.data_as(c_void_p)


class Alx:
    """One context.  Methods carry the C names without the ``alx_`` prefix and only marshal arguments."""

    def __init__(self, n_rows, n_cols, d, lam, alpha0, storage="f32", split=0, kernels=0, device=None,
                 use_torch_allocator=True, solver=0, cg_max_iter=0, cg_tol=0.0, cg_start=0, cg_switch_products=0.0,
                 dual_cond_limit=0.0):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("alx needs a CUDA device (B200, sm_100a); there is no CPU path")
        self.lib = load_library()
        self.torch = torch
        self.n_rows, self.n_cols, self.d = int(n_rows), int(n_cols), int(d)
        self.storage = storage
        self.device = torch.cuda.current_device() if device is None else int(device)
        self._buffers = {}
        opt = alx_options()
        opt.n_rows, opt.n_cols, opt.d = self.n_rows, self.n_cols, self.d
        opt.lambda_, opt.alpha0 = lam, alpha0
        opt.storage = ALX_BF16 if storage == "bf16" else ALX_F32
        opt.device = self.device
        opt.stream = torch.cuda.current_stream(self.device).cuda_stream
        opt.split = split
        opt.kernels = kernels
        opt.solver, opt.cg_max_iter, opt.cg_tol = int(solver), int(cg_max_iter), float(cg_tol)
        opt.cg_start = int(cg_start)
        opt.dual_cond_limit = float(dual_cond_limit)
        opt.cg_switch_products = float(cg_switch_products)
        if use_torch_allocator:
            dev = torch.device("cuda", self.device)

            def _alloc(nbytes, _user):
                try:
                    t = torch.empty(int(nbytes), dtype=torch.uint8, device=dev)
                except Exception:
                    return None
                self._buffers[t.data_ptr()] = t
                return t.data_ptr()

            def _free(ptr, _user):
                self._buffers.pop(ptr, None)

            self._alloc_cb, self._free_cb = ALLOC_FN(_alloc), FREE_FN(_free)
            opt.alloc, opt.free = self._alloc_cb, self._free_cb
        self._opt = opt
        self.ctx = c_void_p()
        st = self.lib.alx_create_ex(byref(opt), byref(self.ctx))
        if st != ALX_OK:
            raise AlxError(st, "alx_create_ex failed")

    # -- helpers
    def _check(self, st):
        if st != ALX_OK:
            raise AlxError(st, self.lib.alx_last_error(self.ctx).decode())

    def _n(self, side):
        return self.n_rows if side == ALX_ROWS else self.n_cols

    def destroy(self):
        if getattr(self, "ctx", None) is not None and self.ctx:
            self.lib.alx_destroy(self.ctx)
            self.ctx = None
            self._buffers.clear()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    # -- the ABI
    def set_csr(self, rowptr, colidx, values=None):
        """numpy arrays (host) or torch CUDA tensors (device): int64 rowptr, int32 colidx, float32 values."""
        torch = self.torch
        if isinstance(rowptr, torch.Tensor):
            assert rowptr.dtype == torch.int64 and colidx.dtype == torch.int32 and rowptr.is_cuda and colidx.is_cuda
            assert rowptr.is_contiguous() and colidx.is_contiguous()
            v = None
            if values is not None:
                assert values.dtype == torch.float32 and values.is_cuda and values.is_contiguous()
                v = values.data_ptr()
            self._check(self.lib.alx_set_csr(self.ctx, rowptr.data_ptr(), colidx.data_ptr(), v,
                                             int(colidx.numel()), 1))
        else:
            rowptr = np.ascontiguousarray(rowptr, dtype=np.int64)
            colidx = np.ascontiguousarray(colidx, dtype=np.int32)
            v = None if values is None else np.ascontiguousarray(values, dtype=np.float32)
            self._check(self.lib.alx_set_csr(self.ctx, _np_ptr(rowptr), _np_ptr(colidx), _np_ptr(v),
                                             int(colidx.size), 0))

    def set_embeddings(self, side, src, dtype=None):
        """src: numpy float32 / uint16 (bf16 bit patterns) array, or a torch CUDA tensor (float32 / bfloat16)."""
        torch = self.torch
        if isinstance(src, torch.Tensor):
            assert src.is_cuda and src.is_contiguous() and src.numel() == self._n(side) * self.d
            dt = ALX_BF16 if src.dtype == torch.bfloat16 else ALX_F32
            assert src.dtype in (torch.bfloat16, torch.float32)
            self._check(self.lib.alx_set_embeddings(self.ctx, side, src.data_ptr(), dt, 1))
        else:
            src = np.ascontiguousarray(src)
            assert src.size == self._n(side) * self.d
            if src.dtype == np.uint16:
                dt = ALX_BF16
            else:
                src = np.ascontiguousarray(src, dtype=np.float32)
                dt = ALX_F32
            self._check(self.lib.alx_set_embeddings(self.ctx, side, _np_ptr(src), dt, 0))

    def set_embedding_rows(self, side, row_begin, src):
        """Rows row_begin .. of one table from a torch CUDA tensor (float32 / bfloat16) or a numpy array
        (float32 / uint16 bf16 bit patterns) holding whole rows."""
        torch = self.torch
        if isinstance(src, torch.Tensor):
            assert src.is_cuda and src.is_contiguous() and src.numel() % self.d == 0
            assert src.dtype in (torch.bfloat16, torch.float32)
            dt = ALX_BF16 if src.dtype == torch.bfloat16 else ALX_F32
            self._check(self.lib.alx_set_embedding_rows(self.ctx, side, row_begin, src.numel() // self.d, src.data_ptr(), dt, 1))
        else:
            src = np.ascontiguousarray(src)
            assert src.size % self.d == 0
            if src.dtype == np.uint16:
                dt = ALX_BF16
            else:
                src = np.ascontiguousarray(src, dtype=np.float32)
                dt = ALX_F32
            self._check(self.lib.alx_set_embedding_rows(self.ctx, side, row_begin, src.size // self.d, _np_ptr(src), dt, 0))

    def half_epoch(self, side):
        self._check(self.lib.alx_half_epoch(self.ctx, side))

    def epoch(self):
        self._check(self.lib.alx_epoch(self.ctx))

    def load_host(self, rowptr, colidx, values, W, H):
        """set_csr + set_embeddings of both tables from host numpy arrays (tables in the storage type: float32, or
        uint16 bf16 bit patterns), with the table uploads overlapped with the set-up kernels."""
        import numpy as np
        rowptr = np.ascontiguousarray(rowptr, dtype=np.int64)
        colidx = np.ascontiguousarray(colidx, dtype=np.int32)
        vals = None if values is None else np.ascontiguousarray(values, dtype=np.float32)
        want = np.uint16 if self.storage == "bf16" else np.float32
        assert W.dtype == want and H.dtype == want and W.flags.c_contiguous and H.flags.c_contiguous
        self._check(self.lib.alx_load_host(self.ctx, rowptr.ctypes.data, colidx.ctypes.data,
                                           None if vals is None else vals.ctypes.data, colidx.size,
                                           W.ctypes.data, H.ctypes.data))

    def epoch_to_host(self, W_out, H_out):
        """epoch + download of both tables into host numpy arrays of the storage type; W is read back during the
        column pass."""
        import numpy as np
        want = np.uint16 if self.storage == "bf16" else np.float32
        assert W_out.dtype == want and H_out.dtype == want and W_out.flags.c_contiguous and H_out.flags.c_contiguous
        self._check(self.lib.alx_epoch_to_host(self.ctx, W_out.ctypes.data, H_out.ctypes.data))

    def half_epoch_capture(self, side, row_ids):
        ids = np.ascontiguousarray(row_ids, dtype=np.int64)
        out = np.empty((ids.size, self.d), dtype=np.float32)
        self._check(self.lib.alx_half_epoch_capture(self.ctx, side, _np_ptr(ids), int(ids.size), _np_ptr(out)))
        return out

    # ---- evaluation (host arrays in, host arrays out)
    def fold_in(self, rowptr, colidx, values=None):
        """Embeddings (float32, after the round to the storage type) of new rows given as CSR over the columns."""
        rp = np.ascontiguousarray(rowptr, dtype=np.int64)
        ci = np.ascontiguousarray(colidx, dtype=np.int32)
        va = None if values is None else np.ascontiguousarray(values, dtype=np.float32)
        n_new = rp.size - 1
        out = np.empty((n_new, self.d), dtype=np.float32)
        self._check(self.lib.alx_fold_in(self.ctx, _np_ptr(rp), _np_ptr(ci), None if va is None else _np_ptr(va), n_new,
                                         int(ci.size), 0, _np_ptr(out)))
        return out

    def topk(self, items_side, queries, k, exclude=None, scores=True):
        """(ids [m, k] int32, scores [m, k] float32 or None); exclude = (ptr, idx) CSR of ids to leave out per query."""
        q = np.ascontiguousarray(queries, dtype=np.float32)
        m = q.shape[0]
        ids = np.empty((m, k), dtype=np.int32)
        sc = np.empty((m, k), dtype=np.float32) if scores else None
        ep = ei = None
        if exclude is not None:
            ep = np.ascontiguousarray(exclude[0], dtype=np.int64)
            ei = np.ascontiguousarray(exclude[1], dtype=np.int32)
            if ei.size == 0:
                ei = np.zeros(1, dtype=np.int32)
        self._check(self.lib.alx_topk(self.ctx, items_side, _np_ptr(q), m, k, None if ep is None else _np_ptr(ep),
                                      None if ei is None else _np_ptr(ei), 0, _np_ptr(ids), None if sc is None else _np_ptr(sc)))
        return ids, sc

    def topk_device(self, items_side, queries, k, ids_out, scores_out=None):
        """Top-K with torch CUDA tensors: queries [m, d] float32, ids_out [m, k] int32, scores_out [m, k] float32."""
        assert queries.is_cuda and queries.is_contiguous() and queries.dtype == self.torch.float32
        assert ids_out.is_cuda and ids_out.is_contiguous() and ids_out.dtype == self.torch.int32
        m = queries.shape[0]
        self._check(self.lib.alx_topk(self.ctx, items_side, queries.data_ptr(), m, k, None, None, 1, ids_out.data_ptr(),
                                      None if scores_out is None else scores_out.data_ptr()))

    def recall_at_k(self, ids, k, truth_ptr, truth_idx):
        """(mean recall over the queries with ground truth, how many those are)"""
        a = np.ascontiguousarray(ids, dtype=np.int32)
        tp = np.ascontiguousarray(truth_ptr, dtype=np.int64)
        ti = np.ascontiguousarray(truth_idx, dtype=np.int32)
        if ti.size == 0:
            ti = np.zeros(1, dtype=np.int32)
        r, n = c_double(), c_int64()
        self._check(self.lib.alx_recall_at_k(self.ctx, _np_ptr(a), a.shape[0], a.shape[1], k, _np_ptr(tp), _np_ptr(ti), 0,
                                             byref(r), byref(n)))
        return r.value, n.value

    def loss(self):
        total = c_double()
        comp = (c_double * 3)()
        self._check(self.lib.alx_loss(self.ctx, byref(total), comp))
        return total.value, (comp[0], comp[1], comp[2])

    def get_embeddings(self, side, dtype="f32", row_begin=0, row_count=None, out=None):
        """Host copy as numpy (float32, or uint16 bf16 bits); or into a torch CUDA tensor given as ``out``."""
        if row_count is None:
            row_count = self._n(side) - row_begin
        if out is not None:
            dt = ALX_BF16 if out.dtype == self.torch.bfloat16 else ALX_F32
            assert out.is_cuda and out.is_contiguous() and out.numel() == row_count * self.d
            self._check(self.lib.alx_get_embeddings(self.ctx, side, out.data_ptr(), dt, row_begin, row_count, 1))
            return out
        arr = np.empty((row_count, self.d), dtype=np.uint16 if dtype == "bf16" else np.float32)
        self._check(self.lib.alx_get_embeddings(self.ctx, side, _np_ptr(arr), ALX_BF16 if dtype == "bf16" else ALX_F32,
                                                row_begin, row_count, 0))
        return arr

    def gramian(self, table_side):
        g = np.empty((self.d, self.d), dtype=np.float64)
        self._check(self.lib.alx_gramian(self.ctx, table_side, _np_ptr(g)))
        return g

    def get_gramian(self, table_side):
        g = np.empty((self.d, self.d), dtype=np.float64)
        self._check(self.lib.alx_get_gramian(self.ctx, table_side, _np_ptr(g)))
        return g

    def get_transpose(self, nnz, with_values=False):
        colptr = np.empty(self.n_cols + 1, dtype=np.int64)
        rowidx = np.empty(nnz, dtype=np.int32)
        vt = np.empty(nnz, dtype=np.float32) if with_values else None
        self._check(self.lib.alx_get_transpose(self.ctx, _np_ptr(colptr), _np_ptr(rowidx), _np_ptr(vt)))
        return colptr, rowidx, vt

    def get_buckets(self, side):
        n = self._n(side)
        order = np.empty(n, dtype=np.int32)
        offs = np.empty(ALX_N_CLASSES + 1, dtype=np.int64)
        nch = c_int64()
        self._check(self.lib.alx_get_buckets(self.ctx, side, None, None, None, byref(nch)))
        desc = np.empty((nch.value, 4), dtype=np.int64)
        self._check(self.lib.alx_get_buckets(self.ctx, side, _np_ptr(order), _np_ptr(offs), _np_ptr(desc), byref(nch)))
        return order, offs, desc

    def get_stats(self):
        s = alx_stats()
        self._check(self.lib.alx_get_stats(self.ctx, byref(s)))
        return s

    def fp32_peak_tflops(self):
        v = c_double()
        self._check(self.lib.alx_fp32_peak_tflops(self.ctx, byref(v)))
        return v.value

    def synchronize(self):
        self._check(self.lib.alx_synchronize(self.ctx))


def gramian_noalloc(table, out):
    """``alx_gramian_noalloc``: table^T table of a CUDA tensor (n x d, float32 or bfloat16) into ``out``
    (a d x d float64 CUDA tensor the caller owns), on the current stream, without any allocation by the
    library.  For callers that may not allocate at call time; see include/alx.h for the limits."""
    import torch
    lib = load_library()
    assert table.is_cuda and table.is_contiguous() and table.dim() == 2
    if table.dtype not in (torch.bfloat16, torch.float32):     # any other element size would make the kernel read past the buffer
        raise TypeError(f"gramian_noalloc: table must be float32 or bfloat16, not {table.dtype}")
    assert out.is_cuda and out.is_contiguous() and out.dtype == torch.float64 and out.numel() == table.shape[1] ** 2
    dt = ALX_BF16 if table.dtype == torch.bfloat16 else ALX_F32
    st = lib.alx_gramian_noalloc(table.data_ptr(), dt, table.shape[0], table.shape[1], out.data_ptr(),
                                 torch.cuda.current_stream().cuda_stream)
    if st != ALX_OK:
        raise AlxError(st, lib.alx_noalloc_last_error().decode())
    return out


def gramian_noalloc_max_rows(d: int) -> int:
    return int(load_library().alx_gramian_noalloc_max_rows(d))
