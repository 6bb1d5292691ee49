"""Fast host-side front end of the embedding generator (``synth/csrc/synth_host.c``): same bits as
``graphs.init_embeddings`` / ``graphs.init_embedding_rows``, OpenMP instead of numpy."""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

from . import graphs

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "csrc", "synth_host.c")
_LIB = os.path.join(_HERE, "libalx_synth_host.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", _LIB, _SRC])
    return _LIB


def _get():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def embedding_rows(d: int, seed: int, stream: int, storage: str, rows=None, row_begin: int = 0,
                   row_count: int = 0, sigma: float | None = None, as_f64: bool = False) -> np.ndarray:
    """Rows of the table ``graphs.init_embeddings(n, d, seed, stream, storage)``: either the ids in ``rows`` or the
    block row_begin .. row_begin + row_count - 1.  float32 or uint16 (bf16 bits); with ``as_f64`` the stored values
    widened to float64 (the same as ``graphs.storage_to_f64`` of the bits, without the detour)."""
    if sigma is None:
        sigma = 0.1 / np.sqrt(d)
    table = np.ascontiguousarray(graphs.normal_table(), dtype=np.int64)
    key = int(graphs.stream_key(seed, stream))
    scale = float(sigma / 2.0 ** graphs.NT_SCALE_BITS)
    if rows is not None:
        rows = np.ascontiguousarray(rows, dtype=np.int64)
        n = rows.size
        rp = rows.ctypes.data_as(ctypes.c_void_p)
    else:
        n = int(row_count)
        rp = None
    out = np.empty((n, d), dtype=np.float64 if as_f64 else (np.uint16 if storage == "bf16" else np.float32))
    _get().synth_host_rows(ctypes.c_uint64(key), table.ctypes.data_as(ctypes.c_void_p), rp, ctypes.c_int64(row_begin),
                           ctypes.c_int64(n), ctypes.c_int(d), ctypes.c_double(scale), ctypes.c_int(storage == "bf16"),
                           ctypes.c_int(1 if as_f64 else 0), out.ctypes.data_as(ctypes.c_void_p))
    return out
