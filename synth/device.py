"""Device-side front end of the input generators (``synth/csrc/synth.cu``): same bits as ``graphs.py``.

Used where a graph is too large to build on the host (the 1-billion-entry benchmark workload).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

from . import graphs

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "csrc", "synth.cu")
_LIB = os.path.join(_HERE, "libalx_synth.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
                               "-Xcompiler", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lcudart_static"])
    return _LIB


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB):
            raise ImportError(f"{_LIB} not found: build it first (synth.device.build())")
        _lib = ctypes.CDLL(_LIB)
        _lib.synth_edges.restype = ctypes.c_int
        _lib.synth_normal.restype = ctypes.c_int
    return _lib


def device_csr(spec: graphs.GraphSpec, deg: np.ndarray):
    """(rowptr int64 CUDA tensor [n+1], colidx int32 CUDA tensor [nnz]) of the whole graph."""
    import torch
    dev = torch.device("cuda")
    degt = torch.from_numpy(np.ascontiguousarray(deg, dtype=np.int64)).to(dev)
    rowptr = torch.zeros(spec.n_rows + 1, dtype=torch.int64, device=dev)
    torch.cumsum(degt, 0, out=rowptr[1:])
    del degt
    nnz = int(rowptr[-1].item())
    colidx = torch.empty(nnz, dtype=torch.int32, device=dev)
    qt = torch.from_numpy(spec.qtable.astype(np.int64)).to(dev)
    key = int(graphs.stream_key(spec.seed, 1))
    err = lib().synth_edges(ctypes.c_int(spec.law), ctypes.c_longlong(spec.n_rows), ctypes.c_longlong(spec.n_cols),
                            ctypes.c_ulonglong(key), ctypes.c_void_p(qt.data_ptr()), ctypes.c_longlong(spec.delta),
                            ctypes.c_longlong(spec.local_num), ctypes.c_longlong(spec.local_den),
                            ctypes.c_void_p(rowptr.data_ptr()), ctypes.c_longlong(nnz),
                            ctypes.c_void_p(colidx.data_ptr()),
                            ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
    if err:
        raise RuntimeError(f"synth_edges: CUDA error {err}")
    torch.cuda.synchronize()
    return rowptr, colidx


def device_embeddings(n: int, d: int, seed: int, stream: int, storage: str, sigma: float | None = None, row_begin: int = 0):
    """n x d CUDA tensor (float32 or bfloat16) with the same bits as rows row_begin .. row_begin + n - 1 of
    graphs.init_embeddings."""
    import torch
    if sigma is None:
        sigma = 0.1 / np.sqrt(d)
    dev = torch.device("cuda")
    table = torch.from_numpy(graphs.normal_table()).to(dev)
    out = torch.empty((n, d), dtype=torch.bfloat16 if storage == "bf16" else torch.float32, device=dev)
    key = int(graphs.stream_key(seed, stream))
    scale = float(sigma / 2.0 ** graphs.NT_SCALE_BITS)
    err = lib().synth_normal(ctypes.c_ulonglong(key), ctypes.c_void_p(table.data_ptr()), ctypes.c_longlong(row_begin * d),
                             ctypes.c_longlong(n * d), ctypes.c_double(scale), ctypes.c_int(storage == "bf16"),
                             ctypes.c_void_p(out.data_ptr()),
                             ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
    if err:
        raise RuntimeError(f"synth_normal: CUDA error {err}")
    torch.cuda.synchronize()
    return out
