"""The C-ABI library loads and exports every symbol the public header declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in os.listdir(inc):
        if f.endswith(".h"):
            text = open(os.path.join(inc, f)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(alx_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


def test_header_declares_the_required_entry_points():
    names = declared_symbols()
    for required in ["alx_create", "alx_set_csr", "alx_half_epoch", "alx_epoch", "alx_loss", "alx_get_embeddings"]:
        assert required in names


def test_library_exports_every_declared_symbol():
    from paper_2112_02194_b200 import build as b
    lib = ctypes.CDLL(b.build())
    for name in declared_symbols():
        assert hasattr(lib, name), name
    from paper_2112_02194_b200 import binding
    assert sorted(set(binding.EXPORTS)) == [n for n in declared_symbols()]
    assert b"sm_100a" in binding.load_library().alx_version()


def test_binding_refuses_to_run_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_2112_02194_b200 import Alx
    with pytest.raises(RuntimeError):
        Alx(10, 10, 16, 0.1, 0.01)


def test_synth_library_builds():
    from synth import device
    lib = ctypes.CDLL(device.build())
    assert hasattr(lib, "synth_edges") and hasattr(lib, "synth_normal")


def test_noalloc_gramian_refuses_bad_pointers_without_a_gpu():
    """The argument checks of alx_gramian_noalloc come before any CUDA call: misaligned or null pointers, unknown
    sizes and types are refused with a status code on a machine without a GPU too (nothing is ever dereferenced)."""
    import ctypes
    from paper_2112_02194_b200 import binding
    lib = binding.load_library()
    buf = ctypes.create_string_buffer(4096)
    base = (ctypes.addressof(buf) + 255) & ~255
    assert lib.alx_gramian_noalloc(None, 0, 16, 128, base, None) == 1
    assert lib.alx_gramian_noalloc(base, 7, 16, 128, base, None) == 1                     # unknown dtype
    assert lib.alx_gramian_noalloc(base, 0, 16, 48, base, None) == 7                      # unsupported d
    assert lib.alx_gramian_noalloc(base + 4, 0, 16, 128, base, None) == 1                 # table not 16-byte aligned
    assert b"aligned" in lib.alx_noalloc_last_error()
    assert lib.alx_gramian_noalloc(base, 0, 16, 128, base + 4, None) == 1                 # gramian not 8-byte aligned
    assert lib.alx_gramian_noalloc(base, 0, (1 << 20) + 1, 128, base, None) == 7          # beyond the fixed array
    assert b"exceed" in lib.alx_noalloc_last_error()
