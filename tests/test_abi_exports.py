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
