"""The allocation-free Gramian entry point against the context-based one and the oracle (collected last on purpose).

Some callers cannot allocate device memory at the moment they need a Gramian (a frozen memory pool, a
thread that must not take the allocator's lock).  ``alx_gramian_noalloc`` serves them from a fixed array
inside the library; here it is called through the C ABI twice in a row and compared with ``alx_gramian``
(bit for bit: the same kernels) and with the CPU oracle's Gramian of the same table.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def reference_gramian(table_bits, storage, n, d):
    from paper_2112_02194_b200 import ALX_ROWS, Alx
    # kernels=1: the FP32-ALU kernels, whose Gramian kernel the allocation-free entry point shares
    a = Alx(n, 4, d, 0.1, 0.01, storage=storage, kernels=1)
    a.set_embeddings(ALX_ROWS, table_bits)
    G = a.gramian(ALX_ROWS)
    a.destroy()
    return G


def test_noalloc_gramian_matches_context_gramian_twice_in_a_row():
    import torch
    from paper_2112_02194_b200 import binding
    from synth import graphs
    dev = torch.device("cuda")
    out = torch.empty((128, 128), dtype=torch.float64, device=dev)
    # first call: bf16, d = 128, several pieces and a ragged last one; second call: fewer rows, fp32, d = 64,
    # so stale pieces of the first call would show if the second call read them
    cases = [("bf16", 9000, 128, 31), ("f32", 4100, 64, 32)]
    from oracle import ials
    tables, refs, oracle_refs = [], [], []
    for storage, n, d, seed in cases:
        bits = graphs.init_embeddings(n, d, seed, 2, storage, sigma=0.5)
        t = torch.from_numpy(bits.view(np.int16) if storage == "bf16" else bits).to(dev)
        tables.append(t.view(torch.bfloat16) if storage == "bf16" else t)
        refs.append(reference_gramian(bits, storage, n, d))
        oracle_refs.append(ials.gramian(graphs.storage_to_f64(bits, storage)))
    free_before = torch.cuda.mem_get_info()[0]
    got = []
    for (storage, n, d, seed), t in zip(cases, tables):
        o = out.view(-1)[: d * d].view(d, d)
        binding.gramian_noalloc(t, o)
        torch.cuda.synchronize()
        got.append(o.cpu().numpy().copy())
    assert torch.cuda.mem_get_info()[0] >= free_before - (1 << 20)      # nothing was allocated by the calls
    for g, ref, oref in zip(got, refs, oracle_refs):
        assert np.abs(g - oref).max() <= 1e-6 * np.abs(oref).max()     # against the CPU oracle (fp32 sums of 4096 rows, fp64 across)
        np.testing.assert_array_equal(g, ref)                           # same kernels, same order of sums as alx_gramian


def test_noalloc_gramian_refuses_oversize_and_bad_arguments():
    import torch
    from paper_2112_02194_b200 import AlxError, binding
    lib = binding.load_library()
    assert binding.gramian_noalloc_max_rows(128) == 1 << 20
    assert binding.gramian_noalloc_max_rows(64) == 1 << 22
    assert binding.gramian_noalloc_max_rows(24) == 0
    out = torch.empty((128, 128), dtype=torch.float64, device="cuda")
    dummy = torch.zeros((16, 128), dtype=torch.float32, device="cuda")
    # size beyond the fixed array: refused before anything is launched (the pointer is never read)
    st = lib.alx_gramian_noalloc(dummy.data_ptr(), 0, (1 << 20) + 1, 128, out.data_ptr(), None)
    assert st == 7 and b"exceed" in lib.alx_noalloc_last_error()
    st = lib.alx_gramian_noalloc(dummy.data_ptr(), 0, 16, 48, out.data_ptr(), None)
    assert st == 7
    st = lib.alx_gramian_noalloc(None, 0, 16, 128, out.data_ptr(), None)
    assert st == 1
    # pointers the 16-byte loads / double stores could not take are refused, not dereferenced
    st = lib.alx_gramian_noalloc(dummy.data_ptr() + 4, 0, 15, 128, out.data_ptr(), None)
    assert st == 1 and b"aligned" in lib.alx_noalloc_last_error()
    st = lib.alx_gramian_noalloc(dummy.data_ptr(), 0, 16, 128, out.data_ptr() + 4, None)
    assert st == 1
    with pytest.raises(TypeError):
        binding.gramian_noalloc(torch.zeros((16, 128), dtype=torch.float16, device="cuda"), out)
    binding.gramian_noalloc(dummy, out)
    torch.cuda.synchronize()
    assert float(out.abs().max()) == 0.0
    with pytest.raises(AlxError):
        binding.gramian_noalloc(torch.zeros((16, 24), device="cuda"), out.view(-1)[:576].view(24, 24))
