"""GPU test of the allocation-free entry point osscar_trace_noalloc.

Some users of this library run where device allocation is off limits (all memory already pooled by the
host application, or a loop that cannot tolerate the stall an allocation may cause).  For them the library
carries one reduction whose scratch is a fixed array inside the shared object.  This test calls it through
the C ABI twice in a row, on two different problems, and compares each result with the value the ordinary,
context-based entry point (osscar_gram's const_term = Tr(W^T G)) returns for the same data.  The second
problem is smaller than the first, so anything left in the shared scratch by call one would show up.
Collected last on purpose: the file name sorts after every other test file.
"""
import ctypes

import numpy as np
import pytest
import torch

import workloads

pytestmark = pytest.mark.gpu


def _const_from_gram(pkg, wl):
    solver = pkg.Solver()
    W = wl.weight().cuda()
    H, G, const = solver.gram([c.cuda() for c in wl.x_chunks()], W, wl.damp)
    solver.close()
    return W, G, const


def test_noalloc_trace_matches_gram_const_twice():
    import paper_2403_12983_b200 as pkg
    b = pkg.binding
    first = workloads.config("c2", n=1024, d1=520, m=150, k=200, chunk_rows=1024, seed=5)
    second = workloads.config("c4", n=49 * 8, d1=9 * 20, m=33, k=7, chunk_rows=49 * 8, seed=6)
    for wl in (first, second):
        W, G, const = _const_from_gram(pkg, wl)
        got = b.osscar_trace_noalloc(W, G)
        assert got == pytest.approx(const, rel=1e-12)
        # and against a host fp64 sum of the same device arrays
        ref = float(np.sum(W.cpu().numpy().astype(np.float64) * G.cpu().numpy().astype(np.float64)))
        assert got == pytest.approx(ref, rel=1e-12)
    # strided views (leading dimension larger than the width) and an empty matrix
    Wv, Gv = W[:, :20], G[:, :20]
    ref = float(np.sum(Wv.cpu().numpy().astype(np.float64) * Gv.cpu().numpy().astype(np.float64)))
    assert b.osscar_trace_noalloc(Wv, Gv) == pytest.approx(ref, rel=1e-12)
    # the entry point's promise: a warmed call leaves the amount of free device memory where it was
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    assert b.osscar_trace_noalloc(Wv, Gv) == pytest.approx(ref, rel=1e-12)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    out = ctypes.c_double(-1.0)          # zero rows: valid pointers, nothing to add
    rc = pkg.lib().osscar_trace_noalloc(ctypes.c_void_p(W.data_ptr()), W.stride(0), ctypes.c_void_p(G.data_ptr()),
                                        G.stride(0), 0, W.shape[1], W.device.index, None, ctypes.byref(out))
    assert rc == b.OK and out.value == 0.0


def test_noalloc_rejects_sizes_beyond_its_scratch():
    import paper_2403_12983_b200 as pkg
    b = pkg.binding
    L = pkg.lib()
    A = torch.zeros(8, 4, device="cuda")
    out = ctypes.c_double(0.0)
    too_many = 65536 + 1
    rc = L.osscar_trace_noalloc(ctypes.c_void_p(A.data_ptr()), 4, ctypes.c_void_p(A.data_ptr()), 4, too_many, 4,
                                A.device.index, None, ctypes.byref(out))
    assert rc == b.E_SHAPE
    rc = L.osscar_trace_noalloc(None, 4, ctypes.c_void_p(A.data_ptr()), 4, 8, 4, A.device.index, None, ctypes.byref(out))
    assert rc == b.E_ARG
    # a matrix that does not live on the named device (here: pinned host memory) is refused, not dereferenced
    Hh = torch.zeros(8, 4).pin_memory()
    rc = L.osscar_trace_noalloc(ctypes.c_void_p(Hh.data_ptr()), 4, ctypes.c_void_p(A.data_ptr()), 4, 8, 4, A.device.index, None,
                                ctypes.byref(out))
    assert rc == b.E_ARG
