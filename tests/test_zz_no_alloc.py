"""tiga_apply_csr_builtin_ws: the CSR forward for callers that may not allocate device memory
(plug-ins that only receive input/output buffers, latency-critical loops, fixed memory budgets).
Its scratch is a fixed 8 MiB array inside the library instead of a caller-provided workspace, so
the checks here are: same results as tiga_apply_csr through the C ABI, on two calls in a row that
reuse the (dirty) array, and a clean refusal when the relation is too big for it.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import ctypes

import numpy as np
import pytest

import gen
import oracle
from parity import SUM_TOL, dev, host, rel_err

torch = pytest.importorskip("torch")


@pytest.mark.gpu
def test_builtin_scratch_matches_the_workspace_entry_point_twice_in_a_row():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2609_24802_b200 import api as T

    # call 1: R-MAT with rows far longer than a tile (many carry-outs), sum reducer
    rowptr, col = gen.rmat_csr(14, 16 << 14, seed=11)
    n = 1 << 14
    x = gen.normal_features(n, 64, 11)
    w = gen.edge_weights(16 << 14, 11)
    g = T.CsrRelation(dev(rowptr, torch), dev(col, torch), n)
    xd, wd = dev(x, torch), dev(w, torch)
    out = torch.empty((n, 64), device="cuda")            # the caller passes inputs and outputs
    ref, _ = T.tiga_apply_csr(g, xd, wd, T.SUM)
    got, _ = T.tiga_apply_csr_builtin_ws(g, xd, wd, T.SUM, out=out)
    torch.cuda.synchronize()
    y, A, _ = oracle.csr_forward(rowptr, col, x, w, oracle.SUM)
    assert got.data_ptr() == out.data_ptr()
    assert torch.equal(got, ref)                          # no atomics in the forward: bit-identical to the sibling
    assert rel_err(host(got), y, A) <= SUM_TOL            # and within tolerance of the oracle itself

    # call 2, straight after: another relation and the max reducer; the array still holds call 1's carries
    rowptr2, col2 = gen.rmat_csr(13, 24 << 13, seed=12)
    n2 = 1 << 13
    x2 = gen.normal_features(n2, 32, 12)
    g2 = T.CsrRelation(dev(rowptr2, torch), dev(col2, torch), n2)
    x2d = dev(x2, torch)
    out2 = torch.empty((n2, 32), device="cuda")
    arg2 = torch.empty((n2, 32), dtype=torch.int32, device="cuda")
    ref2, refarg2 = T.tiga_apply_csr(g2, x2d, None, T.MAX)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    got2, gotarg2 = T.tiga_apply_csr_builtin_ws(g2, x2d, None, T.MAX, out=out2, argmax=arg2)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before, "the call must not allocate (or free) device memory"
    assert torch.equal(got2, ref2) and torch.equal(gotarg2, refarg2)      # max outputs are bit exact
    ym, _, argm = oracle.csr_forward(rowptr2, col2, x2, None, oracle.MAX)
    assert np.array_equal(host(got2), ym.astype(np.float32)) and np.array_equal(host(gotarg2).astype(np.int64), argm)

    # and the first relation once more: results do not depend on what the array held
    got3, _ = T.tiga_apply_csr_builtin_ws(g, xd, wd, T.SUM, out=out)
    torch.cuda.synchronize()
    assert torch.equal(got3, ref) and rel_err(host(got3), y, A) <= SUM_TOL


@pytest.mark.gpu
def test_builtin_scratch_narrow_rows_with_a_row_cut_into_chunks():
    """Feature rows of 16 bytes (F = 8, fp16) take the row-class path, whose queue of chunks of very
    long rows also lives in the built-in array: one row of 20,000 edges among short and empty ones."""
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2609_24802_b200 import api as T
    g0 = gen.rng(13, 900)
    n_src = 5000
    deg = g0.integers(0, 12, size=3000)
    deg[g0.random(3000) < 0.4] = 0
    deg[1234] = 20_000                                   # above the 8192-edge chunk size
    deg[77] = 300                                        # a whole-warp row
    rowptr = np.concatenate([[0], np.cumsum(deg)]).astype(np.int64)
    col = g0.integers(0, n_src, size=int(rowptr[-1])).astype(np.int32)
    x = gen.normal_features(n_src, 8, 13, 31, np.float16)
    g = T.CsrRelation(dev(rowptr.astype(np.int32), torch), dev(col, torch), n_src)
    xd = dev(x, torch)
    out = torch.empty((3000, 8), device="cuda")
    y, A, _ = oracle.csr_forward(rowptr, col, x, None, oracle.SUM)
    ref, _ = T.tiga_apply_csr(g, xd, None, T.SUM)
    for _ in range(2):                                   # twice in a row: the second call finds the first one's queue
        out.fill_(float("nan"))
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        got, _ = T.tiga_apply_csr_builtin_ws(g, xd, None, T.SUM, out=out)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
        assert torch.equal(got, ref)
        assert rel_err(host(got), y, A) <= SUM_TOL


def test_relations_beyond_the_builtin_capacity_are_refused_on_the_host():
    from paper_2609_24802_b200 import build
    build.build_library()
    from paper_2609_24802_b200 import api as T
    from paper_2609_24802_b200.api import _Csr, _Msg
    lib = T.load_library()
    msg = _Msg(0, 0.0, 0.0)
    # (2^23 rows + 2^27 edges) / 1792 tiles * 276 bytes = 20.9 MiB > 8 MiB: refused before any device access
    big = _Csr(256, 0, 256, 1 << 23, 1 << 23, 1 << 27)
    assert lib.tiga_csr_workspace_bytes(ctypes.byref(big), 64, 0, 0, 0) > T.BUILTIN_WS_BYTES
    assert lib.tiga_apply_csr_builtin_ws(ctypes.byref(big), 256, 0, 64, None, ctypes.byref(msg), 0, 256, None, None) == 6
    assert "built-in scratch" in T.tiga_status_string(6)
    # bad arguments are still reported as such
    assert lib.tiga_apply_csr_builtin_ws(None, 256, 0, 64, None, ctypes.byref(msg), 0, 256, None, None) == 1
