"""CPU-only checks of the C ABI: the library builds, loads, exports every symbol the header
declares, and rejects bad arguments on the host before touching a device."""
import ctypes
import os
import re

import numpy as np
import pytest

import gen
import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2609_24802_b200 import build
    build.build_library()
    from paper_2609_24802_b200 import api
    return api


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "tiga.h")).read()
    declared = set(re.findall(r"\b(tiga_[a-z_0-9]+)\s*\(", header))
    assert declared == set(lib.EXPORTS)
    cdll = lib.load_library()
    for name in declared:
        assert getattr(cdll, name) is not None


def test_checked_build_exports_the_same_symbols(lib):
    """libtiga_checked.so (same sources, -DTIGA_CHECKED) loads and exports every declared symbol; the two
    builds tell themselves apart without a device."""
    from paper_2609_24802_b200 import build
    path = build.build_library(checked=True)
    checked = ctypes.CDLL(path)
    for name in lib.EXPORTS:
        assert getattr(checked, name) is not None
    checked.tiga_is_checked_build.restype = ctypes.c_int
    assert checked.tiga_is_checked_build() == 1
    assert lib.load_library().tiga_is_checked_build() == 0


def test_status_strings(lib):
    assert lib.tiga_status_string(0) == "ok"
    assert len({lib.tiga_status_string(s) for s in range(8)}) == 8


def test_grid_matches_the_oracle_reading(lib):
    cases = [(4096, 0.06, [1, 1, 1], [0, 0, 0]), (1_000_000, float(gen.radius_for_expected_neighbours(1_000_000, 32)), [1, 1, 1], [1, 1, 1]),
             (160 ** 3, 2.5, [172.3548] * 3, [1, 1, 1]), (128, 0.35, [1, 1, 1], [1, 0, 1]),
             (10, 0.001, [1, 1, 1], [0, 0, 0]), (5000, 0.07, [1.0, 2.5, 0.3], [1, 0, 0]), (1, 0.1, [1, 1, 1], [0, 0, 0])]
    for n, r, box, per in cases:
        nc, ih = lib.tiga_radius_grid(n, np.float32(r), np.float32(box), per)
        onc, oih = oracle.cell_grid(n, np.float32(r), np.float32(box), per)
        assert nc == onc.tolist() and np.array_equal(np.float32(ih), oih)


def test_host_side_argument_errors(lib):
    cdll = lib.load_library()
    from paper_2609_24802_b200.api import _Box, _Csr, _Msg
    b = _Box()
    for d in range(3):
        b.len[d] = 1.0
        b.periodic[d] = 1
    nc = (ctypes.c_int32 * 3)()
    # periodic box needs r < len/2; r must be positive
    assert cdll.tiga_radius_grid(100, ctypes.c_float(0.6), ctypes.byref(b), nc, None) == 1
    assert cdll.tiga_radius_grid(100, ctypes.c_float(-1.0), ctypes.byref(b), nc, None) == 1
    assert cdll.tiga_radius_grid(100, ctypes.c_float(0.1), None, nc, None) == 1
    assert cdll.tiga_radius_workspace_bytes(100, 4, ctypes.c_float(0.6), ctypes.byref(b), 0) == 0
    # point validation: host-side checks need no device
    assert cdll.tiga_validate_points(None, 10, ctypes.byref(b), 0, None, 0, None) == 1      # no positions
    assert cdll.tiga_validate_points(256, 10, None, 0, None, 0, None) == 1                  # no box
    assert cdll.tiga_validate_points(256, 10, ctypes.byref(b), 0, None, 0, None) == 0       # metadata only
    assert cdll.tiga_validate_points(256, 10, ctypes.byref(b), 1, None, 0, None) == 3       # level 1 needs scratch
    # CSR: null / misaligned pointers, negative sizes, unsupported widths
    g = _Csr(0, 0, 0, 4, 4, 0)
    msg = _Msg(0, 0.0, 0.0)
    assert cdll.tiga_apply_csr(ctypes.byref(g), None, 0, 4, None, ctypes.byref(msg), 0, None, None, None, 0, None) == 1
    g = _Csr(256, 0, 256, -1, 4, 0)
    assert cdll.tiga_apply_csr(ctypes.byref(g), None, 0, 4, None, ctypes.byref(msg), 0, None, None, None, 0, None) == 1
    g = _Csr(260, 0, 256, 4, 4, 8)            # rowptr not 16-byte aligned
    assert cdll.tiga_apply_csr(ctypes.byref(g), 256, 0, 4, None, ctypes.byref(msg), 0, 256, None, 256, 1 << 20, None) == 1
    g = _Csr(256, 0, 256, 4, 4, 8)
    assert cdll.tiga_apply_csr(ctypes.byref(g), 256, 0, 6, None, ctypes.byref(msg), 0, 256, None, 256, 1 << 20, None) == 2   # F % 4
    assert cdll.tiga_apply_csr(ctypes.byref(g), 256, 0, 4, None, ctypes.byref(msg), 0, 256, None, 256, 8, None) == 3        # workspace
    assert cdll.tiga_apply_csr(ctypes.byref(g), 256, 0, 4, None, ctypes.byref(msg), 1, 256, None, 256, 1 << 20, None) == 1  # max needs argmax
    assert cdll.tiga_apply_csr(ctypes.byref(g), 256, 0, 4, 256, ctypes.byref(msg), 0, 256, None, 256, 1 << 20, None) == 1   # COPY with weights
    assert cdll.tiga_csr_workspace_bytes(ctypes.byref(g), 64, 0, 0, 0) >= 2 * 64 * 4
    # the three reducers: unknown values are refused, 64-bit positions need the widest per-tile array, a relation of
    # 2^31 edges and more is refused by the 32-bit max reducer on the host (nothing is read: the pointers are fakes)
    assert cdll.tiga_apply_csr(ctypes.byref(g), 256, 0, 4, None, ctypes.byref(msg), 3, 256, 256, 256, 1 << 20, None) == 1
    ws = [cdll.tiga_csr_workspace_bytes(ctypes.byref(g), 64, 0, red, 0) for red in (0, 1, 2)]
    assert ws[0] < ws[1] < ws[2]
    huge = _Csr(256, 1, 256, 4, 4, (1 << 31) + 5)
    assert cdll.tiga_apply_csr(ctypes.byref(huge), 256, 0, 4, None, ctypes.byref(msg), 1, 256, 256, 256, 1 << 40, None) == 2
    assert cdll.tiga_apply_csr_backward(ctypes.byref(huge), 256, 0, 4, None, ctypes.byref(msg), 1, 256, 256, 256, None, None, 0, None) == 2
    assert cdll.tiga_csr_degree_histogram(ctypes.byref(g), 256, 0, 256, None) == 1                          # nbins < 1
    assert cdll.tiga_validate_csr(ctypes.byref(g), 0, None, 0, None) == 0                                   # metadata only
    # radius: message descriptor, widths, message parameters (all refused before any device access)
    b.periodic[0] = b.periodic[1] = b.periodic[2] = 0
    r = ctypes.c_float(0.1)
    big = 1 << 30
    assert cdll.tiga_apply_radius(256, 256, 100, 8, r, ctypes.byref(b), None, 256, None, 256, big, None) == 1          # no message
    assert cdll.tiga_apply_radius(256, 256, 100, 132, r, ctypes.byref(b), ctypes.byref(_Msg(2, 0.1, 0.0)), 256, None, 256, big, None) == 2
    assert cdll.tiga_apply_radius(256, 256, 100, 8, r, ctypes.byref(b), ctypes.byref(_Msg(2, 0.0, 0.0)), 256, None, 256, big, None) == 1    # sigma <= 0
    assert cdll.tiga_apply_radius(256, None, 100, 4, r, ctypes.byref(b), ctypes.byref(_Msg(4, 1.0, 0.0)), 256, None, 256, big, None) == 1   # s <= 0
    assert cdll.tiga_apply_radius(256, 256, 100, 8, r, ctypes.byref(b), ctypes.byref(_Msg(1, 0.0, 0.0)), 256, None, 256, big, None) == 2    # CSR message kind
    assert cdll.tiga_apply_radius(256, 256, 100, 8, r, ctypes.byref(b), ctypes.byref(_Msg(2, 0.1, 0.0)), 256, None, 256, 64, None) == 3     # workspace
    assert cdll.tiga_apply_radius_backward(256, 256, 100, 8, r, ctypes.byref(b), ctypes.byref(_Msg(4, 1.0, 1.0)), 256, 256, 256, 256, big, 0, None) == 2
    assert cdll.tiga_apply_radius_backward(256, 256, 100, 6, r, ctypes.byref(b), ctypes.byref(_Msg(2, 0.1, 0.0)), 256, 256, 256, 256, big, 0, None) == 2


def test_knn_and_attention_host_checks(lib):
    """Workspace sizing and argument checks of the widened entry points run on the host only."""
    cdll = lib.load_library()
    from paper_2609_24802_b200.api import _Box, _Csr
    box = _Box()
    for d in range(3):
        box.len[d] = 1.0
        box.periodic[d] = 0
    small = cdll.tiga_knn_workspace_bytes(1000, 16, ctypes.byref(box))
    large = cdll.tiga_knn_workspace_bytes(1_000_000, 16, ctypes.byref(box))
    assert 0 < small < large
    assert cdll.tiga_knn_workspace_bytes(1000, 33, ctypes.byref(box)) == 0          # k above the envelope
    assert cdll.tiga_knn_workspace_bytes(1000, 0, ctypes.byref(box)) == 0
    box.periodic[1] = 1
    assert cdll.tiga_knn_workspace_bytes(1000, 16, ctypes.byref(box)) == 0          # periodic boxes are not supported
    # statuses without touching a device: bad k, periodic box, bad width
    assert cdll.tiga_apply_knn(None, None, 10, 1, 0, ctypes.byref(box), None, None, None, None, 0, None) == 1
    assert cdll.tiga_apply_knn(None, None, 10, 1, 4, ctypes.byref(box), None, None, None, None, 0, None) == 2
    g = _Csr(0, 0, 0, 1_000_000, 1_000_000, 16_000_000)
    assert cdll.tiga_csr_attention_workspace_bytes(ctypes.byref(g), 64) > cdll.tiga_csr_attention_workspace_bytes(ctypes.byref(g), 8) > 0
    assert cdll.tiga_csr_attention_workspace_bytes(ctypes.byref(g), 6) == 0
    assert cdll.tiga_csr_attention_workspace_bytes(ctypes.byref(g), 256) == 0
    assert cdll.tiga_apply_csr_attention(ctypes.byref(g), None, None, None, 6, ctypes.c_float(1.0), None, None, None, 0, None) == 1
    assert cdll.tiga_apply_csr_attention(ctypes.byref(g), None, None, None, 132, ctypes.c_float(1.0), None, None, None, 0, None) == 2


def test_bench_probe_library_builds_and_checks_its_arguments(lib):
    """The benchmark's row-gather probe lives in a library of its own, outside the product ABI."""
    from paper_2609_24802_b200 import bench_probe
    cdll = bench_probe.load()
    assert cdll.tiga_bench_probe_row_gather(None, 10, 256, None, 10, None, None) == 1
    import subprocess
    syms = subprocess.run(["nm", "-D", lib.LIB_PATH], capture_output=True, text=True).stdout
    assert "probe" not in syms
