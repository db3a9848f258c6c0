"""CPU oracle -- TEST INFRASTRUCTURE, not part of the product path.

Thin numpy/ctypes wrappers around ``tiga_oracle.c`` (plain fp64 loops written from the
paper's definitions).  Only ``tests/``, the smoke check and the benchmark's CPU-baseline
leg may import this package; the CUDA library never does, and this package never imports
the CUDA library.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tiga_oracle.c")
_SO = os.path.join(_HERE, "liboracle.so")
_lib = None

SUM, MAX = 0, 1
MSG_GAUSS, MSG_DIST, MSG_LJ = 2, 3, 4
_DT = {np.dtype(np.float32): 0, np.dtype(np.float16): 1, np.dtype(np.float64): 2}


def build(force: bool = False) -> str:
    """Compile the oracle (gcc -O2 -fopenmp -ffp-contract=off) next to its source."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC",
                               "-o", _SO, _SRC, "-lm"])
    return _SO


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_SO)
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _p(a):
    return ctypes.c_void_p(a.ctypes.data) if a is not None else ctypes.c_void_p(0)


def _field(a):
    """(contiguous array, dtype code) for an fp16/fp32/fp64 field; None -> (None, 0)."""
    if a is None:
        return None, 0
    a = np.ascontiguousarray(a)
    return a, _DT[a.dtype]


def _i64(a):
    return np.ascontiguousarray(a, dtype=np.int64)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


# ------------------------------------------------------------------------------ CSR
def csr_forward(rowptr, col, x, w=None, reducer=SUM):
    """Returns (y fp64 [n_dst,F], A fp64 [n_dst,F], arg int64 [n_dst,F] or None).

    For the max reducer with fp32 / fp16 features each message is rounded once to fp32
    before the comparison (the precision the messages exist in); fp64 features compare in fp64."""
    lib = _load()
    rowptr = _i64(rowptr); col = _i32(col)
    x, xdt = _field(x); w, wdt = _field(w)
    n = len(rowptr) - 1
    F = x.shape[1]
    y = np.empty((n, F), np.float64)
    A = np.empty((n, F), np.float64)
    arg = np.empty((n, F), np.int64) if reducer == MAX else None
    rc = lib.oracle_csr_forward(_p(rowptr), _p(col), ctypes.c_int64(n), _p(w), wdt, _p(x), xdt,
                                ctypes.c_int(F), ctypes.c_int(reducer), ctypes.c_int(int(xdt != 2)),
                                _p(y), _p(A), _p(arg))
    assert rc == 0
    return y, A, arg


def csr_backward_sum(rowptr, col, x, w, gy, n_src=None, want_gw=True, want_gx=True):
    """Returns dict(gw, Aw, gx, Ax) in fp64 (entries None when not requested)."""
    lib = _load()
    rowptr = _i64(rowptr); col = _i32(col)
    x, xdt = _field(x); w, wdt = _field(w); gy, gdt = _field(gy)
    n = len(rowptr) - 1
    E = len(col)
    n_src = x.shape[0] if n_src is None else n_src
    F = x.shape[1]
    gw = np.empty(E, np.float64) if want_gw else None
    Aw = np.empty(E, np.float64) if want_gw else None
    gx = np.empty((n_src, F), np.float64) if want_gx else None
    Ax = np.empty((n_src, F), np.float64) if want_gx else None
    rc = lib.oracle_csr_backward_sum(_p(rowptr), _p(col), ctypes.c_int64(n), ctypes.c_int64(n_src),
                                     _p(w), wdt, _p(x), xdt, ctypes.c_int(F), _p(gy), gdt,
                                     _p(gw), _p(Aw), _p(gx), _p(Ax))
    assert rc == 0
    return dict(gw=gw, Aw=Aw, gx=gx, Ax=Ax)


def csr_backward_max(rowptr, col, x, w, gy, arg, n_src=None):
    lib = _load()
    col = _i32(col); arg = _i64(arg)
    x, xdt = _field(x); w, wdt = _field(w); gy, gdt = _field(gy)
    n = len(rowptr) - 1
    E = len(col)
    n_src = x.shape[0] if n_src is None else n_src
    F = x.shape[1]
    gw = np.empty(E, np.float64); Aw = np.empty(E, np.float64)
    gx = np.empty((n_src, F), np.float64); Ax = np.empty((n_src, F), np.float64)
    rc = lib.oracle_csr_backward_max(_p(col), ctypes.c_int64(n), ctypes.c_int64(n_src),
                                     ctypes.c_int64(E), _p(w), wdt, _p(x), xdt, ctypes.c_int(F),
                                     _p(gy), gdt, _p(arg), _p(gw), _p(Aw), _p(gx), _p(Ax))
    assert rc == 0
    return dict(gw=gw, Aw=Aw, gx=gx, Ax=Ax)


def degree_histogram(rowptr, nbins=4096):
    """Returns (hist int64[nbins], max_degree)."""
    lib = _load()
    rowptr = _i64(rowptr)
    hist = np.empty(nbins, np.int64)
    mx = ctypes.c_int64(0)
    rc = lib.oracle_degree_histogram(_p(rowptr), ctypes.c_int64(len(rowptr) - 1),
                                     ctypes.c_int64(nbins), _p(hist), ctypes.byref(mx))
    assert rc == 0
    return hist, int(mx.value)


# ------------------------------------------------------------------------------ cells
def cell_grid(n, r, box, periodic):
    """Returns (ncell int32[3], invh fp32[3]) for n points, cutoff r (fp32), box (fp32[3])."""
    lib = _load()
    box = np.ascontiguousarray(box, np.float32); periodic = _i32(periodic)
    ncell = np.empty(3, np.int32); invh = np.empty(3, np.float32)
    rc = lib.oracle_cell_grid(ctypes.c_int64(n), ctypes.c_float(float(np.float32(r))), _p(box),
                              _p(periodic), _p(ncell), _p(invh))
    assert rc == 0
    return ncell, invh


def bin_points(pos, r, box, periodic):
    """Returns dict(ncell, invh, cell int32[n], cell_start int32[ncells+1], order int32[n])."""
    lib = _load()
    pos = np.ascontiguousarray(pos, np.float32)
    n = pos.shape[0]
    ncell, invh = cell_grid(n, r, box, periodic)
    nc = int(ncell[0]) * int(ncell[1]) * int(ncell[2])
    cell = np.empty(n, np.int32); start = np.empty(nc + 1, np.int32); order = np.empty(n, np.int32)
    rc = lib.oracle_bin(_p(pos), ctypes.c_int64(n), _p(ncell), _p(invh), _p(cell), _p(start), _p(order))
    assert rc == 0
    return dict(ncell=ncell, invh=invh, cell=cell, cell_start=start, order=order)


def csr_attention(rowptr, col, q, k, v, scale):
    """Online-softmax reducer over the rows of a stored relation: returns (y, A, lse) in fp64."""
    lib = _load()
    rowptr = _i64(rowptr); col = _i32(col)
    q = np.ascontiguousarray(q, dtype=np.float64)
    k = np.ascontiguousarray(k, dtype=np.float64)
    v = np.ascontiguousarray(v, dtype=np.float64)
    n, D = q.shape
    assert len(rowptr) == n + 1 and k.shape[1] == D and v.shape == k.shape
    y = np.empty((n, D), np.float64); A = np.empty((n, D), np.float64); lse = np.empty(n, np.float64)
    rc = lib.oracle_csr_attention(_p(rowptr), _p(col), ctypes.c_int64(n), _p(q), _p(k), _p(v), ctypes.c_int(D),
                                  ctypes.c_double(float(scale)), _p(y), _p(A), _p(lse))
    assert rc == 0
    return y, A, lse


# ------------------------------------------------------------------------------ radius
def _geom(pos, r, box, periodic):
    pos = np.ascontiguousarray(pos, dtype=np.float64)      # exact for fp32 input
    box = np.ascontiguousarray(np.asarray(box, dtype=np.float64))
    periodic = _i32(periodic)
    return pos, float(r), box, periodic


def radius_forward(pos, feat, r, box, periodic, kind=MSG_GAUSS, p0=1.0, p1=1.0,
                   rows=None, use_cells=False):
    """Returns (y fp64 [n_rows,Fout], A fp64, count int32[n_rows]).  r, p0, p1 are the
    caller's fp32 parameters converted exactly to double."""
    lib = _load()
    pos, r, box, periodic = _geom(pos, r, box, periodic)
    n = pos.shape[0]
    if kind == MSG_LJ:
        F = 0; Fo = 4; feat = None
    else:
        feat = np.ascontiguousarray(feat, dtype=np.float64)
        F = feat.shape[1]; Fo = F
    rows = None if rows is None else _i64(rows)
    nr = n if rows is None else len(rows)
    y = np.empty((nr, Fo), np.float64); A = np.empty((nr, Fo), np.float64)
    cnt = np.empty(nr, np.int32)
    rc = lib.oracle_radius_forward(_p(pos), _p(feat), ctypes.c_int64(n), ctypes.c_int(F),
                                   ctypes.c_double(r), _p(box), _p(periodic), ctypes.c_int(kind),
                                   ctypes.c_double(float(p0)), ctypes.c_double(float(p1)),
                                   _p(rows), ctypes.c_int64(nr), ctypes.c_int(int(use_cells)),
                                   _p(y), _p(A), _p(cnt))
    assert rc == 0
    return y, A, cnt


def radius_backward_gauss(pos, feat, gy, r, box, periodic, sigma, rows=None, use_cells=False):
    """Returns dict(gx, Agx [n_rows,F], gp, Agp [n_rows,3]) in fp64."""
    lib = _load()
    pos, r, box, periodic = _geom(pos, r, box, periodic)
    n = pos.shape[0]
    feat = np.ascontiguousarray(feat, dtype=np.float64)
    gy = np.ascontiguousarray(gy, dtype=np.float64)
    F = feat.shape[1]
    rows = None if rows is None else _i64(rows)
    nr = n if rows is None else len(rows)
    gx = np.empty((nr, F), np.float64); Agx = np.empty((nr, F), np.float64)
    gp = np.empty((nr, 3), np.float64); Agp = np.empty((nr, 3), np.float64)
    rc = lib.oracle_radius_backward_gauss(_p(pos), _p(feat), _p(gy), ctypes.c_int64(n),
                                          ctypes.c_int(F), ctypes.c_double(r), _p(box), _p(periodic),
                                          ctypes.c_double(float(sigma)), _p(rows), ctypes.c_int64(nr),
                                          ctypes.c_int(int(use_cells)), _p(gx), _p(Agx), _p(gp), _p(Agp))
    assert rc == 0
    return dict(gx=gx, Agx=Agx, gp=gp, Agp=Agp)


# ------------------------------------------------------------------------------ generated kNN
def knn(pos, feat, k, rows=None):
    """Exact k nearest neighbours by the key (fp32 squared distance, index) and their neighbour
    sum.  Returns (idx int32 [n_rows,k], d2 fp32 [n_rows,k], y fp64 [n_rows,F], A fp64)."""
    lib = _load()
    pos = np.ascontiguousarray(pos, dtype=np.float32)
    feat = np.ascontiguousarray(feat, dtype=np.float64)
    n = pos.shape[0]
    F = feat.shape[1]
    rows = None if rows is None else _i64(rows)
    nr = n if rows is None else len(rows)
    idx = np.empty((nr, k), np.int32); d2 = np.empty((nr, k), np.float32)
    y = np.empty((nr, F), np.float64); A = np.empty((nr, F), np.float64)
    rc = lib.oracle_knn(_p(pos), _p(feat), ctypes.c_int64(n), ctypes.c_int(F), ctypes.c_int(int(k)),
                        _p(rows), ctypes.c_int64(nr), _p(idx), _p(d2), _p(y), _p(A))
    assert rc == 0
    return idx, d2, y, A


# ------------------------------------------------------------------------------ edge neural network
def _mlp_args(W1, b1, W2, b2):
    W1 = np.ascontiguousarray(W1, np.float64); b1 = np.ascontiguousarray(b1, np.float64)
    W2 = np.ascontiguousarray(W2, np.float64); b2 = np.ascontiguousarray(b2, np.float64)
    return W1, b1, W2, b2


def radius_mlp_forward(pos, feat, r, box, periodic, W1, b1, W2, b2, use_cells=False):
    """y_i = sum_{j in N(i)} [W2 relu(W1 [p_j - p_i; x_j] + b1) + b2]  (Appendix A).
    Returns (y [n,Fout], A, count)."""
    lib = _load()
    pos, r, box, periodic = _geom(pos, r, box, periodic)
    feat = np.ascontiguousarray(feat, np.float64)
    W1, b1, W2, b2 = _mlp_args(W1, b1, W2, b2)
    n, Fin = feat.shape
    H, Fout = W1.shape[0], W2.shape[0]
    assert W1.shape == (H, 3 + Fin) and W2.shape == (Fout, H) and H <= 64 and Fout <= 16 and 3 + Fin <= 64
    y = np.empty((n, Fout)); A = np.empty((n, Fout)); cnt = np.empty(n, np.int32)
    rc = lib.oracle_radius_mlp_forward(_p(pos), _p(feat), ctypes.c_int64(n), ctypes.c_int(Fin), ctypes.c_double(r),
                                       _p(box), _p(periodic), _p(W1), _p(b1), _p(W2), _p(b2), ctypes.c_int(H),
                                       ctypes.c_int(Fout), ctypes.c_int(int(use_cells)), _p(y), _p(A), _p(cnt))
    assert rc == 0
    return y, A, cnt


def radius_mlp_backward(pos, feat, gy, r, box, periodic, W1, b1, W2, b2, use_cells=False, kink_eps=0.0):
    """Returns dict with gx, gp, gW1, gb1, gW2, gb2, their abs-sum companions A<name>, and
    ``kink`` (int32 [n]): 1 where some pair the point takes part in has a pre-activation with
    |h| < kink_eps (the ReLU derivative is discontinuous there)."""
    lib = _load()
    pos, r, box, periodic = _geom(pos, r, box, periodic)
    feat = np.ascontiguousarray(feat, np.float64); gy = np.ascontiguousarray(gy, np.float64)
    W1, b1, W2, b2 = _mlp_args(W1, b1, W2, b2)
    n, Fin = feat.shape
    H, Fout = W1.shape[0], W2.shape[0]
    shapes = dict(gx=(n, Fin), gp=(n, 3), gW1=W1.shape, gb1=b1.shape, gW2=W2.shape, gb2=b2.shape)
    out = {"kink": np.zeros(n, np.int32)}
    args = []
    for k, shp in shapes.items():
        out[k] = np.empty(shp); out["A" + k] = np.empty(shp)
        args += [_p(out[k]), _p(out["A" + k])]
    rc = lib.oracle_radius_mlp_backward(_p(pos), _p(feat), _p(gy), ctypes.c_int64(n), ctypes.c_int(Fin),
                                        ctypes.c_double(r), _p(box), _p(periodic), _p(W1), _p(b1), _p(W2), _p(b2),
                                        ctypes.c_int(H), ctypes.c_int(Fout), ctypes.c_int(int(use_cells)),
                                        ctypes.c_double(float(kink_eps)), _p(out["kink"]), *args)
    assert rc == 0
    return out
