"""ctypes binding of libtiga.so -- argument marshalling only.

Every function has the name of the C entry point it calls (see ``include/tiga.h``) and takes
torch CUDA tensors for the device arrays.  Nothing is computed here; when the library is
missing the import fails, there is no fallback of any kind.
"""
from __future__ import annotations

import ctypes
import os

import torch

__all__ = [
    "TigaError", "load_library", "EXPORTS", "SUM", "MAX", "MAX64", "F32", "F16",
    "MSG_COPY", "MSG_WEIGHTED", "MSG_GAUSS", "MSG_DIST", "MSG_LJ",
    "CsrRelation", "tiga_status_string", "tiga_csr_workspace_bytes", "tiga_validate_csr",
    "tiga_apply_csr", "tiga_apply_csr_builtin_ws", "tiga_apply_csr_backward", "tiga_csr_degree_histogram",
    "CsrPlan", "tiga_csr_plan_build", "tiga_csr_planned_workspace_bytes", "tiga_apply_csr_planned",
    "tiga_radius_grid", "tiga_validate_points", "tiga_radius_workspace_bytes", "tiga_radius_bin",
    "tiga_apply_radius", "tiga_apply_radius_backward", "tiga_apply_radius_mlp",
    "tiga_apply_radius_mlp_backward", "tiga_knn_workspace_bytes", "tiga_apply_knn",
    "tiga_csr_attention_workspace_bytes", "tiga_apply_csr_attention", "launch_count",
]

SUM, MAX, MAX64 = 0, 1, 2      # MAX64: max reducer whose argmax holds 64-bit edge positions (int64)
F32, F16 = 0, 1
I32, I64 = 0, 1
MSG_COPY, MSG_WEIGHTED, MSG_GAUSS, MSG_DIST, MSG_LJ = 0, 1, 2, 3, 4

EXPORTS = [
    "tiga_status_string", "tiga_kernel_launches", "tiga_checked_status", "tiga_is_checked_build", "tiga_csr_workspace_bytes", "tiga_validate_csr", "tiga_apply_csr",
    "tiga_apply_csr_builtin_ws", "tiga_apply_csr_backward", "tiga_csr_degree_histogram", "tiga_radius_grid",
    "tiga_csr_plan_bytes", "tiga_csr_plan_workspace_bytes", "tiga_csr_plan_build", "tiga_csr_planned_workspace_bytes",
    "tiga_apply_csr_planned",
    "tiga_validate_points", "tiga_radius_workspace_bytes", "tiga_radius_bin", "tiga_apply_radius",
    "tiga_apply_radius_backward", "tiga_apply_radius_mlp", "tiga_apply_radius_mlp_backward",
    "tiga_knn_workspace_bytes", "tiga_apply_knn", "tiga_csr_attention_workspace_bytes", "tiga_apply_csr_attention",
]

_HERE = os.path.dirname(os.path.abspath(__file__))
# TIGA_CHECKED=1 in the environment selects the checked build (range-checked indices, status word)
CHECKED = os.environ.get("TIGA_CHECKED", "0") not in ("", "0")
LIB_PATH = os.path.join(_HERE, "libtiga_checked.so" if CHECKED else "libtiga.so")


class TigaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {tiga_status_string(status)} (status {status})")


class _Msg(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("p0", ctypes.c_float), ("p1", ctypes.c_float)]


class _Csr(ctypes.Structure):
    _fields_ = [("rowptr", ctypes.c_void_p), ("rowptr_type", ctypes.c_int32), ("col", ctypes.c_void_p),
                ("n_dst", ctypes.c_int64), ("n_src", ctypes.c_int64), ("n_edges", ctypes.c_int64)]


class _Box(ctypes.Structure):
    _fields_ = [("len", ctypes.c_float * 3), ("periodic", ctypes.c_int32 * 3)]


class _EdgeMlp(ctypes.Structure):
    _fields_ = [("f_in", ctypes.c_int32), ("hidden", ctypes.c_int32), ("f_out", ctypes.c_int32),
                ("W1", ctypes.c_void_p), ("b1", ctypes.c_void_p), ("W2", ctypes.c_void_p), ("b2", ctypes.c_void_p)]


class _Plan(ctypes.Structure):
    _fields_ = [("n_dst", ctypes.c_int64), ("n_src", ctypes.c_int64), ("n_edges", ctypes.c_int64), ("n_hot", ctypes.c_int64),
                ("min_hot_degree", ctypes.c_int64), ("hot_edges", ctypes.c_int64), ("off_col", ctypes.c_int64),
                ("off_hot_id", ctypes.c_int64), ("used_bytes", ctypes.c_int64)]


_lib = None


def load_library() -> ctypes.CDLL:
    """Load libtiga.so; raises ImportError when it has not been built (no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with "
                          "`python -m paper_2609_24802_b200.build` (nvcc, sm_100a)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, sz, f = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t, ctypes.c_float
    lib.tiga_status_string.restype = ctypes.c_char_p
    lib.tiga_status_string.argtypes = [ctypes.c_int]
    lib.tiga_kernel_launches.restype = i64
    lib.tiga_kernel_launches.argtypes = []
    lib.tiga_checked_status.restype = ctypes.c_uint32
    lib.tiga_checked_status.argtypes = [ctypes.c_int]
    lib.tiga_is_checked_build.restype = ctypes.c_int
    lib.tiga_is_checked_build.argtypes = []
    lib.tiga_csr_workspace_bytes.restype = sz
    lib.tiga_csr_workspace_bytes.argtypes = [ctypes.POINTER(_Csr), i32, ctypes.c_int, ctypes.c_int, ctypes.c_int]
    lib.tiga_validate_csr.restype = ctypes.c_int
    lib.tiga_validate_csr.argtypes = [ctypes.POINTER(_Csr), ctypes.c_int, vp, sz, vp]
    lib.tiga_apply_csr.restype = ctypes.c_int
    lib.tiga_apply_csr.argtypes = [ctypes.POINTER(_Csr), vp, ctypes.c_int, i32, vp, ctypes.POINTER(_Msg), ctypes.c_int,
                                   vp, vp, vp, sz, vp]
    lib.tiga_apply_csr_builtin_ws.restype = ctypes.c_int
    lib.tiga_apply_csr_builtin_ws.argtypes = [ctypes.POINTER(_Csr), vp, ctypes.c_int, i32, vp, ctypes.POINTER(_Msg),
                                              ctypes.c_int, vp, vp, vp]
    lib.tiga_apply_csr_backward.restype = ctypes.c_int
    lib.tiga_apply_csr_backward.argtypes = [ctypes.POINTER(_Csr), vp, ctypes.c_int, i32, vp, ctypes.POINTER(_Msg), ctypes.c_int,
                                            vp, vp, vp, vp, vp, sz, vp]
    lib.tiga_csr_plan_bytes.restype = sz
    lib.tiga_csr_plan_bytes.argtypes = [ctypes.POINTER(_Csr), i64]
    lib.tiga_csr_plan_workspace_bytes.restype = sz
    lib.tiga_csr_plan_workspace_bytes.argtypes = [ctypes.POINTER(_Csr)]
    lib.tiga_csr_plan_build.restype = ctypes.c_int
    lib.tiga_csr_plan_build.argtypes = [ctypes.POINTER(_Csr), i64, vp, sz, vp, sz, ctypes.POINTER(_Plan), vp]
    lib.tiga_csr_planned_workspace_bytes.restype = sz
    lib.tiga_csr_planned_workspace_bytes.argtypes = [ctypes.POINTER(_Csr), ctypes.POINTER(_Plan), i32, ctypes.c_int, ctypes.c_int]
    lib.tiga_apply_csr_planned.restype = ctypes.c_int
    lib.tiga_apply_csr_planned.argtypes = [ctypes.POINTER(_Csr), ctypes.POINTER(_Plan), vp, vp, ctypes.c_int, i32, vp,
                                           ctypes.POINTER(_Msg), ctypes.c_int, vp, vp, vp, sz, vp]
    lib.tiga_csr_degree_histogram.restype = ctypes.c_int
    lib.tiga_csr_degree_histogram.argtypes = [ctypes.POINTER(_Csr), vp, i64, vp, vp]
    lib.tiga_radius_grid.restype = ctypes.c_int
    lib.tiga_radius_grid.argtypes = [i64, f, ctypes.POINTER(_Box), ctypes.POINTER(i32), ctypes.POINTER(f)]
    lib.tiga_validate_points.restype = ctypes.c_int
    lib.tiga_validate_points.argtypes = [vp, i64, ctypes.POINTER(_Box), ctypes.c_int, vp, sz, vp]
    lib.tiga_radius_workspace_bytes.restype = sz
    lib.tiga_radius_workspace_bytes.argtypes = [i64, i32, f, ctypes.POINTER(_Box), ctypes.c_int]
    lib.tiga_radius_bin.restype = ctypes.c_int
    lib.tiga_radius_bin.argtypes = [vp, i64, f, ctypes.POINTER(_Box), vp, vp, vp, vp, sz, vp]
    lib.tiga_apply_radius.restype = ctypes.c_int
    lib.tiga_apply_radius.argtypes = [vp, vp, i64, i32, f, ctypes.POINTER(_Box), ctypes.POINTER(_Msg), vp, vp, vp, sz, vp]
    lib.tiga_apply_radius_backward.restype = ctypes.c_int
    lib.tiga_apply_radius_backward.argtypes = [vp, vp, i64, i32, f, ctypes.POINTER(_Box), ctypes.POINTER(_Msg), vp, vp, vp,
                                               vp, sz, ctypes.c_int, vp]
    lib.tiga_apply_radius_mlp.restype = ctypes.c_int
    lib.tiga_apply_radius_mlp.argtypes = [vp, vp, i64, f, ctypes.POINTER(_Box), ctypes.POINTER(_EdgeMlp), vp, vp, vp, sz, vp]
    lib.tiga_apply_radius_mlp_backward.restype = ctypes.c_int
    lib.tiga_apply_radius_mlp_backward.argtypes = [vp, vp, i64, f, ctypes.POINTER(_Box), ctypes.POINTER(_EdgeMlp), vp,
                                                   vp, vp, vp, vp, vp, vp, vp, sz, ctypes.c_int, vp]
    lib.tiga_csr_attention_workspace_bytes.restype = sz
    lib.tiga_csr_attention_workspace_bytes.argtypes = [ctypes.POINTER(_Csr), i32]
    lib.tiga_apply_csr_attention.restype = ctypes.c_int
    lib.tiga_apply_csr_attention.argtypes = [ctypes.POINTER(_Csr), vp, vp, vp, i32, f, vp, vp, vp, sz, vp]
    lib.tiga_knn_workspace_bytes.restype = sz
    lib.tiga_knn_workspace_bytes.argtypes = [i64, i32, ctypes.POINTER(_Box)]
    lib.tiga_apply_knn.restype = ctypes.c_int
    lib.tiga_apply_knn.argtypes = [vp, vp, i64, i32, i32, ctypes.POINTER(_Box), vp, vp, vp, vp, sz, vp]
    _lib = lib
    return lib


load_library()      # fail at import time, loudly, when the CUDA library is not there


def checked_status(reset: bool = True) -> int:
    """Bits of the checked build's status word (0 in the normal build): 1 source index, 2 edge position,
    4 point id, 8 slot.  Synchronises the device."""
    return int(load_library().tiga_checked_status(int(reset)))


def is_checked_build() -> bool:
    return bool(load_library().tiga_is_checked_build())


def launch_count() -> int:
    """Kernels launched by the library so far in this process (counted inside the library)."""
    return int(load_library().tiga_kernel_launches())


def _ptr(t):
    if t is None:
        return ctypes.c_void_p(0)
    assert t.is_cuda and t.is_contiguous(), "device arrays must be contiguous CUDA tensors"
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _ok(st, where):
    if st != 0:
        raise TigaError(st, where)


def _ws(nbytes, like):
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=like.device)


def _dt(t):
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.float16:
        return F16
    raise TypeError("features must be float32 or float16")


def tiga_status_string(status: int) -> str:
    return load_library().tiga_status_string(int(status)).decode()


class CsrRelation:
    """Host-side descriptor (the C struct ``tiga_csr``) of device CSR arrays."""

    def __init__(self, rowptr: torch.Tensor, col: torch.Tensor, n_src: int):
        assert rowptr.dtype in (torch.int32, torch.int64) and col.dtype == torch.int32
        self.rowptr, self.col = rowptr, col
        self.n_dst = rowptr.numel() - 1
        self.n_src = int(n_src)
        self.n_edges = col.numel()
        self.c = _Csr(rowptr.data_ptr(), I32 if rowptr.dtype == torch.int32 else I64,
                      col.data_ptr() if col.numel() else 0, self.n_dst, self.n_src, self.n_edges)

    @property
    def ref(self):
        return ctypes.byref(self.c)


def tiga_csr_workspace_bytes(g: CsrRelation, F: int, x_dtype: int = F32, reducer: int = SUM,
                             backward: bool = False) -> int:
    return int(load_library().tiga_csr_workspace_bytes(g.ref, F, x_dtype, reducer, int(backward)))


def tiga_validate_csr(g: CsrRelation, level: int = 1, stream=None) -> None:
    ws = _ws(256, g.rowptr)
    _ok(load_library().tiga_validate_csr(g.ref, level, _ptr(ws), ws.numel(), _stream(stream)), "tiga_validate_csr")


def tiga_apply_csr(g: CsrRelation, x, w=None, reducer: int = SUM, out=None, argmax=None, ws=None, stream=None):
    """out[i,:] = reduce over the row's edges of w[e] * x[col[e],:].  Returns (out, argmax)."""
    F = x.shape[1]
    if out is None:
        out = torch.empty((g.n_dst, F), dtype=torch.float32, device=x.device)
    if reducer in (MAX, MAX64) and argmax is None:
        argmax = torch.empty((g.n_dst, F), dtype=torch.int32 if reducer == MAX else torch.int64, device=x.device)
    if ws is None:
        ws = _ws(tiga_csr_workspace_bytes(g, F, _dt(x), reducer, False), x)
    msg = _Msg(MSG_COPY if w is None else MSG_WEIGHTED, 0.0, 0.0)
    _ok(load_library().tiga_apply_csr(g.ref, _ptr(x), _dt(x), F, _ptr(w), ctypes.byref(msg), reducer, _ptr(out),
                                      _ptr(argmax), _ptr(ws), ws.numel(), _stream(stream)), "tiga_apply_csr")
    return out, argmax


BUILTIN_WS_BYTES = 8 << 20


def tiga_apply_csr_builtin_ws(g: CsrRelation, x, w=None, reducer: int = SUM, out=None, argmax=None, stream=None):
    """tiga_apply_csr without a workspace argument: the library's fixed 8 MiB device array is the
    scratch, for callers that may not allocate device memory.  Raises TigaError (status 6) when the
    relation needs more than that.  Calls that overlap on the GPU race on the shared array.
    `out` (and `argmax` for MAX) should be passed in by such callers; they are created here only
    as a convenience when omitted.  Returns (out, argmax)."""
    F = x.shape[1]
    if out is None:
        out = torch.empty((g.n_dst, F), dtype=torch.float32, device=x.device)
    if reducer in (MAX, MAX64) and argmax is None:
        argmax = torch.empty((g.n_dst, F), dtype=torch.int32 if reducer == MAX else torch.int64, device=x.device)
    msg = _Msg(MSG_COPY if w is None else MSG_WEIGHTED, 0.0, 0.0)
    _ok(load_library().tiga_apply_csr_builtin_ws(g.ref, _ptr(x), _dt(x), F, _ptr(w), ctypes.byref(msg), reducer,
                                                 _ptr(out), _ptr(argmax), _stream(stream)), "tiga_apply_csr_builtin_ws")
    return out, argmax


def tiga_apply_csr_backward(g: CsrRelation, x, w, grad_out, reducer: int = SUM, argmax=None,
                            grad_x=None, grad_w=None, want_x=True, want_w=True, ws=None, stream=None):
    """Returns (grad_x, grad_w); either is None when not requested."""
    F = x.shape[1]
    if want_x and grad_x is None:
        grad_x = torch.empty((g.n_src, F), dtype=torch.float32, device=x.device)
    if want_w and grad_w is None:
        grad_w = torch.empty((g.n_edges,), dtype=torch.float32, device=x.device)
    if ws is None:
        ws = _ws(tiga_csr_workspace_bytes(g, F, _dt(x), reducer, True), x)
    msg = _Msg(MSG_COPY if w is None else MSG_WEIGHTED, 0.0, 0.0)
    _ok(load_library().tiga_apply_csr_backward(g.ref, _ptr(x), _dt(x), F, _ptr(w), ctypes.byref(msg), reducer, _ptr(grad_out),
                                               _ptr(argmax), _ptr(grad_x), _ptr(grad_w), _ptr(ws), ws.numel(),
                                               _stream(stream)), "tiga_apply_csr_backward")
    return grad_x, grad_w


class CsrPlan:
    """A built hot-source plan: the host struct ``tiga_csr_plan``, the device buffer it describes and
    the relation it was built for."""

    def __init__(self, g, c, buf, scratch_bytes):
        self.g, self.c, self.buf, self.scratch_bytes = g, c, buf, int(scratch_bytes)

    n_hot = property(lambda self: int(self.c.n_hot))
    hot_edges = property(lambda self: int(self.c.hot_edges))
    min_hot_degree = property(lambda self: int(self.c.min_hot_degree))
    nbytes = property(lambda self: int(self.c.used_bytes))

    def array(self, name):
        """View of one of the plan's device arrays: 'col' or 'hot_id'."""
        off, n = {"col": (self.c.off_col, self.c.n_edges), "hot_id": (self.c.off_hot_id, self.c.n_hot)}[name]
        return self.buf[off:off + 4 * n].view(torch.int32)


def tiga_csr_plan_build(g: CsrRelation, max_hot_rows: int = None, row_bytes: int = 16, hot_bytes: int = 48 << 20,
                        stream=None) -> CsrPlan:
    """Builds the hot-source plan of a relation (one-time, synchronises).  ``max_hot_rows`` defaults to
    as many rows as fit ``hot_bytes`` of compact feature table."""
    lib = load_library()
    if max_hot_rows is None:
        max_hot_rows = max(1, hot_bytes // row_bytes)
    max_hot_rows = int(min(max_hot_rows, g.n_src))
    nbytes = int(lib.tiga_csr_plan_bytes(g.ref, max_hot_rows))
    wbytes = int(lib.tiga_csr_plan_workspace_bytes(g.ref))
    if nbytes == 0:
        raise TigaError(2, "tiga_csr_plan_bytes")
    buf = torch.empty(nbytes, dtype=torch.uint8, device=g.col.device)
    ws = torch.empty(wbytes, dtype=torch.uint8, device=g.col.device)
    c = _Plan()
    _ok(lib.tiga_csr_plan_build(g.ref, max_hot_rows, _ptr(buf), nbytes, _ptr(ws), wbytes, ctypes.byref(c), _stream(stream)),
        "tiga_csr_plan_build")
    return CsrPlan(g, c, buf, wbytes)


def tiga_csr_planned_workspace_bytes(plan: CsrPlan, F: int, x_dtype: int = F32, reducer: int = SUM) -> int:
    return int(load_library().tiga_csr_planned_workspace_bytes(plan.g.ref, ctypes.byref(plan.c), F, x_dtype, reducer))


def tiga_apply_csr_planned(plan: CsrPlan, x, w=None, reducer: int = SUM, out=None, argmax=None, ws=None, stream=None):
    """tiga_apply_csr through a hot-source plan.  Returns (out, argmax)."""
    F = x.shape[1]
    g = plan.g
    if out is None:
        out = torch.empty((g.n_dst, F), dtype=torch.float32, device=x.device)
    if reducer in (MAX, MAX64) and argmax is None:
        argmax = torch.empty((g.n_dst, F), dtype=torch.int32 if reducer == MAX else torch.int64, device=x.device)
    if ws is None:
        ws = _ws(tiga_csr_planned_workspace_bytes(plan, F, _dt(x), reducer), x)
    msg = _Msg(MSG_COPY if w is None else MSG_WEIGHTED, 0.0, 0.0)
    _ok(load_library().tiga_apply_csr_planned(g.ref, ctypes.byref(plan.c), _ptr(plan.buf), _ptr(x), _dt(x), F, _ptr(w),
                                              ctypes.byref(msg), reducer, _ptr(out), _ptr(argmax), _ptr(ws), ws.numel(),
                                              _stream(stream)), "tiga_apply_csr_planned")
    return out, argmax


def tiga_csr_degree_histogram(g: CsrRelation, nbins: int = 4096, stream=None):
    """Returns (hist int64[nbins], max_degree int64[1]) as device tensors."""
    hist = torch.empty(nbins, dtype=torch.int64, device=g.rowptr.device)
    mx = torch.empty(1, dtype=torch.int64, device=g.rowptr.device)
    _ok(load_library().tiga_csr_degree_histogram(g.ref, _ptr(hist), nbins, _ptr(mx), _stream(stream)),
        "tiga_csr_degree_histogram")
    return hist, mx


def _box(box, periodic):
    b = _Box()
    for d in range(3):
        b.len[d] = float(box[d])
        b.periodic[d] = int(periodic[d])
    return b


def tiga_radius_grid(n: int, r: float, box, periodic):
    """Returns (ncell list[3], invh list[3]) -- host only."""
    b = _box(box, periodic)
    nc = (ctypes.c_int32 * 3)()
    ih = (ctypes.c_float * 3)()
    _ok(load_library().tiga_radius_grid(n, float(r), ctypes.byref(b), nc, ih), "tiga_radius_grid")
    return list(nc), list(ih)


def tiga_validate_points(pos, box, periodic=(0, 0, 0), level: int = 1, stream=None) -> None:
    """Raises TigaError (status 7) when a coordinate is not finite or lies outside [0, len]."""
    b = _box(box, periodic)
    ws = _ws(256, pos)
    _ok(load_library().tiga_validate_points(_ptr(pos), pos.shape[0], ctypes.byref(b), level, _ptr(ws), ws.numel(),
                                            _stream(stream)), "tiga_validate_points")


def tiga_radius_workspace_bytes(n: int, F: int, r: float, box, periodic, backward: bool = False) -> int:
    b = _box(box, periodic)
    return int(load_library().tiga_radius_workspace_bytes(n, F, float(r), ctypes.byref(b), int(backward)))


def tiga_radius_bin(pos, r: float, box, periodic, ws=None, stream=None):
    """Returns dict(cell, cell_start, order, ncell, ws)."""
    n = pos.shape[0]
    b = _box(box, periodic)
    ncell, _ = tiga_radius_grid(n, r, box, periodic)
    nc = ncell[0] * ncell[1] * ncell[2]
    cell = torch.empty(n, dtype=torch.int32, device=pos.device)
    start = torch.empty(nc + 1, dtype=torch.int32, device=pos.device)
    order = torch.empty(n, dtype=torch.int32, device=pos.device)
    if ws is None:
        ws = _ws(tiga_radius_workspace_bytes(n, 0, r, box, periodic), pos)
    _ok(load_library().tiga_radius_bin(_ptr(pos), n, float(r), ctypes.byref(b), _ptr(cell), _ptr(start),
                                       _ptr(order), _ptr(ws), ws.numel(), _stream(stream)), "tiga_radius_bin")
    return dict(cell=cell, cell_start=start, order=order, ncell=ncell, ws=ws)


def tiga_apply_radius(pos, feat, r: float, box, periodic, kind: int = MSG_GAUSS, p0: float = 1.0,
                      p1: float = 1.0, out=None, count=None, want_count=False, ws=None, stream=None):
    """Fused bin + traverse + message + sum.  Returns (out, count, ws)."""
    n = pos.shape[0]
    F = 4 if kind == MSG_LJ else feat.shape[1]
    b = _box(box, periodic)
    if out is None:
        out = torch.empty((n, F), dtype=torch.float32, device=pos.device)
    if want_count and count is None:
        count = torch.empty(n, dtype=torch.int32, device=pos.device)
    if ws is None:
        ws = _ws(tiga_radius_workspace_bytes(n, F, r, box, periodic), pos)
    _ok(load_library().tiga_apply_radius(_ptr(pos), _ptr(feat), n, F, float(r), ctypes.byref(b),
                                         ctypes.byref(_Msg(kind, float(p0), float(p1))), _ptr(out), _ptr(count), _ptr(ws),
                                         ws.numel(), _stream(stream)), "tiga_apply_radius")
    return out, count, ws


def tiga_apply_radius_backward(pos, feat, grad_out, r: float, box, periodic, sigma: float, ws=None,
                               reuse_plan=False, grad_feat=None, grad_pos=None, want_feat=True, want_pos=True,
                               stream=None):
    """Reverse mode of the Gaussian message.  Returns (grad_feat, grad_pos)."""
    n, F = feat.shape
    b = _box(box, periodic)
    if want_feat and grad_feat is None:
        grad_feat = torch.empty((n, F), dtype=torch.float32, device=pos.device)
    if want_pos and grad_pos is None:
        grad_pos = torch.empty((n, 3), dtype=torch.float32, device=pos.device)
    if ws is None:
        assert not reuse_plan
        ws = _ws(tiga_radius_workspace_bytes(n, F, r, box, periodic, True), pos)
    _ok(load_library().tiga_apply_radius_backward(_ptr(pos), _ptr(feat), n, F, float(r), ctypes.byref(b),
                                                  ctypes.byref(_Msg(MSG_GAUSS, float(sigma), 0.0)), _ptr(grad_out),
                                                  _ptr(grad_feat), _ptr(grad_pos), _ptr(ws), ws.numel(),
                                                  int(bool(reuse_plan)), _stream(stream)),
        "tiga_apply_radius_backward")
    return grad_feat, grad_pos


def _edge_mlp(W1, b1, W2, b2):
    for t in (W1, b1, W2, b2):
        assert t.is_cuda and t.is_contiguous() and t.dtype == torch.float32
    H, K = W1.shape
    return _EdgeMlp(K - 3, H, W2.shape[0], W1.data_ptr(), b1.data_ptr(), W2.data_ptr(), b2.data_ptr())


def tiga_apply_radius_mlp(pos, feat, r: float, box, periodic, W1, b1, W2, b2, out=None, count=None,
                          want_count=False, ws=None, stream=None):
    """out[i] = sum_{j in N(i)} [W2 relu(W1 [p_j - p_i; x_j] + b1) + b2].  Returns (out, count, ws)."""
    n = pos.shape[0]
    m = _edge_mlp(W1, b1, W2, b2)
    bx = _box(box, periodic)
    if out is None:
        out = torch.empty((n, m.f_out), dtype=torch.float32, device=pos.device)
    if want_count and count is None:
        count = torch.empty(n, dtype=torch.int32, device=pos.device)
    if ws is None:
        ws = _ws(tiga_radius_workspace_bytes(n, m.f_in, r, box, periodic), pos)
    _ok(load_library().tiga_apply_radius_mlp(_ptr(pos), _ptr(feat), n, float(r), ctypes.byref(bx), ctypes.byref(m),
                                             _ptr(out), _ptr(count), _ptr(ws), ws.numel(), _stream(stream)),
        "tiga_apply_radius_mlp")
    return out, count, ws


def tiga_apply_radius_mlp_backward(pos, feat, grad_out, r: float, box, periodic, W1, b1, W2, b2, ws=None,
                                   reuse_plan=False, stream=None):
    """Returns dict(grad_feat, grad_pos, grad_W1, grad_b1, grad_W2, grad_b2)."""
    n = pos.shape[0]
    m = _edge_mlp(W1, b1, W2, b2)
    bx = _box(box, periodic)
    dev = pos.device
    g = dict(grad_feat=torch.empty((n, m.f_in), device=dev), grad_pos=torch.empty((n, 3), device=dev),
             grad_W1=torch.empty_like(W1), grad_b1=torch.empty_like(b1), grad_W2=torch.empty_like(W2),
             grad_b2=torch.empty_like(b2))
    if ws is None:
        assert not reuse_plan
        ws = _ws(tiga_radius_workspace_bytes(n, m.f_in, r, box, periodic, True), pos)
    _ok(load_library().tiga_apply_radius_mlp_backward(_ptr(pos), _ptr(feat), n, float(r), ctypes.byref(bx), ctypes.byref(m),
                                                      _ptr(grad_out), _ptr(g["grad_feat"]), _ptr(g["grad_pos"]),
                                                      _ptr(g["grad_W1"]), _ptr(g["grad_b1"]), _ptr(g["grad_W2"]),
                                                      _ptr(g["grad_b2"]), _ptr(ws), ws.numel(), int(bool(reuse_plan)),
                                                      _stream(stream)), "tiga_apply_radius_mlp_backward")
    return g


def tiga_knn_workspace_bytes(n: int, k: int, box) -> int:
    b = _box(box, (0, 0, 0))
    return int(load_library().tiga_knn_workspace_bytes(n, k, ctypes.byref(b)))


def tiga_apply_knn(pos, feat, k: int, box, periodic=(0, 0, 0), out=None, nbr=None, nbr_d2=None,
                   want_nbr=True, ws=None, stream=None):
    """out[i] = sum of feat[j] over the k nearest j != i by the key (fp32 squared distance, index).
    Returns (out, nbr int32 [n,k] or None, nbr_d2 fp32 [n,k] or None, ws)."""
    n, F = feat.shape
    b = _box(box, periodic)
    dev = pos.device
    if out is None:
        out = torch.empty((n, F), dtype=torch.float32, device=dev)
    if want_nbr and nbr is None:
        nbr = torch.empty((n, k), dtype=torch.int32, device=dev)
    if want_nbr and nbr_d2 is None:
        nbr_d2 = torch.empty((n, k), dtype=torch.float32, device=dev)
    if ws is None:
        ws = _ws(tiga_knn_workspace_bytes(n, k, box), pos)
    _ok(load_library().tiga_apply_knn(_ptr(pos), _ptr(feat), n, F, int(k), ctypes.byref(b), _ptr(out), _ptr(nbr),
                                      _ptr(nbr_d2), _ptr(ws), ws.numel(), _stream(stream)), "tiga_apply_knn")
    return out, nbr, nbr_d2, ws


def tiga_csr_attention_workspace_bytes(g: CsrRelation, D: int) -> int:
    return int(load_library().tiga_csr_attention_workspace_bytes(g.ref, int(D)))


def tiga_apply_csr_attention(g: CsrRelation, q, key, value, scale: float, out=None, lse=None, want_lse=True,
                             ws=None, stream=None):
    """out[i] = sum_e softmax_e(scale * <q[i], key[col[e]]>) value[col[e]] over the edges of row i
    (online-softmax reducer).  Returns (out, lse, ws)."""
    D = q.shape[1]
    if out is None:
        out = torch.empty((g.n_dst, D), dtype=torch.float32, device=q.device)
    if want_lse and lse is None:
        lse = torch.empty(g.n_dst, dtype=torch.float32, device=q.device)
    if ws is None:
        ws = _ws(tiga_csr_attention_workspace_bytes(g, D), q)
    _ok(load_library().tiga_apply_csr_attention(g.ref, _ptr(q), _ptr(key), _ptr(value), D, float(scale), _ptr(out),
                                                _ptr(lse), _ptr(ws), ws.numel(), _stream(stream)), "tiga_apply_csr_attention")
    return out, lse, ws
