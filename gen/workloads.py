"""Seeded synthetic workloads (host side, numpy + a small C generator for R-MAT).

Everything is derived from an integer seed through counter-based generators
(numpy's Philox keyed by (seed, stream); a splitmix hash in ``rmat.c``), so the bytes do
not depend on thread count.  Nothing here performs the method's arithmetic.
"""
from __future__ import annotations

import ctypes
import hashlib
import math
import os
import subprocess

import numpy as np

__all__ = [
    "DEFAULT_SEED", "build_generators", "rng", "sha256_of", "rmat_csr", "rmat_edge",
    "edge_weights", "normal_features", "small_int_features", "small_int_weights",
    "uniform_points", "jittered_lattice", "hex_mesh_csr", "periodic_offset_csr",
    "regular_random_csr", "radius_for_expected_neighbours", "config", "surface_points", "mlp_params",
    "clustered_points",
]

DEFAULT_SEED = 20260921
_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libtigagen.so")
_lib = None


def build_generators(force: bool = False) -> str:
    """Compile ``rmat.c`` into ``libtigagen.so`` next to this file (gcc, OpenMP)."""
    src = os.path.join(_HERE, "rmat.c")
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(src):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _SO, src])
    return _SO


def _load():
    global _lib
    if _lib is None:
        build_generators()
        lib = ctypes.CDLL(_SO)
        lib.tigagen_rmat_csr.restype = ctypes.c_int
        lib.tigagen_rmat_csr.argtypes = [ctypes.c_uint64, ctypes.c_int, ctypes.c_int64,
                                         ctypes.c_double, ctypes.c_double, ctypes.c_double,
                                         ctypes.c_void_p, ctypes.c_void_p]
        lib.tigagen_rmat_edge.restype = None
        lib.tigagen_rmat_edge.argtypes = [ctypes.c_uint64, ctypes.c_int, ctypes.c_double,
                                          ctypes.c_double, ctypes.c_double, ctypes.c_int64,
                                          ctypes.c_void_p, ctypes.c_void_p]
        _lib = lib
    return _lib


def rng(seed: int, stream: int) -> np.random.Generator:
    """Counter-based generator for (seed, stream)."""
    return np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), int(stream)]))


def sha256_of(*arrays) -> str:
    h = hashlib.sha256()
    for a in arrays:
        h.update(np.ascontiguousarray(a).view(np.uint8).tobytes())
    return h.hexdigest()


# ----------------------------------------------------------------------------- graphs
def rmat_csr(scale: int, n_edges: int, seed: int = DEFAULT_SEED, a=0.57, b=0.19, c=0.19,
             index64: bool = False):
    """Destination-oriented CSR of an R-MAT graph (see ``rmat.c`` for the recipe).

    Returns (rowptr, col): rowptr int32 (or int64 when ``index64``) of length 2^scale+1,
    col int32 of length n_edges.  Duplicates and self loops are kept.
    """
    lib = _load()
    n = 1 << scale
    rowptr = np.zeros(n + 1, dtype=np.int64)
    col = np.empty(n_edges, dtype=np.int32)
    rc = lib.tigagen_rmat_csr(seed, scale, n_edges, a, b, c, rowptr.ctypes.data, col.ctypes.data)
    if rc != 0:
        raise RuntimeError("tigagen_rmat_csr failed")
    if not index64:
        if n_edges >= 2**31:
            raise ValueError("int32 rowptr cannot index this many edges")
        rowptr = rowptr.astype(np.int32)
    return rowptr, col


def rmat_edge(scale: int, e: int, seed: int = DEFAULT_SEED, a=0.57, b=0.19, c=0.19):
    """(row, col) of generation index ``e`` -- for spot checks of the CSR."""
    lib = _load()
    r = ctypes.c_int64()
    cc = ctypes.c_int64()
    lib.tigagen_rmat_edge(seed, scale, a, b, c, e, ctypes.byref(r), ctypes.byref(cc))
    return r.value, cc.value


def hex_mesh_csr(L: int):
    """Structured non-periodic hexahedral mesh with L^3 nodes, x-major numbering.

    Nodes that share an element are connected in both directions, no self entries:
    the 26-neighbourhood clipped at the boundary (paper, two-host experiment).
    Directed edge count is (3L-2)^3 - L^3.
    """
    idx = np.arange(L, dtype=np.int64)
    X, Y, Z = np.meshgrid(idx, idx, idx, indexing="ij")      # node id = (x*L + y)*L + z
    X = X.ravel(); Y = Y.ravel(); Z = Z.ravel()
    rows = []
    cols = []
    node = (X * L + Y) * L + Z
    for dx in (-1, 0, 1):
        for dy in (-1, 0, 1):
            for dz in (-1, 0, 1):
                if dx == 0 and dy == 0 and dz == 0:
                    continue
                ok = ((X + dx >= 0) & (X + dx < L) & (Y + dy >= 0) & (Y + dy < L)
                      & (Z + dz >= 0) & (Z + dz < L))
                rows.append(node[ok])
                cols.append(((X[ok] + dx) * L + (Y[ok] + dy)) * L + (Z[ok] + dz))
    rows = np.concatenate(rows)
    cols = np.concatenate(cols)
    order = np.lexsort((cols, rows))
    rows = rows[order]
    cols = cols[order]
    rowptr = np.zeros(L ** 3 + 1, dtype=np.int64)
    np.add.at(rowptr, rows + 1, 1)
    rowptr = np.cumsum(rowptr)
    return rowptr.astype(np.int32), cols.astype(np.int32)


def periodic_offset_csr(n: int, offsets, index64: bool = False):
    """Regular periodic graph: row i has sources (i + o_k) mod n, k = 0..len(offsets)-1."""
    offsets = np.asarray(offsets, dtype=np.int64)
    k = len(offsets)
    it = np.int64 if index64 else np.int32
    rowptr = (np.arange(n + 1, dtype=np.int64) * k).astype(it)
    col = ((np.arange(n, dtype=np.int64)[:, None] + offsets[None, :]) % n).astype(np.int32).ravel()
    return rowptr, col


def regular_random_csr(n: int, deg: int, seed: int = DEFAULT_SEED):
    """Every row has exactly ``deg`` uniformly random sources (the paper's degree-32 shape)."""
    g = rng(seed, 11)
    rowptr = (np.arange(n + 1, dtype=np.int64) * deg).astype(np.int32)
    col = g.integers(0, n, size=n * deg, dtype=np.int32)
    return rowptr, col


# ----------------------------------------------------------------------------- fields
def edge_weights(n_edges: int, seed: int = DEFAULT_SEED) -> np.ndarray:
    """fp32 weights (k+1)*2^-24 with k uniform in [0, 2^24-1): strictly inside (0,1)."""
    g = rng(seed, 21)
    k = g.integers(0, 2**24 - 1, size=n_edges, dtype=np.int64)
    return ((k + 1).astype(np.float64) * 2.0**-24).astype(np.float32)


def normal_features(n: int, F: int, seed: int = DEFAULT_SEED, stream: int = 31,
                    dtype=np.float32) -> np.ndarray:
    """N(0,1) features, drawn in fp32 and (for fp16) rounded once."""
    g = rng(seed, stream)
    x = g.standard_normal(size=(n, F), dtype=np.float32)
    return x.astype(dtype) if dtype != np.float32 else x


def small_int_features(n: int, F: int, seed: int = DEFAULT_SEED, lo=-4, hi=5,
                       dtype=np.float32) -> np.ndarray:
    """Small integers stored as floats: every partial sum stays exactly representable."""
    g = rng(seed, 41)
    return g.integers(lo, hi, size=(n, F)).astype(dtype)


def small_int_weights(n_edges: int, seed: int = DEFAULT_SEED, lo=1, hi=5) -> np.ndarray:
    g = rng(seed, 42)
    return g.integers(lo, hi, size=n_edges).astype(np.float32)


# ----------------------------------------------------------------------------- points
def uniform_points(n: int, seed: int = DEFAULT_SEED, stream: int = 51) -> np.ndarray:
    """i.i.d. uniform points k*2^-24 in [0,1)^3, fp32 (exactly representable)."""
    g = rng(seed, stream)
    k = g.integers(0, 2**24, size=(n, 3), dtype=np.int64)
    return (k.astype(np.float64) * 2.0**-24).astype(np.float32)


def jittered_lattice(m: int, density: float = 0.8, jitter: float = 0.1,
                     seed: int = DEFAULT_SEED):
    """m^3 particles on a simple cubic lattice of reduced density ``density`` with
    per-coordinate jitter U(-jitter, jitter), wrapped into the periodic box.

    Returns (pos fp32 [m^3,3], L fp32 box edge).  Lattice constant a = density^(-1/3).
    """
    a = density ** (-1.0 / 3.0)
    L = np.float32(m * a)
    idx = np.arange(m, dtype=np.float64) * a
    X, Y, Z = np.meshgrid(idx, idx, idx, indexing="ij")
    pos = np.stack([X.ravel(), Y.ravel(), Z.ravel()], axis=1)
    if jitter > 0:
        g = rng(seed, 61)
        pos = pos + g.uniform(-jitter, jitter, size=pos.shape)
    Ld = float(L)
    pos = pos - Ld * np.floor(pos / Ld)
    pos = pos.astype(np.float32)
    pos[pos >= L] = 0.0            # rounding up to L wraps to 0
    return pos, L


def radius_for_expected_neighbours(n: int, nbrs: float, volume: float = 1.0) -> np.float32:
    """r with (4/3) pi r^3 n / volume = nbrs, computed in double, rounded to fp32."""
    return np.float32((nbrs * 3.0 * volume / (4.0 * math.pi * n)) ** (1.0 / 3.0))


# ----------------------------------------------------------------------------- recipes
def config(name: str, seed: int = DEFAULT_SEED, **over):
    """Named workload recipes.  Returns a dict of host arrays and parameters.

    cfg0  radius tiny   : 4096 uniform points, non-periodic, r=0.06, sigma=0.03, F=16
    cfg1  CSR           : R-MAT scale 20, 16*2^20 edges, int32, F=64 fp32, w in (0,1)
    cfg2  radius mid    : 1e6 uniform points, periodic unit cube, 32 expected nbrs, F=32
    cfg3  Lennard-Jones : 160^3 jittered lattice, density 0.8, cutoff 2.5, periodic
    cfg4  CSR large     : R-MAT scale 26, 2^30 edges, int64 rowptr, F=8 fp16, unit weights
    Keyword overrides shrink a recipe (``n=``, ``scale=``, ``edge_factor=``, ``m=``, ``F=``).
    """
    if name in ("cfg0", "cfg2"):
        tiny = name == "cfg0"
        n = over.get("n", 4096 if tiny else 1_000_000)
        F = over.get("F", 16 if tiny else 32)
        periodic = over.get("periodic", not tiny)
        if tiny and "r" not in over and "n" not in over:
            r = np.float32(0.06)
        else:
            r = np.float32(over["r"]) if "r" in over else radius_for_expected_neighbours(
                n, over.get("nbrs", 32.0 if not tiny else 3.6191))
        sigma = np.float32(over["sigma"]) if "sigma" in over else np.float32(float(r) / 2.0)
        return dict(name=name, kind="radius_gauss", n=n, F=F, r=r, sigma=sigma,
                    box=np.ones(3, np.float32), periodic=np.full(3, int(periodic), np.int32),
                    pos=uniform_points(n, seed), x=normal_features(n, F, seed, 31),
                    gy=normal_features(n, F, seed, 32))
    if name == "cfg3":
        m = over.get("m", 160)
        pos, L = jittered_lattice(m, 0.8, over.get("jitter", 0.1), seed)
        return dict(name=name, kind="radius_lj", n=m ** 3, r=np.float32(2.5), eps=np.float32(1.0),
                    s=np.float32(1.0), box=np.full(3, L, np.float32),
                    periodic=np.ones(3, np.int32), pos=pos)
    if name in ("cfg1", "cfg4"):
        big = name == "cfg4"
        scale = over.get("scale", 26 if big else 20)
        ef = over.get("edge_factor", 16)
        F = over.get("F", 8 if big else 64)
        n = 1 << scale
        E = ef * n
        rowptr, col = rmat_csr(scale, E, seed, index64=big)
        d = dict(name=name, kind="csr", n=n, E=E, F=F, rowptr=rowptr, col=col,
                 x=normal_features(n, F, seed, 31, np.float16 if big else np.float32))
        if not big:
            d["w"] = edge_weights(E, seed)
            d["gy"] = normal_features(n, F, seed, 32)
        else:
            d["w"] = None
        return d
    raise KeyError(name)


def surface_points(n: int, seed: int = DEFAULT_SEED) -> np.ndarray:
    """n points on a closed, bumpy surface inside the unit cube (a stand-in for a scanned mesh's
    vertex list: positions only, roughly uniform over the surface)."""
    g = rng(seed, 81)
    v = g.standard_normal((n, 3))
    v /= np.linalg.norm(v, axis=1, keepdims=True)
    rad = 0.34 + 0.05 * np.sin(5.0 * v[:, 0]) * np.cos(3.0 * v[:, 1]) + 0.04 * v[:, 2] ** 2
    return (0.5 + v * rad[:, None]).astype(np.float32)


def clustered_points(n: int, seed: int = DEFAULT_SEED, blobs: int = 12, frac: float = 0.7) -> np.ndarray:
    """Uneven density in the unit cube: ``frac`` of the points in tight Gaussian blobs (clipped to
    the cube), the rest a thin uniform background.  Coordinates are k*2^-24."""
    g = rng(seed, 83)
    nb = int(n * frac)
    centres = g.random((blobs, 3)) * 0.8 + 0.1
    sig = g.uniform(0.004, 0.03, blobs)
    which = g.integers(0, blobs, nb)
    pts = centres[which] + g.standard_normal((nb, 3)) * sig[which, None]
    pts = np.concatenate([pts, g.random((n - nb, 3))], 0)
    pts = np.clip(pts, 0.0, 1.0 - 2.0**-24)
    return (np.floor(pts * 2.0**24) * 2.0**-24).astype(np.float32)[g.permutation(n)]


def mlp_params(f_in: int, hidden: int, f_out: int, seed: int = DEFAULT_SEED):
    """Random edge-network parameters (W1 [hidden, 3+f_in], b1, W2 [f_out, hidden], b2), fp32."""
    g = rng(seed, 82)
    k = 3 + f_in
    W1 = (g.uniform(-1, 1, (hidden, k)) / np.sqrt(k)).astype(np.float32)
    b1 = (g.uniform(-1, 1, hidden) / np.sqrt(k)).astype(np.float32)
    W2 = (g.uniform(-1, 1, (f_out, hidden)) / np.sqrt(hidden)).astype(np.float32)
    b2 = (g.uniform(-1, 1, f_out) / np.sqrt(hidden)).astype(np.float32)
    return W1, b1, W2, b2
