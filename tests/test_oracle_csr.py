"""Pins for the CSR part of the CPU oracle: printed values, closed forms, library special
cases, brute force on tiny graphs, adjoint identities and finite differences."""
import numpy as np
import pytest
import scipy.sparse as sp

import gen
import oracle
from conftest import read_golden


def _tiny_graph(seed, n_dst=9, n_src=7, max_deg=5, F=3):
    g = gen.rng(seed, 900)
    deg = g.integers(0, max_deg + 1, size=n_dst)
    deg[2] = 0
    rowptr = np.concatenate([[0], np.cumsum(deg)]).astype(np.int64)
    col = g.integers(0, n_src, size=rowptr[-1]).astype(np.int32)   # duplicates are likely
    x = g.standard_normal((n_src, F)).astype(np.float32)
    w = g.uniform(0.1, 1.0, size=rowptr[-1]).astype(np.float32)
    gy = g.standard_normal((n_dst, F)).astype(np.float32)
    return rowptr, col, x, w, gy


# ------------------------------------------------------------------ printed worked example
def test_worked_example_forward_and_backward():
    gd = read_golden("csr_worked_example.txt")
    rowptr = np.array(gd["rowptr"], np.int64)
    col = np.array(gd["col"], np.int32)
    x = np.array(gd["x"], np.float32)[:, None]
    w = np.array(gd["w"], np.float32)
    y, A, _ = oracle.csr_forward(rowptr, col, x, w, oracle.SUM)
    assert y[:, 0].tolist() == gd["y"]
    assert A[:, 0].tolist() == gd["y"]          # all contributions positive
    ones = np.ones((3, 1), np.float32)
    b = oracle.csr_backward_sum(rowptr, col, x, w, ones)
    assert b["gx"][:, 0].tolist() == gd["dx"]
    assert b["gw"].tolist() == gd["dw"]
    # max reducer on the same graph: row 0 = max(8, 15), row 1 = 6, empty row -> 0 / -1
    ym, _, arg = oracle.csr_forward(rowptr, col, x, w, oracle.MAX)
    assert ym[:, 0].tolist() == [15.0, 6.0, 0.0]
    assert arg[:, 0].tolist() == [1, 2, -1]


# ------------------------------------------------------------------ brute force, pure python
def _brute_forward(rowptr, col, x, w, reducer):
    n = len(rowptr) - 1
    F = x.shape[1]
    y = np.zeros((n, F)); arg = -np.ones((n, F), np.int64)
    for i in range(n):
        for f in range(F):
            msgs = [(float(w[e]) * float(x[col[e], f]), e) for e in range(rowptr[i], rowptr[i + 1])]
            if not msgs:
                continue
            if reducer == oracle.SUM:
                s = 0.0
                for m, _ in msgs:
                    s += m
                y[i, f] = s
            else:
                # fp32 inputs: the selection compares messages rounded once to fp32
                msgs = [(float(np.float32(m)), e) for m, e in msgs]
                best = max(m for m, _ in msgs)
                y[i, f] = best
                arg[i, f] = min(e for m, e in msgs if m == best)
    return y, arg


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_forward_matches_brute_force(seed):
    rowptr, col, x, w, _ = _tiny_graph(seed)
    for red in (oracle.SUM, oracle.MAX):
        y, _, arg = oracle.csr_forward(rowptr, col, x, w, red)
        yb, argb = _brute_forward(rowptr, col, x, w, red)
        assert np.array_equal(y, yb)
        if red == oracle.MAX:
            assert np.array_equal(arg, argb)


def test_max_tie_goes_to_lowest_edge_position():
    rowptr = np.array([0, 4, 4, 6], np.int64)
    col = np.array([1, 0, 1, 0, 2, 2], np.int32)        # duplicates
    x = np.array([[2.0, -1.0], [2.0, -1.0], [0.5, 0.5]], np.float32)
    w = np.array([1.0, 1.0, 1.0, 1.0, 3.0, 3.0], np.float32)
    y, _, arg = oracle.csr_forward(rowptr, col, x, w, oracle.MAX)
    assert arg.tolist() == [[0, 0], [-1, -1], [4, 4]]
    assert y.tolist() == [[2.0, -1.0], [0.0, 0.0], [1.5, 1.5]]


def test_max_values_match_torch_scatter_reduce():
    torch = pytest.importorskip("torch")
    rowptr, col, x, w, _ = _tiny_graph(11, n_dst=40, n_src=30, max_deg=9, F=4)
    y, _, _ = oracle.csr_forward(rowptr, col, x, w, oracle.MAX)
    rows = np.repeat(np.arange(len(rowptr) - 1), np.diff(rowptr))
    msg = torch.from_numpy(w.astype(np.float64))[:, None] * torch.from_numpy(x.astype(np.float64))[col]
    ref = torch.full((len(rowptr) - 1, 4), float("-inf"), dtype=torch.float64)
    ref = ref.scatter_reduce(0, torch.from_numpy(rows)[:, None].expand(-1, 4), msg, "amax")
    ref[torch.isinf(ref)] = 0.0
    assert np.array_equal(y, ref.numpy().astype(np.float32).astype(np.float64))   # rounding is monotone


# ------------------------------------------------------------------ library special case
def test_sum_is_sparse_matmul_and_backward_is_transpose():
    rowptr, col = gen.rmat_csr(10, 16 << 10, seed=5)
    n = 1 << 10
    x = gen.normal_features(n, 8, 5)
    w = gen.edge_weights(16 << 10, 5)
    gy = gen.normal_features(n, 8, 5, 32)
    Amat = sp.csr_matrix((w.astype(np.float64), col, rowptr.astype(np.int64)), shape=(n, n))
    y, A, _ = oracle.csr_forward(rowptr, col, x, w, oracle.SUM)
    ref = Amat @ x.astype(np.float64)
    assert np.max(np.abs(y - ref) / (A + 1e-300)) < 1e-14
    b = oracle.csr_backward_sum(rowptr, col, x, w, gy)
    refx = Amat.T @ gy.astype(np.float64)
    assert np.max(np.abs(b["gx"] - refx) / (b["Ax"] + 1e-300)) < 1e-14
    rows = np.repeat(np.arange(n), np.diff(rowptr))
    refw = np.einsum("ef,ef->e", x.astype(np.float64)[col], gy.astype(np.float64)[rows])
    assert np.max(np.abs(b["gw"] - refw) / (b["Aw"] + 1e-300)) < 1e-14
    # adjoint identity <ybar, A x> = <A^T ybar, x>
    lhs = np.sum(gy.astype(np.float64) * y)
    rhs = np.sum(b["gx"] * x.astype(np.float64))
    assert abs(lhs - rhs) < 1e-9 * np.sum(np.abs(gy) * A)


def test_unit_weights_when_w_is_none():
    rowptr, col, x, _, gy = _tiny_graph(4)
    y, _, _ = oracle.csr_forward(rowptr, col, x, None, oracle.SUM)
    y1, _, _ = oracle.csr_forward(rowptr, col, x, np.ones(len(col), np.float32), oracle.SUM)
    assert np.array_equal(y, y1)


def test_fp16_features_are_converted_exactly():
    rowptr, col, x, w, _ = _tiny_graph(6)
    xh = x.astype(np.float16)
    y16, _, _ = oracle.csr_forward(rowptr, col, xh, w, oracle.SUM)
    y32, _, _ = oracle.csr_forward(rowptr, col, xh.astype(np.float32), w, oracle.SUM)
    assert np.array_equal(y16, y32)
    sub = np.array([[2.0 ** -24, -2.0 ** -15, 65504.0]], np.float16)   # subnormal, tiny, max
    ys, _, _ = oracle.csr_forward(np.array([0, 1]), np.array([0], np.int32), sub, None, oracle.SUM)
    assert ys[0].tolist() == [2.0 ** -24, -2.0 ** -15, 65504.0]


# ------------------------------------------------------------------ closed forms
def test_periodic_offset_graph_closed_form_is_exact():
    # the paper validates its billion-edge run with a periodic closed form (Section 7,
    # "Billion-edge execution"); with small-integer fields every partial sum is an integer
    n, F = 4096, 4
    offs = [1, 2, 3, 5, 8, 13, 21, 34, -1, -2, -3, -5, -8, -13, -21, -34]
    rowptr, col = gen.periodic_offset_csr(n, offs)
    x = gen.small_int_features(n, F, 3)
    w = gen.small_int_weights(n * 16, 3)
    y, _, _ = oracle.csr_forward(rowptr, col, x, w, oracle.SUM)
    ref = np.zeros((n, F))
    for k, o in enumerate(offs):
        ref += w[k::16, None].astype(np.float64) * np.roll(x.astype(np.float64), -o, axis=0)
    assert np.array_equal(y, ref)


def test_hex_mesh_counts_and_degrees():
    gd = read_golden("hex_mesh_counts.txt")
    for L, nodes, edges in zip(gd["side"][:2], gd["nodes"][:2], gd["directed_edges"][:2]):
        L = int(L)
        rowptr, col = gen.hex_mesh_csr(L)
        assert len(rowptr) - 1 == int(nodes)
        assert rowptr[-1] == int(edges)
        assert int(edges) == (3 * L - 2) ** 3 - L ** 3
        ones = np.ones((L ** 3, 1), np.float32)
        y, _, _ = oracle.csr_forward(rowptr, col, ones, None, oracle.SUM)   # = degree
        hist, mx = oracle.degree_histogram(rowptr, 64)
        assert mx == int(gd["interior_degree"][0])
        assert hist[7] == 8 and hist[11] == 12 * (L - 2) and hist[17] == 6 * (L - 2) ** 2
        assert hist[26] == (L - 2) ** 3 and hist.sum() == L ** 3
        assert np.array_equal(np.bincount(y[:, 0].astype(np.int64), minlength=64), hist)


def test_degree_histogram_identities():
    rowptr, col = gen.rmat_csr(12, 16 << 12, seed=9)
    hist, mx = oracle.degree_histogram(rowptr, 4096)
    deg = np.diff(rowptr)
    assert np.array_equal(hist, np.bincount(np.minimum(deg, 4095), minlength=4096))
    assert mx == deg.max()
    assert hist.sum() == len(deg)
    hs, _ = oracle.degree_histogram(rowptr, 8)              # overflow bin
    assert hs[7] == np.sum(deg >= 7) and np.array_equal(hs[:7], np.bincount(deg, minlength=7)[:7])
    full, _ = oracle.degree_histogram(rowptr, int(mx) + 2)
    assert np.sum(np.arange(len(full)) * full) == rowptr[-1]   # degree sums equal E


def test_rmat_generator_shape():
    scale, E = 12, 16 << 12
    rowptr, col = gen.rmat_csr(scale, E, seed=9)
    assert rowptr[0] == 0 and rowptr[-1] == E and np.all(np.diff(rowptr) >= 0)
    assert col.min() >= 0 and col.max() < (1 << scale)
    # stable in generation order: rebuild the CSR from the raw edge stream
    rows = np.empty(E, np.int64); cols = np.empty(E, np.int64)
    for e in range(0, E, 97):
        rows[e], cols[e] = gen.rmat_edge(scale, e, seed=9)
    seen = {}
    deg_row0 = rowptr[1]
    # expected degree of row 0 is E (a+b)^scale
    assert abs(deg_row0 - E * 0.76 ** scale) < 6 * np.sqrt(E * 0.76 ** scale)
    for e in range(0, E, 97):
        r = rows[e]
        assert cols[e] in col[rowptr[r]:rowptr[r + 1]]


# ------------------------------------------------------------------ finite differences
def test_sum_backward_matches_central_differences():
    rowptr, col, x, w, gy = _tiny_graph(21)
    x = x.astype(np.float64); w = w.astype(np.float64); gy = gy.astype(np.float64)
    b = oracle.csr_backward_sum(rowptr, col, x, w, gy)

    def loss(xx, ww):
        y, _, _ = oracle.csr_forward(rowptr, col, xx, ww, oracle.SUM)
        return np.sum(gy * y)

    h = 1e-6
    for (j, f) in [(0, 0), (3, 2), (6, 1)]:
        xp = x.copy(); xm = x.copy(); xp[j, f] += h; xm[j, f] -= h
        assert abs((loss(xp, w) - loss(xm, w)) / (2 * h) - b["gx"][j, f]) < 1e-8
    for e in [0, len(col) // 2, len(col) - 1]:
        wp = w.copy(); wm = w.copy(); wp[e] += h; wm[e] -= h
        assert abs((loss(x, wp) - loss(x, wm)) / (2 * h) - b["gw"][e]) < 1e-8


def test_max_backward_matches_central_differences_away_from_ties():
    rowptr, col, x, w, gy = _tiny_graph(22)
    x = x.astype(np.float64); w = w.astype(np.float64); gy = gy.astype(np.float64)
    y, _, arg = oracle.csr_forward(rowptr, col, x, w, oracle.MAX)
    b = oracle.csr_backward_max(rowptr, col, x, w, gy, arg)

    def loss(xx, ww):
        yy, _, _ = oracle.csr_forward(rowptr, col, xx, ww, oracle.MAX)
        return np.sum(gy * yy)

    h = 1e-7
    gx = np.zeros_like(x); gw = np.zeros_like(w)
    for j in range(x.shape[0]):
        for f in range(x.shape[1]):
            xp = x.copy(); xm = x.copy(); xp[j, f] += h; xm[j, f] -= h
            gx[j, f] = (loss(xp, w) - loss(xm, w)) / (2 * h)
    for e in range(len(w)):
        wp = w.copy(); wm = w.copy(); wp[e] += h; wm[e] -= h
        gw[e] = (loss(x, wp) - loss(x, wm)) / (2 * h)
    assert np.max(np.abs(gx - b["gx"])) < 1e-6
    assert np.max(np.abs(gw - b["gw"])) < 1e-6
    # empty rows contribute nothing; every unselected edge has zero gradient
    sel = np.unique(arg[arg >= 0])
    mask = np.ones(len(w), bool); mask[sel] = False
    assert np.all(b["gw"][mask] == 0.0)


def test_max_selection_is_taken_in_message_precision():
    # two products that differ in fp64 but round to the same fp32 value are a tie:
    # the earlier edge wins and the output is that fp32 value
    x = np.array([[1.0 + 2 * 2.0 ** -23], [1.0]], np.float32)
    w = np.array([1.0 - 2 * 2.0 ** -24, 1.0 + 2.0 ** -23], np.float32)
    p0 = float(w[0]) * float(x[0, 0]); p1 = float(w[1]) * float(x[1, 0])
    assert p0 != p1 and np.float32(p0) == np.float32(p1) and p1 > p0
    y, _, arg = oracle.csr_forward(np.array([0, 2]), np.array([0, 1], np.int32), x, w, oracle.MAX)
    assert arg[0, 0] == 0 and y[0, 0] == float(np.float32(p0))
    # the same data in fp64 is no tie
    y, _, arg = oracle.csr_forward(np.array([0, 2]), np.array([0, 1], np.int32),
                                   x.astype(np.float64), w.astype(np.float64), oracle.MAX)
    assert arg[0, 0] == 1 and y[0, 0] == p1
