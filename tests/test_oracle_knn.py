"""Pins for the kNN oracle: closed forms on lattices and a line, a k-d tree from a library,
a sort-based brute force, degenerate inputs.  No GPU."""
import numpy as np
import pytest

import oracle


def lattice(m, a):
    g = np.arange(m, dtype=np.float32) * np.float32(a)
    z, y, x = np.meshgrid(g, g, g, indexing="ij")
    return np.stack([x.ravel(), y.ravel(), z.ravel()], 1).astype(np.float32)   # index = (z*m + y)*m + x


def test_cubic_lattice_shells():
    # spacing 1/8 is a power of two: all squared distances are exact, shells are a^2, 2a^2, 3a^2
    m, a = 7, 0.125
    pos = lattice(m, a)
    x = np.ones((m ** 3, 1))
    c = (3 * m + 3) * m + 3                                     # interior point
    face = sorted([c - 1, c + 1, c - m, c + m, c - m * m, c + m * m])
    idx, d2, y, A = oracle.knn(pos, x, 6, rows=[c])
    assert idx[0].tolist() == face                               # equal distances: index order
    assert np.all(d2[0] == np.float32(a * a))
    assert y[0, 0] == 6.0 and A[0, 0] == 6.0
    idx, d2, _, _ = oracle.knn(pos, x, 18, rows=[c])
    assert idx[0, :6].tolist() == face
    edge = sorted(c + s1 * u + s2 * v for u, v in [(1, m), (1, m * m), (m, m * m)] for s1 in (-1, 1) for s2 in (-1, 1))
    assert idx[0, 6:].tolist() == edge
    assert np.all(d2[0, 6:] == np.float32(2 * a * a))
    idx, d2, _, _ = oracle.knn(pos, x, 26, rows=[c])
    assert np.all(d2[0, 18:] == np.float32(3 * a * a)) and len(set(idx[0].tolist())) == 26


def test_tie_goes_to_lowest_index():
    m, a = 5, 0.25
    pos = lattice(m, a)
    c = (2 * m + 2) * m + 2
    idx, _, _, _ = oracle.knn(pos, np.ones((m ** 3, 1)), 4, rows=[c])
    assert idx[0].tolist() == sorted([c - 1, c + 1, c - m, c + m, c - m * m, c + m * m])[:4]
    corner, _, _, _ = oracle.knn(pos, np.ones((m ** 3, 1)), 3, rows=[0])
    assert corner[0].tolist() == [1, m, m * m]


def test_points_on_a_line():
    xs = np.array([0, 1, 2, 4, 8, 16, 17], dtype=np.float32) / 32
    pos = np.stack([xs, np.zeros_like(xs), np.zeros_like(xs)], 1)
    feat = np.arange(7, dtype=np.float64)[:, None] + 1.0          # x_j = j + 1
    idx, d2, y, _ = oracle.knn(pos, feat, 2)
    assert idx.tolist() == [[1, 2], [0, 2], [1, 0], [2, 1], [3, 2], [6, 4], [5, 4]]
    assert d2[3].tolist() == [np.float32((2 / 32) ** 2), np.float32((3 / 32) ** 2)]
    assert y[:, 0].tolist() == [2 + 3, 1 + 3, 2 + 1, 3 + 2, 4 + 3, 7 + 5, 6 + 5]


def test_against_kd_tree():
    from scipy.spatial import cKDTree
    rng = np.random.default_rng(11)
    n, k = 4000, 16
    pos = rng.random((n, 3), dtype=np.float32)
    p64 = pos.astype(np.float64)
    d, i = cKDTree(p64).query(p64, k + 2)
    assert np.all(i[:, 0] == np.arange(n))                        # the query itself at distance 0
    idx, d2, _, _ = oracle.knn(pos, np.ones((n, 1)), k)
    sq = d[:, 1:] ** 2
    gaps = np.diff(sq, axis=1) / sq[:, 1:]
    clear = np.all(gaps > 1e-5, axis=1)                           # order not decided by fp32 rounding
    assert clear.mean() > 0.99
    assert np.array_equal(idx[clear], i[clear, 1:k + 1])
    assert np.allclose(d2, sq[:, :k], rtol=1e-6, atol=0)


def test_against_sorted_brute_force_with_duplicates():
    rng = np.random.default_rng(5)
    n, k, F = 300, 7, 3
    pos = (rng.integers(0, 12, (n, 3)) / 16).astype(np.float32)   # coarse grid: many ties and coincident points
    feat = rng.standard_normal((n, F))
    idx, d2, y, A = oracle.knn(pos, feat, k)
    for i in range(n):
        d = pos[i] - pos
        s = (d[:, 0] * d[:, 0] + d[:, 1] * d[:, 1]) + d[:, 2] * d[:, 2]     # float32 throughout
        assert s.dtype == np.float32
        others = np.array([j for j in range(n) if j != i])
        order = others[np.lexsort((others, s[others]))][:k]
        assert idx[i].tolist() == order.tolist()
        assert np.array_equal(d2[i], s[order])
        assert np.allclose(y[i], feat[order].sum(0), rtol=1e-13, atol=1e-13)
        assert np.allclose(A[i], np.abs(feat[order]).sum(0), rtol=1e-13)


def test_fewer_points_than_k_and_rows_subset():
    pos = np.array([[0, 0, 0], [0.5, 0, 0], [0, 0.25, 0]], dtype=np.float32)
    feat = np.array([[1.0], [10.0], [100.0]])
    idx, d2, y, _ = oracle.knn(pos, feat, 4)
    assert idx.tolist() == [[2, 1, -1, -1], [0, 2, -1, -1], [0, 1, -1, -1]]
    assert np.isinf(d2[:, 2:]).all() and d2[0, 0] == np.float32(0.0625)
    assert y[:, 0].tolist() == [110.0, 101.0, 11.0]
    one, _, _, _ = oracle.knn(pos[:1], feat[:1], 2)
    assert one.tolist() == [[-1, -1]]
    rng = np.random.default_rng(2)
    p = rng.random((500, 3), dtype=np.float32)
    f = rng.standard_normal((500, 2))
    full = oracle.knn(p, f, 5)
    rows = [499, 0, 17]
    part = oracle.knn(p, f, 5, rows=rows)
    for a, b in zip(full, part):
        assert np.array_equal(a[rows], b)
