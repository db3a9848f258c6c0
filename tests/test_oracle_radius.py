"""Pins for the radius part of the CPU oracle: an independent numpy all-pairs evaluation,
a k-d tree library routine, lattice closed forms, invariants (symmetry, Newton's third
law, translation / rotation invariance, adjoint identity) and finite differences."""
import itertools

import numpy as np
import pytest
from scipy.spatial import cKDTree

import gen
import oracle


def _points(n, seed, periodic, F=5):
    pos = gen.uniform_points(n, seed)
    x = gen.normal_features(n, F, seed, 31)
    gy = gen.normal_features(n, F, seed, 32)
    box = np.ones(3, np.float32)
    per = np.full(3, int(periodic), np.int32)
    return pos, x, gy, box, per


def _numpy_pairs(pos, r, box, per):
    """Independent all-pairs membership: displacement tensor by broadcasting."""
    p = pos.astype(np.float64)
    D = p[:, None, :] - p[None, :, :]
    for d in range(3):
        if per[d]:
            L = float(box[d])
            D[:, :, d] -= L * np.round(D[:, :, d] / L)
    d2 = np.einsum("ijk,ijk->ij", D, D)
    M = d2 <= float(r) ** 2
    np.fill_diagonal(M, False)
    return D, d2, M


# ------------------------------------------------------------------ grid constants / binning
def test_cell_grid_for_the_named_workloads():
    ones = np.ones(3, np.float32)
    n, _ = oracle.cell_grid(4096, np.float32(0.06), ones, [0, 0, 0])
    assert n.tolist() == [16, 16, 16]
    r2 = gen.radius_for_expected_neighbours(1_000_000, 32.0)
    n, invh = oracle.cell_grid(1_000_000, r2, ones, [1, 1, 1])
    assert n.tolist() == [50, 50, 50] and invh.tolist() == [50.0] * 3
    L = np.float32(160 * 0.8 ** (-1 / 3))
    n, _ = oracle.cell_grid(160 ** 3, np.float32(2.5), np.full(3, L, np.float32), [1, 1, 1])
    assert n.tolist() == [68, 68, 68]
    # periodic dimensions with fewer than 3 cells collapse to one cell; non-periodic keep 2
    n, _ = oracle.cell_grid(128, np.float32(0.35), ones, [1, 0, 1])
    assert n.tolist() == [1, 2, 1]
    # the number of cells never exceeds 8 n
    n, _ = oracle.cell_grid(10, np.float32(0.001), ones, [0, 0, 0])
    assert n.tolist() == [4, 4, 4]


@pytest.mark.parametrize("periodic", [0, 1])
def test_binning_matches_numpy_stable_sort(periodic):
    pos, _, _, box, per = _points(3000, 3, periodic)
    pos[0] = [0.0, 0.0, 0.0]
    pos[1] = [1.0, 1.0, 1.0]          # exactly on the upper faces: clamped into the last cell
    r = np.float32(0.11)
    b = oracle.bin_points(pos, r, box, per)
    nc = b["ncell"]
    assert nc.tolist() == [9, 9, 9]
    c = np.minimum(np.floor(pos * b["invh"][None, :]).astype(np.int64), nc[None, :] - 1)
    cid = (c[:, 2] * nc[1] + c[:, 1]) * nc[0] + c[:, 0]
    assert np.array_equal(b["cell"], cid)
    assert np.array_equal(b["order"], np.argsort(cid, kind="stable"))
    counts = np.bincount(cid, minlength=int(np.prod(nc)))
    assert np.array_equal(np.diff(b["cell_start"]), counts) and b["cell_start"][-1] == 3000
    assert sorted(b["order"].tolist()) == list(range(3000))
    # every point lies inside its cell's bounds (up to the fp32 product rounding)
    h = 1.0 / nc.astype(np.float64)
    assert np.all(pos >= c * h - 1e-6) and np.all(pos <= (c + 1) * h + 1e-6)


# ------------------------------------------------------------------ membership and counts
@pytest.mark.parametrize("periodic", [0, 1])
def test_counts_match_numpy_and_kdtree(periodic):
    pos, x, _, box, per = _points(700, 5, periodic)
    r = np.float32(0.13)
    _, _, cnt = oracle.radius_forward(pos, x, r, box, per, oracle.MSG_GAUSS, p0=0.07)
    _, _, M = _numpy_pairs(pos, r, box, per)
    assert np.array_equal(cnt, M.sum(1))
    assert cnt.sum() % 2 == 0
    tree = cKDTree(pos.astype(np.float64), boxsize=1.0 if periodic else None)
    nb = tree.query_ball_point(pos.astype(np.float64), float(r))
    assert np.array_equal(cnt, np.array([len(v) - 1 for v in nb]))


def test_cell_directory_variant_equals_all_pairs():
    for periodic, r in itertools.product([0, 1], [0.05, 0.2, 0.45]):
        pos, x, gy, box, per = _points(900, 7, periodic)
        r = np.float32(r)
        a = oracle.radius_forward(pos, x, r, box, per, oracle.MSG_GAUSS, p0=float(r) / 2)
        b = oracle.radius_forward(pos, x, r, box, per, oracle.MSG_GAUSS, p0=float(r) / 2, use_cells=True)
        for u, v in zip(a, b):
            assert np.array_equal(u, v)
        ga = oracle.radius_backward_gauss(pos, x, gy, r, box, per, float(r) / 2)
        gb = oracle.radius_backward_gauss(pos, x, gy, r, box, per, float(r) / 2, use_cells=True)
        for k in ga:
            assert np.array_equal(ga[k], gb[k])
    # anisotropic box, mixed periodicity, row subset
    pos, x, gy, _, _ = _points(600, 8, 0)
    box = np.array([1.0, 2.0, 0.5], np.float32)
    pos = pos * box[None, :]
    per = np.array([1, 0, 1], np.int32)
    rows = np.array([5, 17, 599, 0])
    a = oracle.radius_forward(pos, x, np.float32(0.2), box, per, oracle.MSG_DIST, rows=rows)
    b = oracle.radius_forward(pos, x, np.float32(0.2), box, per, oracle.MSG_DIST, rows=rows, use_cells=True)
    full = oracle.radius_forward(pos, x, np.float32(0.2), box, per, oracle.MSG_DIST)
    for u, v, w in zip(a, b, full):
        assert np.array_equal(u, v) and np.array_equal(u, w[rows])


# ------------------------------------------------------------------ Gaussian forward
@pytest.mark.parametrize("periodic", [0, 1])
def test_gaussian_forward_matches_numpy_all_pairs(periodic):
    pos, x, _, box, per = _points(400, 9, periodic)
    r = np.float32(0.17); sigma = np.float32(0.08)
    y, A, cnt = oracle.radius_forward(pos, x, r, box, per, oracle.MSG_GAUSS, p0=sigma)
    _, d2, M = _numpy_pairs(pos, r, box, per)
    Gm = np.where(M, np.exp(-d2 / (2 * float(sigma) ** 2)), 0.0)
    ref = Gm @ x.astype(np.float64)
    assert np.max(np.abs(y - ref) / (A + 1e-300)) < 1e-13
    assert np.max(np.abs(A - Gm @ np.abs(x.astype(np.float64))) / (A + 1e-300)) < 1e-13
    # features identically one: every column is the sum of the weights
    y1, _, _ = oracle.radius_forward(pos, np.ones((400, 3), np.float32), r, box, per,
                                     oracle.MSG_GAUSS, p0=sigma)
    assert np.allclose(y1, Gm.sum(1, keepdims=True), rtol=1e-13, atol=0)
    # DIST message: weights are the distances
    yd, _, _ = oracle.radius_forward(pos, x, r, box, per, oracle.MSG_DIST)
    refd = np.where(M, np.sqrt(d2), 0.0) @ x.astype(np.float64)
    assert np.max(np.abs(yd - refd)) < 1e-12


def test_no_neighbours_gives_zero_vector_and_self_is_excluded_by_index():
    pos = np.array([[0.1, 0.1, 0.1], [0.9, 0.9, 0.9], [0.5, 0.5, 0.5], [0.5, 0.5, 0.5]], np.float32)
    x = np.arange(8, dtype=np.float32).reshape(4, 2) + 1
    y, _, cnt = oracle.radius_forward(pos, x, np.float32(0.1), np.ones(3, np.float32), [0, 0, 0],
                                      oracle.MSG_GAUSS, p0=0.05)
    assert cnt.tolist() == [0, 0, 1, 1]                   # coincident distinct points are neighbours
    assert y[:2].tolist() == [[0, 0], [0, 0]]
    assert y[2].tolist() == x[3].tolist() and y[3].tolist() == x[2].tolist()   # exp(0) = 1
    # inclusive cutoff: binary-grid coordinates, distance exactly r
    pos = np.array([[0.25, 0.5, 0.5], [0.5, 0.5, 0.5]], np.float32)
    _, _, cnt = oracle.radius_forward(pos, x[:2], np.float32(0.25), np.ones(3, np.float32), [0, 0, 0],
                                      oracle.MSG_DIST)
    assert cnt.tolist() == [1, 1]
    # periodic wrap: 0.0625 and 0.9375 are 0.125 apart through the boundary
    pos = np.array([[0.0625, 0.5, 0.5], [0.9375, 0.5, 0.5]], np.float32)
    yp, _, cnt = oracle.radius_forward(pos, x[:2], np.float32(0.125), np.ones(3, np.float32),
                                       [1, 1, 1], oracle.MSG_DIST)
    assert cnt.tolist() == [1, 1] and yp[0].tolist() == (0.125 * x[1]).tolist()


# ------------------------------------------------------------------ Gaussian backward
def _numpy_two_scatter_backward(pos, x, gy, r, box, per, sigma):
    """Chain rule written as two scatters over directed pairs (i, j in N(i))."""
    D, d2, M = _numpy_pairs(pos, r, box, per)
    x = x.astype(np.float64); gy = gy.astype(np.float64)
    n = len(pos)
    gx = np.zeros_like(x); gp = np.zeros((n, 3))
    s2 = float(sigma) ** 2
    for i, j in zip(*np.nonzero(M)):
        g = np.exp(-d2[i, j] / (2 * s2))
        dot = gy[i] @ x[j]
        gx[j] += g * gy[i]
        gp[i] += -g / s2 * D[i, j] * dot
        gp[j] += +g / s2 * D[i, j] * dot
    return gx, gp


@pytest.mark.parametrize("periodic", [0, 1])
def test_backward_matches_two_scatter_chain_rule_and_invariants(periodic):
    pos, x, gy, box, per = _points(300, 13, periodic)
    r = np.float32(0.2); sigma = np.float32(0.1)
    b = oracle.radius_backward_gauss(pos, x, gy, r, box, per, sigma)
    gx, gp = _numpy_two_scatter_backward(pos, x, gy, r, box, per, sigma)
    assert np.max(np.abs(b["gx"] - gx) / (b["Agx"] + 1e-300)) < 1e-12
    assert np.max(np.abs(b["gp"] - gp) / (b["Agp"] + 1e-300)) < 1e-12
    # translation invariance: the position gradients sum to zero
    assert np.max(np.abs(b["gp"].sum(0))) < 1e-12 * b["Agp"].sum()
    if not periodic:   # rotation invariance (no box): net torque vanishes
        tq = np.cross(pos.astype(np.float64), b["gp"]).sum(0)
        assert np.max(np.abs(tq)) < 1e-12 * b["Agp"].sum()
    # adjoint identity: <ybar, y(x)> = <x, xbar(ybar)>
    y, A, _ = oracle.radius_forward(pos, x, r, box, per, oracle.MSG_GAUSS, p0=sigma)
    lhs = np.sum(gy.astype(np.float64) * y); rhs = np.sum(x.astype(np.float64) * b["gx"])
    assert abs(lhs - rhs) < 1e-12 * np.sum(np.abs(gy) * A)


@pytest.mark.parametrize("periodic", [0, 1])
def test_backward_matches_central_differences_on_frozen_membership(periodic):
    pos, x, gy, box, per = _points(120, 17, periodic, F=3)
    r = np.float32(0.3); sigma = np.float32(0.15)
    _, d2, _ = _numpy_pairs(pos, r, box, per)
    assert np.min(np.abs(np.sqrt(d2) - float(r))) > 1e-3 * float(r) * 0.01   # nobody on the cutoff
    b = oracle.radius_backward_gauss(pos, x, gy, r, box, per, sigma)
    P = pos.astype(np.float64); X = x.astype(np.float64); GY = gy.astype(np.float64)

    def loss(pp, xx):
        y, _, _ = oracle.radius_forward(pp, xx, r, box, per, oracle.MSG_GAUSS, p0=sigma)
        return np.sum(GY * y)

    h = 1e-6
    for (k, d) in [(0, 0), (7, 1), (55, 2), (119, 0)]:
        pp = P.copy(); pm = P.copy(); pp[k, d] += h; pm[k, d] -= h
        fd = (loss(pp, X) - loss(pm, X)) / (2 * h)
        assert abs(fd - b["gp"][k, d]) < 1e-6 * max(1.0, b["Agp"][k, d])
    for (k, f) in [(3, 0), (60, 2)]:
        xp = X.copy(); xm = X.copy(); xp[k, f] += h; xm[k, f] -= h
        fd = (loss(P, xp) - loss(P, xm)) / (2 * h)
        assert abs(fd - b["gx"][k, f]) < 1e-7 * max(1.0, b["Agx"][k, f])


# ------------------------------------------------------------------ Lennard-Jones
def _lattice_shell_sum(a, rc):
    """Closed form on a perfect simple cubic lattice: neighbours within rc and the energy
    per particle (1/2) sum 4 ((1/d)^12 - (1/d)^6)."""
    m = int(rc / a) + 1
    cnt = 0; e = 0.0
    for v in itertools.product(range(-m, m + 1), repeat=3):
        n2 = v[0] ** 2 + v[1] ** 2 + v[2] ** 2
        if n2 == 0:
            continue
        d2 = n2 * a * a
        if d2 <= rc * rc:
            cnt += 1
            q3 = (1.0 / d2) ** 3
            e += 0.5 * 4.0 * (q3 * q3 - q3)
    return cnt, e


def test_lj_perfect_lattice_closed_form():
    m = 8
    pos, L = gen.jittered_lattice(m, 0.8, 0.0)
    box = np.full(3, L, np.float32)
    y, A, cnt = oracle.radius_forward(pos, None, np.float32(2.5), box, [1, 1, 1], oracle.MSG_LJ, 1.0, 1.0)
    nref, eref = _lattice_shell_sum(0.8 ** (-1 / 3), 2.5)
    assert nref == 56 and np.all(cnt == 56)
    assert abs(eref - (-5.264771118950892)) < 1e-12
    assert np.max(np.abs(y[:, 3] - eref)) < 2e-5          # fp32 lattice coordinates
    assert np.max(np.abs(y[:, :3])) < 1e-4 * np.max(A[:, :3])


def test_lj_two_particles_and_third_law():
    d = 2.0 ** (1.0 / 6.0)
    pos = np.array([[1.0, 1.0, 1.0], [1.0 + d, 1.0, 1.0]], np.float64)
    y, _, cnt = oracle.radius_forward(pos, None, 2.5, np.full(3, 10.0), [0, 0, 0], oracle.MSG_LJ, 1.0, 1.0)
    assert cnt.tolist() == [1, 1]
    assert np.max(np.abs(y[:, :3])) < 1e-13               # force vanishes at the minimum
    assert abs(y[:, 3].sum() - (-1.0)) < 1e-14            # U = -eps, split in halves
    # closer than the minimum: repulsive, pushes particle 0 towards -x
    pos[1, 0] = 2.0
    y, _, _ = oracle.radius_forward(pos, None, 2.5, np.full(3, 10.0), [0, 0, 0], oracle.MSG_LJ, 1.0, 1.0)
    assert y[0, 0] == -24.0 and y[1, 0] == 24.0 and y[0, 3] == 0.0
    # eps and s scale as they should: U(d) = 4 eps ((s/d)^12 - (s/d)^6)
    y2, _, _ = oracle.radius_forward(pos * 2, None, 5.0, np.full(3, 20.0), [0, 0, 0], oracle.MSG_LJ, 3.0, 2.0)
    assert y2[0, 0] == -24.0 * 3.0 / 2.0
    c = gen.config("cfg3", m=6)
    y, A, cnt = oracle.radius_forward(c["pos"], None, c["r"], c["box"], c["periodic"], oracle.MSG_LJ, 1.0, 1.0)
    assert np.max(np.abs(y[:, :3].sum(0))) < 1e-12 * A[:, :3].sum()
    assert 50 < cnt.mean() < 60


def test_lj_force_is_minus_energy_gradient():
    c = gen.config("cfg3", m=5)
    P = c["pos"].astype(np.float64)
    box = c["box"].astype(np.float64)

    def energy(pp):
        y, _, _ = oracle.radius_forward(pp, None, 2.5, box, [1, 1, 1], oracle.MSG_LJ, 1.0, 1.0)
        return y[:, 3].sum()

    y, _, _ = oracle.radius_forward(P, None, 2.5, box, [1, 1, 1], oracle.MSG_LJ, 1.0, 1.0)
    h = 1e-6
    for (k, d) in [(0, 0), (31, 1), (124, 2)]:
        pp = P.copy(); pm = P.copy(); pp[k, d] += h; pm[k, d] -= h
        fd = -(energy(pp) - energy(pm)) / (2 * h)
        assert abs(fd - y[k, d]) < 1e-5 * max(1.0, abs(y[k, d]))
