"""GPU parity: cell binning and the fused radius traversal (through the C ABI) against the
fp64 CPU oracle.  Cells, offsets, order and neighbour counts must match bit-exactly; sums
within 1e-5 and gradients within 1e-4 of the sum of absolute contributions."""
import numpy as np
import pytest

import gen
import oracle
from parity import GRAD_TOL, SUM_TOL, Guard, dev, host, rel_err

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tiga():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2609_24802_b200 import api
    return api


def _check_bin(tiga, pos, r, box, per):
    ref = oracle.bin_points(pos, r, box, per)
    got = tiga.tiga_radius_bin(dev(pos, torch), r, box, per)
    assert got["ncell"] == ref["ncell"].tolist()
    assert np.array_equal(host(got["cell"]), ref["cell"])
    assert np.array_equal(host(got["cell_start"]), ref["cell_start"])
    assert np.array_equal(host(got["order"]), ref["order"])


def _check_gauss(tiga, pos, x, gy, r, box, per, sigma, kind=None, use_cells=False, backward=True):
    kind = tiga.MSG_GAUSS if kind is None else kind
    y, A, cnt = oracle.radius_forward(pos, x, r, box, per, kind, p0=sigma, use_cells=use_cells)
    pd, xd = dev(pos, torch), dev(x, torch)
    guard = Guard(torch)
    n, F = x.shape
    ws = guard.workspace(tiga.tiga_radius_workspace_bytes(n, F, r, box, per))
    out, count, ws = tiga.tiga_apply_radius(pd, xd, r, box, per, kind, p0=sigma, out=guard.empty((n, F)),
                                            count=guard.empty((n,), torch.int32), ws=ws)
    guard.check()
    assert np.array_equal(host(count), cnt), "neighbour counts must be bit exact"
    assert rel_err(host(out), y, A) <= SUM_TOL
    if backward and kind == tiga.MSG_GAUSS:
        ref = oracle.radius_backward_gauss(pos, x, gy, r, box, per, sigma, use_cells=use_cells)
        gyd = dev(gy, torch)
        gx, gp = tiga.tiga_apply_radius_backward(pd, xd, gyd, r, box, per, sigma, ws=ws, reuse_plan=True,
                                                 grad_feat=guard.empty((n, F)), grad_pos=guard.empty((n, 3)))
        guard.check()
        assert rel_err(host(gx), ref["gx"], ref["Agx"]) <= GRAD_TOL
        assert rel_err(host(gp), ref["gp"], ref["Agp"]) <= GRAD_TOL
        gx2, gp2 = tiga.tiga_apply_radius_backward(pd, xd, gyd, r, box, per, sigma)      # rebuilds the bins
        assert torch.equal(gx, gx2) and torch.equal(gp, gp2)
    return out, count


# ------------------------------------------------------------------------------ binning
def test_binning_is_bit_exact(tiga):
    ones = np.ones(3, np.float32)
    for n, r, per, seed in [(4096, 0.06, [0, 0, 0], 1), (50_000, 0.05, [1, 1, 1], 2), (128, 0.35, [0, 0, 0], 7),
                            (3000, 0.3, [1, 0, 1], 3), (1000, 0.45, [1, 1, 1], 4), (7, 0.2, [0, 0, 0], 5),
                            (200_000, 0.004, [1, 1, 1], 6)]:
        pos = gen.uniform_points(n, seed)
        pos[0] = 0.0
        pos[-1] = 1.0                     # on the upper faces: clamped into the last cell
        _check_bin(tiga, pos, np.float32(r), ones, per)
    # everything in one cell; clustered points (a few very full cells)
    _check_bin(tiga, gen.uniform_points(500, 9) * np.float32(0.01), np.float32(0.1), ones, [0, 0, 0])
    p = gen.uniform_points(20_000, 10)
    p[:15_000] = p[:15_000] * np.float32(0.02) + np.float32(0.5)
    _check_bin(tiga, p, np.float32(0.05), ones, [1, 1, 1])
    # cell occupancies on both sides of the limits of the dense-cell ordering (256 by rank counting,
    # above that a sorting network: in shared memory up to 2048 ids, in place beyond), ids interleaved
    rng = np.random.default_rng(12)
    sizes = [256, 257, 2048, 2049, 8193]
    parts = [gen.uniform_points(m, 13 + k) * np.float32(0.2) + np.float32([0.25 * (k % 4), 0.25 * (k // 4), 0.0])
             for k, m in enumerate(sizes)]
    p = np.concatenate(parts)[rng.permutation(sum(sizes))]
    _check_bin(tiga, p, np.float32(0.25), ones, [0, 0, 0])
    # anisotropic box
    box = np.array([1.0, 2.5, 0.3], np.float32)
    _check_bin(tiga, gen.uniform_points(5000, 11) * box[None, :], np.float32(0.07), box, [1, 0, 0])
    c = gen.config("cfg3", m=20)
    _check_bin(tiga, c["pos"], c["r"], c["box"], c["periodic"])


# ------------------------------------------------------------------------------ Gaussian
def test_cfg0_tiny_forward_and_backward(tiga):
    c = gen.config("cfg0")
    _check_gauss(tiga, c["pos"], c["x"], c["gy"], c["r"], c["box"], c["periodic"], c["sigma"])


@pytest.mark.parametrize("periodic", [0, 1])
@pytest.mark.parametrize("F", [4, 16, 32, 64, 128])
def test_gaussian_small(tiga, periodic, F):
    n = 6000
    pos = gen.uniform_points(n, 20 + F)
    x = gen.normal_features(n, F, 20 + F, 31)
    gy = gen.normal_features(n, F, 20 + F, 32)
    r = gen.radius_for_expected_neighbours(n, 24.0)
    _check_gauss(tiga, pos, x, gy, r, np.ones(3, np.float32), [periodic] * 3, np.float32(float(r) / 2))


@pytest.mark.parametrize("F", [1, 3, 6])
def test_forward_widths_that_are_not_multiples_of_four(tiga, F):
    n = 5000
    pos = gen.uniform_points(n, 40 + F)
    x = gen.normal_features(n, F, 40 + F, 31)
    r = gen.radius_for_expected_neighbours(n, 32.0)
    ones = np.ones(3, np.float32)
    _check_gauss(tiga, pos, x, None, r, ones, [0, 0, 0], np.float32(float(r) / 2), backward=False)
    _check_gauss(tiga, pos, x, None, r, ones, [1, 1, 1], np.float32(float(r) / 2), kind=tiga.MSG_DIST)
    with pytest.raises(tiga.TigaError) as ei:      # the backward needs 128-bit rows
        tiga.tiga_apply_radius_backward(dev(pos, torch), dev(x, torch), dev(x, torch), r, ones, [0, 0, 0], 0.1)
    assert ei.value.status == 2


def test_few_cells_mixed_periodicity_and_anisotropic_box(tiga):
    # the paper's tiny radius shape: 128 points, cutoff 0.35 (two cells per dimension)
    pos = gen.uniform_points(128, 7)
    x = gen.normal_features(128, 8, 7); gy = gen.normal_features(128, 8, 7, 32)
    ones = np.ones(3, np.float32)
    _check_gauss(tiga, pos, x, gy, np.float32(0.35), ones, [0, 0, 0], np.float32(0.2))
    _check_gauss(tiga, pos, x, gy, np.float32(0.35), ones, [1, 1, 1], np.float32(0.2))   # one cell, minimum image
    _check_gauss(tiga, pos, x, gy, np.float32(0.3), ones, [1, 0, 1], np.float32(0.2))    # three cells where periodic
    box = np.array([1.0, 2.5, 0.3], np.float32)
    n = 4000
    pos = gen.uniform_points(n, 12) * box[None, :]
    x = gen.normal_features(n, 16, 12); gy = gen.normal_features(n, 16, 12, 32)
    _check_gauss(tiga, pos, x, gy, np.float32(0.09), box, [1, 0, 1], np.float32(0.05))
    # the paper's own message: distance-weighted sum
    _check_gauss(tiga, pos, x, gy, np.float32(0.09), box, [1, 0, 1], np.float32(0.05), kind=tiga.MSG_DIST)


def test_pairs_exactly_on_the_cutoff_are_neighbours(tiga):
    # binary-grid coordinates: many pairs at distance exactly r (inclusive predicate)
    k = np.arange(16, dtype=np.float32) / 16
    X, Y, Z = np.meshgrid(k, k, k, indexing="ij")
    pos = np.stack([X.ravel(), Y.ravel(), Z.ravel()], 1).astype(np.float32)
    n = pos.shape[0]
    x = gen.normal_features(n, 8, 5); gy = gen.normal_features(n, 8, 5, 32)
    for per in ([0, 0, 0], [1, 1, 1]):
        out, count = _check_gauss(tiga, pos, x, gy, np.float32(3.0 / 16), np.ones(3, np.float32), per, np.float32(0.1))
        if per[0]:
            # |v| <= 3 on the integer lattice: 123 points minus the origin
            assert np.all(host(count) == 122)


def test_no_neighbours_and_coincident_points(tiga):
    pos = np.array([[0.1, 0.1, 0.1], [0.9, 0.9, 0.9], [0.5, 0.5, 0.5], [0.5, 0.5, 0.5], [0.5, 0.5, 0.5]], np.float32)
    x = gen.normal_features(5, 4, 1); gy = gen.normal_features(5, 4, 1, 32)
    out, count = _check_gauss(tiga, pos, x, gy, np.float32(0.05), np.ones(3, np.float32), [0, 0, 0], np.float32(0.02))
    assert host(count).tolist() == [0, 0, 2, 2, 2]
    assert np.all(host(out)[:2] == 0.0)


def test_clustered_points_overflow_the_pair_list(tiga):
    n = 3000
    pos = gen.uniform_points(n, 15) * np.float32(0.1) + np.float32(0.3)       # ~500 neighbours each
    x = gen.normal_features(n, 32, 15); gy = gen.normal_features(n, 32, 15, 32)
    _check_gauss(tiga, pos, x, gy, np.float32(0.05), np.ones(3, np.float32), [0, 0, 0], np.float32(0.03))


def test_gaussian_mid_replica(tiga):
    """A 131,072-point replica of the 1M-point periodic workload (32 expected neighbours, F=32),
    every row against the oracle's cell-directory variant (itself pinned to all pairs)."""
    c = gen.config("cfg2", n=131_072)
    _check_gauss(tiga, c["pos"], c["x"], c["gy"], c["r"], c["box"], c["periodic"], c["sigma"], use_cells=True)


# ------------------------------------------------------------------------------ Lennard-Jones
def _check_lj(tiga, pos, r, box, per, eps=1.0, s=1.0, use_cells=False, tol=SUM_TOL):
    y, A, cnt = oracle.radius_forward(pos, None, r, box, per, oracle.MSG_LJ, eps, s, use_cells=use_cells)
    guard = Guard(torch)
    n = len(pos)
    out, count, _ = tiga.tiga_apply_radius(dev(pos, torch), None, r, box, per, tiga.MSG_LJ, p0=eps, p1=s,
                                           out=guard.empty((n, 4)), count=guard.empty((n,), torch.int32),
                                           ws=guard.workspace(tiga.tiga_radius_workspace_bytes(n, 4, r, box, per)))
    guard.check()
    assert np.array_equal(host(count), cnt)
    err = rel_err(host(out), y, A)
    print(f"Lennard-Jones: largest normalised error {err:.3e} (tolerance {tol:.1e})")
    assert err <= tol
    return host(out), A


def test_lennard_jones_lattices(tiga):
    c = gen.config("cfg3", m=12)
    out, A = _check_lj(tiga, c["pos"], c["r"], c["box"], c["periodic"])
    assert np.max(np.abs(out[:, :3].astype(np.float64).sum(0))) < 1e-6 * A[:, :3].sum()   # Newton's third law
    # perfect lattice: 56 neighbours, zero force, closed-form energy per particle
    pos, L = gen.jittered_lattice(10, 0.8, 0.0)
    out, A = _check_lj(tiga, pos, np.float32(2.5), np.full(3, L, np.float32), [1, 1, 1])
    assert np.max(np.abs(out[:, 3] - (-5.264771118950892))) < 2e-4
    # other eps / s, non-periodic
    pos = gen.uniform_points(2000, 3) * np.float32(12.0)
    keep = np.ones(len(pos), bool)
    d = np.linalg.norm(pos[:, None, :].astype(np.float64) - pos[None, :, :], axis=2) + np.eye(len(pos)) * 9
    keep[np.unique(np.nonzero(d < 0.7)[0])] = False          # no overlapping particles
    _check_lj(tiga, pos[keep], np.float32(2.0), np.full(3, 12.0, np.float32), [0, 0, 0], eps=1.5, s=0.8)


def test_lennard_jones_replica(tiga):
    c = gen.config("cfg3", m=40)          # 64,000 particles
    out, A = _check_lj(tiga, c["pos"], c["r"], c["box"], c["periodic"], use_cells=True)
    assert np.max(np.abs(out[:, :3].astype(np.float64).sum(0))) < 1e-6 * A[:, :3].sum()


def _separated_points(n, box, seed, dmin):
    """Uniform points in the box with no pair closer than dmin (Lennard-Jones inputs never overlap)."""
    pos = (gen.uniform_points(n, seed).astype(np.float64) * np.asarray(box, np.float64)).astype(np.float32)
    d = pos[:, None, :].astype(np.float64) - pos[None, :, :]
    d -= np.asarray(box, np.float64) * np.rint(d / np.asarray(box, np.float64))      # strictest reading: periodic in all
    dist = np.sqrt((d * d).sum(2)) + np.eye(n) * 1e9
    keep = np.ones(n, bool)
    for i in range(n):
        if keep[i]:
            keep[(dist[i] < dmin) & (np.arange(n) > i)] = False
    return pos[keep]


def _box_of(cells):
    return np.array([c * 1.05 + 0.3 for c in cells], np.float32)       # floor(len / (r (1 + 2^-10))) = cells at r = 1


# a periodic dimension must be longer than twice the cutoff: such combinations are left out
_SMALL_GRIDS = [(cells, per) for cells in [(1, 1, 1), (2, 2, 2), (3, 3, 3), (4, 3, 2), (1, 5, 3), (6, 1, 1), (3, 4, 1)]
                for per in [(0, 0, 0), (1, 1, 1), (1, 0, 1), (0, 1, 0)]
                if not any(p and b <= 2.0 for p, b in zip(per, _box_of(cells)))]


@pytest.mark.parametrize("cells,periodic", _SMALL_GRIDS)
def test_lennard_jones_small_grids(tiga, cells, periodic):
    """Every unordered pair must be visited exactly once whatever the grid: one, two or three
    cells per dimension, wrapped or clipped (a periodic dimension with fewer than three cells
    collapses to one cell with the explicit minimum image)."""
    r = np.float32(1.0)
    box = _box_of(cells)
    pos = _separated_points(600, box, 40 + sum(cells), 0.45)
    grid, _ = tiga.tiga_radius_grid(len(pos), r, box, list(periodic))
    expect = [1 if (p and c < 3) else c for c, p in zip(cells, periodic)]
    cap = int(round((8 * len(pos)) ** (1 / 3) - 0.5))
    assert list(grid) == [min(e, cap) for e in expect]
    out, A = _check_lj(tiga, pos, r, box, list(periodic), eps=0.7, s=0.5)
    assert np.max(np.abs(out[:, :3].astype(np.float64).sum(0))) < 1e-5 * max(A[:, :3].sum(), 1e-30)


def test_lennard_jones_dense_cells_span_several_stage_chunks(tiga):
    """Hundreds of points per cell: the cell's own points alone overflow the stage, so the half
    stencil is processed in several chunks and the own-cell rule (each pair once, by index) is
    applied across chunk borders."""
    box = np.array([6.0, 6.0, 6.0], np.float32)
    pos = _separated_points(2600, box, 77, 0.25)
    assert len(pos) > 1800
    # The pair force goes like d^-14 and the closest pairs (0.25 apart in cells of edge 3) dominate the
    # sums: a displacement formed from coordinates relative to a cell corner would carry an fp32
    # rounding of the CELL size and miss the tolerance here.  The kernel subtracts stored original
    # coordinates (periodic images by exact shifts), so the plain tolerance holds.
    for periodic in ([0, 0, 0], [1, 1, 1]):
        grid, _ = tiga.tiga_radius_grid(len(pos), np.float32(2.0), box, periodic)
        assert max(grid) <= 2
        _check_lj(tiga, pos, np.float32(2.0), box, periodic, eps=0.3, s=0.3)


def test_lennard_jones_rows_are_summed_by_atomics(tiga):
    """Two runs agree to rounding (the summation order of a row depends on scheduling) and the
    neighbour counts, being integers, agree exactly."""
    c = gen.config("cfg3", m=24)
    pd = dev(c["pos"], torch)
    a, ca, _ = tiga.tiga_apply_radius(pd, None, c["r"], c["box"], c["periodic"], tiga.MSG_LJ, p0=1.0, p1=1.0, want_count=True)
    b, cb, _ = tiga.tiga_apply_radius(pd, None, c["r"], c["box"], c["periodic"], tiga.MSG_LJ, p0=1.0, p1=1.0, want_count=True)
    assert torch.equal(ca, cb)
    y, A, cnt = oracle.radius_forward(c["pos"], None, c["r"], c["box"], c["periodic"], oracle.MSG_LJ, 1.0, 1.0, use_cells=True)
    assert np.max(np.abs(host(a).astype(np.float64) - host(b)) / A) <= 2 * SUM_TOL
    nocount, none, _ = tiga.tiga_apply_radius(pd, None, c["r"], c["box"], c["periodic"], tiga.MSG_LJ, p0=1.0, p1=1.0)
    assert none is None and rel_err(host(nocount), y, A) <= SUM_TOL


# ------------------------------------------------------------------------------ full size
def test_cfg2_full_size_sampled_rows(tiga):
    """1M points, periodic, F=32: 4096 sampled rows against all-pairs brute force, all rows
    against the oracle's cell-directory variant, plus global invariants."""
    c = gen.config("cfg2")
    n = c["n"]
    pd, xd, gyd = dev(c["pos"], torch), dev(c["x"], torch), dev(c["gy"], torch)
    out, count, ws = tiga.tiga_apply_radius(pd, xd, c["r"], c["box"], c["periodic"], tiga.MSG_GAUSS,
                                            p0=c["sigma"], want_count=True)
    gx, gp = tiga.tiga_apply_radius_backward(pd, xd, gyd, c["r"], c["box"], c["periodic"], c["sigma"], ws=ws, reuse_plan=True)
    out, count, gx, gp = host(out), host(count), host(gx), host(gp)
    rows = np.sort(gen.rng(1, 77).choice(n, 4096, replace=False))
    y, A, cnt = oracle.radius_forward(c["pos"], c["x"], c["r"], c["box"], c["periodic"], oracle.MSG_GAUSS,
                                      p0=c["sigma"], rows=rows)
    assert np.array_equal(count[rows], cnt)
    assert rel_err(out[rows], y, A) <= SUM_TOL
    b = oracle.radius_backward_gauss(c["pos"], c["x"], c["gy"], c["r"], c["box"], c["periodic"], c["sigma"], rows=rows)
    assert rel_err(gx[rows], b["gx"], b["Agx"]) <= GRAD_TOL
    assert rel_err(gp[rows], b["gp"], b["Agp"]) <= GRAD_TOL
    y, A, cnt = oracle.radius_forward(c["pos"], c["x"], c["r"], c["box"], c["periodic"], oracle.MSG_GAUSS,
                                      p0=c["sigma"], use_cells=True)
    assert np.array_equal(count, cnt) and count.sum() % 2 == 0
    assert rel_err(out, y, A) <= SUM_TOL
    assert abs(count.mean() - 32.0) < 0.1
    b = oracle.radius_backward_gauss(c["pos"], c["x"], c["gy"], c["r"], c["box"], c["periodic"], c["sigma"], use_cells=True)
    assert rel_err(gx, b["gx"], b["Agx"]) <= GRAD_TOL
    assert rel_err(gp, b["gp"], b["Agp"]) <= GRAD_TOL
    assert np.max(np.abs(gp.astype(np.float64).sum(0))) < 1e-5 * b["Agp"].sum()     # translation invariance


def test_cfg3_full_size(tiga):
    """160^3 = 4,096,000 jittered-lattice particles, periodic, cutoff 2.5: 2048 sampled rows against
    all-pairs brute force, every row against the oracle's cell-directory variant, and Newton's
    third law over the whole system."""
    c = gen.config("cfg3")
    n = c["n"]
    assert n == 4_096_000
    out, count, _ = tiga.tiga_apply_radius(dev(c["pos"], torch), None, c["r"], c["box"], c["periodic"], tiga.MSG_LJ,
                                           p0=1.0, p1=1.0, want_count=True)
    out, count = host(out), host(count)
    rows = np.sort(gen.rng(3, 78).choice(n, 2048, replace=False))
    y, A, cnt = oracle.radius_forward(c["pos"], None, c["r"], c["box"], c["periodic"], oracle.MSG_LJ, 1.0, 1.0, rows=rows)
    assert np.array_equal(count[rows], cnt)
    assert rel_err(out[rows], y, A) <= SUM_TOL
    y, A, cnt = oracle.radius_forward(c["pos"], None, c["r"], c["box"], c["periodic"], oracle.MSG_LJ, 1.0, 1.0, use_cells=True)
    assert np.array_equal(count, cnt) and count.sum() % 2 == 0
    assert rel_err(out, y, A) <= SUM_TOL
    assert 50 < count.mean() < 58
    assert np.max(np.abs(out[:, :3].astype(np.float64).sum(0))) < 1e-6 * A[:, :3].sum()


def test_sparse_periodic_box_pairs_at_the_cutoff_across_a_face(tiga):
    """Few points, small cutoff: the grid is capped (cells eleven times the cutoff), and pairs sit
    within a few ulps of r on both sides of it across the lower x face and inside the box.  The
    neighbour counts must equal the fp64 predicate's, pair by pair."""
    r = np.float32(0.01)
    ones = np.ones(3, np.float32)
    rows = []
    for k in range(24):
        y, z = np.float32(0.04 * k + 0.013), np.float32(0.9 - 0.031 * k)
        xa = np.float32(0.003 + 0.0001 * k)
        xb = np.float32(1.0) - (r - xa)                      # across the face, about r away
        xb = np.nextafter(xb, np.float32(2.0 if k % 2 else 0.0), dtype=np.float32)
        for _ in range(k % 5):
            xb = np.nextafter(xb, np.float32(2.0 if k % 2 else 0.0), dtype=np.float32)
        rows += [[xa, y, z], [xb, y, z]]
        xc = np.float32(0.4 + 0.01 * k)                      # the same inside the box
        xd = xc + r
        for _ in range(k % 4):
            xd = np.nextafter(xd, np.float32(2.0 if k % 2 else 0.0), dtype=np.float32)
        rows += [[xc, y, np.float32(z * 0.5)], [xd, y, np.float32(z * 0.5)]]
    pos = np.array(rows, np.float32)
    assert tiga.tiga_radius_grid(len(pos), float(r), ones, [1, 1, 1])[0][0] < 12      # capped grid
    x = gen.normal_features(len(pos), 8, 5)
    gy = gen.normal_features(len(pos), 8, 6)
    _, cnt = _check_gauss(tiga, pos, x, gy, r, ones, [1, 1, 1], float(r) / 2)
    c = host(cnt)
    assert 0 < c.sum() < len(pos)                            # some of the pairs are inside, some outside


# ------------------------------------------------------------------------------ validation
def test_point_validation(tiga):
    box = np.array([1.0, 2.0, 0.5], np.float32)
    pos = gen.uniform_points(10_000, 3) * box[None, :]
    pos[17] = box                                              # the upper faces belong to the box
    tiga.tiga_validate_points(dev(pos, torch), box)            # passes
    for bad in (np.float32(-1e-6), np.float32(np.nan), np.float32(np.inf), np.float32(0.5000001)):
        q = pos.copy()
        q[4321, 2] = bad
        with pytest.raises(tiga.TigaError) as e:
            tiga.tiga_validate_points(dev(q, torch), box)
        assert e.value.status == 7
        tiga.tiga_validate_points(dev(q, torch), box, level=0)     # metadata only: nothing is read
    tiga.tiga_validate_points(dev(pos[:0], torch), box)


# ------------------------------------------------------------------------------ uneven density
def test_clustered_points_are_spread_over_many_warps(tiga):
    """Most points in a dozen tight blobs: some cells hold hundreds of points (the cell's warp takes
    16 queries, the other slices of 16 wait in a queue that many warps walk).  Parity as usual, and the call must stay within
    5x of a uniform cloud with the same number of accepted pairs."""
    n, F = 200_000, 8
    pos = gen.clustered_points(n, 21)
    x = gen.normal_features(n, F, 21, 31); gy = gen.normal_features(n, F, 21, 32)
    ones = np.ones(3, np.float32)
    r = np.float32(0.01)
    grid, _ = tiga.tiga_radius_grid(n, r, ones, [0, 0, 0])
    cell = np.minimum((pos * np.float32(grid)).astype(np.int64), np.array(grid) - 1)
    occupancy = np.bincount((cell[:, 2] * grid[1] + cell[:, 1]) * grid[0] + cell[:, 0])
    assert occupancy.max() > 4 * 64                                   # several slices per cell
    out, count = _check_gauss(tiga, pos, x, gy, r, ones, [0, 0, 0], np.float32(0.005), use_cells=True)
    pairs = int(host(count).sum())
    # Lennard-Jones on the same cloud (scaled): the length s lies below the smallest distance of any pair, so no pair
    # energy is a difference of two nearly equal powers (the normalisation by |contributions| would not cover that)
    # (cutoff 0.8: a few dozen neighbours per particle as in the workload, while the cells -- their number is capped
    # by the point count -- still hold hundreds of points; rows of a thousand atomically added terms would exceed
    # what fp32 accumulation in arbitrary order can promise)
    _check_lj(tiga, pos * np.float32(300.0), np.float32(0.8), np.full(3, 300.0, np.float32), [0, 0, 0], eps=1e-3, s=0.005, use_cells=True)

    def timed(p, rr):
        pd, xd = dev(p, torch), dev(x, torch)
        o, c, ws = tiga.tiga_apply_radius(pd, xd, rr, ones, [0, 0, 0], tiga.MSG_GAUSS, p0=float(rr) / 2, want_count=True)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(5):
            tiga.tiga_apply_radius(pd, xd, rr, ones, [0, 0, 0], tiga.MSG_GAUSS, p0=float(rr) / 2, out=o, count=c, ws=ws)
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / 5, int(c.sum().item())

    r_uniform = np.float32((pairs * 3.0 / (4.0 * np.pi * n * n)) ** (1.0 / 3.0))
    t_c, p_c = timed(pos, r)
    t_u, p_u = timed(gen.uniform_points(n, 22), r_uniform)
    print(f"clustered: {p_c} pairs in {t_c:.3f} ms; uniform: {p_u} pairs in {t_u:.3f} ms")
    assert 0.7 * p_c < p_u < 1.4 * p_c
    assert t_c < 5.0 * t_u
