"""GPU parity of the generated exact kNN relation with neighbour sum (paper Section 4.9) against the
oracle: neighbour indices and key distances bit-exact (both sides form the key in fp32 by direct
differences in the same operation order), neighbour sums within 1e-5 of the sum of absolute
contributions."""
import numpy as np
import pytest

import gen
import oracle
from parity import SUM_TOL, Guard, dev, host, rel_err

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

UNIT = np.ones(3, np.float32)


@pytest.fixture(scope="module")
def tiga():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2609_24802_b200 import api
    return api


def _check(tiga, pos, x, k, box=UNIT, rows=None):
    guard = Guard(torch)
    n, F = x.shape
    out, nbr, d2, _ = tiga.tiga_apply_knn(dev(pos, torch), dev(x, torch), k, box, out=guard.empty((n, F)),
                                          nbr=guard.empty((n, k), torch.int32), nbr_d2=guard.empty((n, k)),
                                          ws=guard.workspace(tiga.tiga_knn_workspace_bytes(n, k, box)))
    guard.check()
    idx, rd2, y, A = oracle.knn(pos, x, k, rows=rows)
    sel = slice(None) if rows is None else np.asarray(rows)
    assert np.array_equal(host(nbr)[sel], idx), "neighbour indices must be bit exact, in key order"
    assert np.array_equal(host(d2)[sel], rd2), "key distances must be bit exact"
    assert rel_err(host(out)[sel], y, A) <= SUM_TOL
    return out


@pytest.mark.parametrize("k,F", [(16, 1), (1, 1), (5, 3), (16, 8), (32, 32), (7, 40)])
def test_uniform_cloud(tiga, k, F):
    n = 6000
    _check(tiga, gen.uniform_points(n, 90 + k), gen.normal_features(n, F, 91, 31), k)


def test_uneven_density_uses_shells_and_list_cuts(tiga):
    n = 30000
    pos = gen.clustered_points(n, 5)
    _check(tiga, pos, gen.normal_features(n, 1, 92, 31), 16)
    _check(tiga, pos, gen.normal_features(n, 4, 92, 31), 32)


@pytest.mark.parametrize("cloud", ["uniform", "clustered"])
def test_selection_agrees_with_exact_geometry(tiga, cloud):
    """Independent of the oracle's fp32 key: in exact (fp64) geometry every selected neighbour is at
    least as near as every point left out, up to the rounding of the fp32 key (relative 1e-6), for
    every query; no self, no duplicates, keys in non-decreasing order."""
    n, k = 6000, 16
    pos = gen.uniform_points(n, 97) if cloud == "uniform" else gen.clustered_points(n, 98)
    x = gen.normal_features(n, 1, 99, 31)
    _, nbr, d2, _ = tiga.tiga_apply_knn(dev(pos, torch), dev(x, torch), k, UNIT)
    nbr, d2 = host(nbr).astype(np.int64), host(d2)
    p64 = pos.astype(np.float64)
    assert np.all(np.diff(d2, axis=1) >= 0)
    for lo in range(0, n, 1000):
        q = p64[lo:lo + 1000]
        D = ((q[:, None, :] - p64[None, :, :]) ** 2).sum(-1)            # exact squared distances (fp64 of fp32 inputs)
        rows = np.arange(len(q))
        D[rows, lo + rows] = np.inf                                       # a point is not its own neighbour
        sel = nbr[lo:lo + 1000]
        assert np.all(sel != (lo + rows)[:, None])
        assert all(len(set(r)) == k for r in sel)
        far_in = np.take_along_axis(D, sel, 1).max(1)
        Dout = D.copy()
        np.put_along_axis(Dout, sel, np.inf, 1)
        near_out = Dout.min(1)
        assert np.all(far_in <= near_out * (1 + 1e-6) + 1e-300)
        # the reported keys are the exact squared distances rounded like an fp32 evaluation
        exact = np.take_along_axis(D, sel, 1)
        assert np.all(np.abs(d2[lo:lo + 1000] - exact) <= 1e-6 * exact + 1e-30)


def test_points_on_a_surface(tiga):
    n = 35947
    _check(tiga, gen.surface_points(n, 3), gen.normal_features(n, 1, 93, 31), 16)


@pytest.mark.parametrize("k", [4, 6, 18, 26])
def test_lattice_ties_by_index(tiga, k):
    m = 12
    g = np.arange(m, dtype=np.float32) / 16
    z, y, x = np.meshgrid(g, g, g, indexing="ij")
    pos = np.stack([x.ravel(), y.ravel(), z.ravel()], 1).astype(np.float32)
    out = _check(tiga, pos, np.ones((m ** 3, 2), np.float32), k)
    assert torch.all(out == float(k))


def test_coincident_points(tiga):
    pos = np.full((300, 3), 0.375, np.float32)
    pos[200:] = gen.uniform_points(100, 4)
    _check(tiga, pos, gen.normal_features(300, 2, 94, 31), 16)


@pytest.mark.parametrize("n", [1, 2, 5, 16, 17, 18, 40])
def test_fewer_points_than_k(tiga, n):
    out = _check(tiga, gen.uniform_points(n, 6), gen.normal_features(n, 3, 95, 31), 16)
    assert out.shape == (n, 3)


def test_empty_input(tiga):
    pos = torch.empty((0, 3), device="cuda")
    out, nbr, d2, _ = tiga.tiga_apply_knn(pos, torch.empty((0, 2), device="cuda"), 4, UNIT)
    assert out.shape == (0, 2) and nbr.shape == (0, 4)


def test_flat_slab_and_long_box(tiga):
    n = 20000
    pos = gen.uniform_points(n, 7)
    box = np.array([4.0, 1.0, 0.05], np.float32)
    pos = (pos * box).astype(np.float32)
    _check(tiga, pos, gen.normal_features(n, 1, 96, 31), 16, box=box)


def test_rejects_what_it_does_not_support(tiga):
    pos = dev(gen.uniform_points(100, 8), torch)
    x = dev(gen.normal_features(100, 1, 97, 31), torch)
    for kwargs, status in ((dict(k=33), 2), (dict(k=0), 1)):
        with pytest.raises(tiga.TigaError) as e:
            tiga.tiga_apply_knn(pos, x, kwargs["k"], UNIT)
        assert e.value.status == status
    with pytest.raises(tiga.TigaError) as e:
        tiga.tiga_apply_knn(pos, x, 4, UNIT, periodic=(1, 0, 0))
    assert e.value.status == 2
    with pytest.raises(tiga.TigaError) as e:
        tiga.tiga_apply_knn(pos, x, 4, UNIT, ws=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 3


def test_paper_size_131072_points(tiga):
    # the largest size the paper reports for this relation: scalar neighbour sum, k = 16
    n = 131072
    pos = gen.uniform_points(n, 9)
    x = gen.normal_features(n, 1, 98, 31)
    rows = np.sort(gen.rng(9, 99).choice(n, 8192, replace=False))
    _check(tiga, pos, x, 16, rows=rows)
    out, nbr, _, _ = tiga.tiga_apply_knn(dev(pos, torch), dev(x, torch), 16, UNIT)
    nb = host(nbr)
    assert nb.min() >= 0 and np.all(nb != np.arange(n)[:, None])
    assert np.all(np.sort(nb, 1)[:, 1:] != np.sort(nb, 1)[:, :-1])          # k distinct neighbours per row
    assert np.allclose(host(out)[:, 0], x[nb, 0].sum(1), rtol=1e-4, atol=1e-4)
