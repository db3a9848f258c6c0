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
