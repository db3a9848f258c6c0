"""GPU parity of the hot-source plan of a stored relation and of the planned forward.

The plan is unique (sources above an in-degree threshold, numbered in source order), so its arrays
are compared bit for bit with a numpy restatement.  The planned forward visits the edges in the same
order as the plain one: it must equal tiga_apply_csr bit for bit and the fp64 oracle within the
usual tolerances (1e-5 of the sum of absolute contributions; maxima and argmax exactly)."""
import numpy as np
import pytest

import gen
import oracle
from parity import SUM_TOL, Guard, dev, host, rel_err

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tiga():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2609_24802_b200 import api
    return api


def _reference_plan(col, n_src, max_hot):
    indeg = np.bincount(col, minlength=n_src)
    capped = np.minimum(indeg, 4095)
    thr, n_hot = None, 0
    for d in range(4095, 0, -1):
        k = int((capped == d).sum())
        if n_hot + k > max_hot:
            break
        n_hot += k
        thr = d
    hot = indeg >= thr if thr is not None else np.zeros(n_src, bool)
    hot_id = np.nonzero(hot)[0].astype(np.int32)
    remap = np.where(hot, np.cumsum(hot) - 1, len(hot_id) + np.arange(n_src))
    return dict(n_hot=len(hot_id), thr=(thr or 0) if len(hot_id) else 0, hot_id=hot_id, col=remap[col].astype(np.int32), hot_edges=int(indeg[hot].sum()))


def _check(tiga, rowptr, col, x, w, max_hot, index64=False, reducers=(0, 1)):
    n_src = x.shape[0]
    rp = dev(rowptr.astype(np.int64 if index64 else np.int32), torch)
    g = tiga.CsrRelation(rp, dev(col.astype(np.int32), torch), n_src)
    plan = tiga.tiga_csr_plan_build(g, max_hot_rows=max_hot)
    ref = _reference_plan(col, n_src, max_hot)
    assert plan.n_hot == ref["n_hot"] <= max_hot and plan.min_hot_degree == ref["thr"] and plan.hot_edges == ref["hot_edges"]
    assert np.array_equal(host(plan.array("hot_id")), ref["hot_id"])
    assert np.array_equal(host(plan.array("col")), ref["col"])
    xd = dev(x, torch)
    wd = None if w is None else dev(w, torch)
    F = x.shape[1]
    dt = tiga.F16 if x.dtype == np.float16 else tiga.F32
    for red in reducers:
        y, A, arg = oracle.csr_forward(rowptr, col, x, w, red)
        guard = Guard(torch)
        ws = guard.workspace(tiga.tiga_csr_planned_workspace_bytes(plan, F, dt, red))
        out, am = tiga.tiga_apply_csr_planned(plan, xd, wd, red, out=guard.empty((len(rowptr) - 1, F)),
                                              argmax=guard.empty((len(rowptr) - 1, F), torch.int32) if red else None, ws=ws)
        guard.check()
        plain, plain_am = tiga.tiga_apply_csr(g, xd, wd, red)
        torch.cuda.synchronize()
        assert torch.equal(out, plain), "the plan must not change a single bit of the result"
        if red == tiga.SUM:
            assert rel_err(host(out), y, A) <= SUM_TOL
        else:
            assert np.array_equal(host(out), y.astype(np.float32)) and np.array_equal(host(am).astype(np.int64), arg)
            assert torch.equal(am, plain_am)
    return plan


@pytest.mark.parametrize("max_hot", [0, 50, 1000, 100_000])
@pytest.mark.parametrize("dtype,F", [(np.float16, 8), (np.float32, 4), (np.float32, 8), (np.float16, 16)])
def test_skewed_random_graph(tiga, max_hot, dtype, F):
    g0 = gen.rng(5 + F, 901)
    n_dst, n_src = 5000, 7000
    deg = g0.integers(0, 30, size=n_dst)
    deg[g0.random(n_dst) < 0.4] = 0
    deg[321] = 40_000                 # cut into chunks of 8192 edges
    deg[4000] = 700
    rowptr = np.concatenate([[0], np.cumsum(deg)]).astype(np.int64)
    E = int(rowptr[-1])
    # a few sources are named very often, most rarely or never
    col = np.where(g0.random(E) < 0.6, g0.integers(0, 40, size=E), g0.integers(0, n_src, size=E)).astype(np.int32)
    x = gen.normal_features(n_src, F, 5, 31, dtype)
    w = gen.edge_weights(E, 5) if F == 4 else None
    plan = _check(tiga, rowptr, col, x, w, max_hot)
    if max_hot == 50:
        assert 0 < plan.n_hot <= 50 and plan.hot_edges > 0.5 * E


def test_rmat_with_int64_row_pointers(tiga):
    c = gen.config("cfg4", 7, scale=18)
    plan = _check(tiga, c["rowptr"], c["col"], c["x"], None, c["n"] // 16, index64=True, reducers=(0,))
    assert plan.hot_edges > 0.75 * c["E"]          # a sixteenth of the sources is named by most edges


def test_unsupported_and_bad_arguments(tiga):
    rowptr = np.array([0, 2, 2, 3], np.int64)
    col = np.array([0, 2, 0], np.int32)
    g = tiga.CsrRelation(dev(rowptr.astype(np.int32), torch), dev(col, torch), 3)
    plan = tiga.tiga_csr_plan_build(g, max_hot_rows=1)
    assert plan.n_hot == 1 and host(plan.array("hot_id")).tolist() == [0] and host(plan.array("col")).tolist() == [0, 3, 0]
    x = torch.ones((3, 64), device="cuda")
    with pytest.raises(tiga.TigaError) as e:
        tiga.tiga_apply_csr_planned(plan, x)                       # 256-byte rows: not what the plan is for
    assert e.value.status == 2
    x = torch.arange(12, device="cuda", dtype=torch.float32).reshape(3, 4)
    out, _ = tiga.tiga_apply_csr_planned(plan, x)
    assert host(out)[:, 0].tolist() == [8.0, 0.0, 0.0]
    other = tiga.CsrRelation(dev(np.array([0, 1], np.int32), torch), dev(np.array([0], np.int32), torch), 3)
    plan.g = other                                                 # a plan is tied to the relation it was built for
    with pytest.raises(tiga.TigaError) as e:
        tiga.tiga_apply_csr_planned(plan, x)
    assert e.value.status == 1
