"""GPU parity: the CUDA CSR traversal (through the C ABI) against the fp64 CPU oracle, element
by element on the same seeded inputs.  Integers and max outputs must match bit-exactly, sums
within 1e-5 and gradients within 1e-4 of the sum of absolute contributions."""
import numpy as np
import pytest

import gen
import oracle
from conftest import read_golden
from parity import GRAD_TOL, SUM_TOL, Guard, dev, host, rel_err

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tiga():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2609_24802_b200 import api
    return api


def _relation(tiga, rowptr, col, n_src, index64=False):
    rp = dev(rowptr.astype(np.int64 if index64 else np.int32), torch)
    return tiga.CsrRelation(rp, dev(col.astype(np.int32), torch), n_src)


def _check_forward(tiga, rowptr, col, x, w, index64=False, reducers=(0, 1)):
    g = _relation(tiga, rowptr, col, x.shape[0], index64)
    xd = dev(x, torch)
    wd = None if w is None else dev(w, torch)
    res = {}
    for red in reducers:
        y, A, arg = oracle.csr_forward(rowptr, col, x, w, red)
        guard = Guard(torch)
        F = x.shape[1]
        ws = guard.workspace(tiga.tiga_csr_workspace_bytes(g, F, tiga.F16 if xd.dtype == torch.float16 else tiga.F32, red))
        out, am = tiga.tiga_apply_csr(g, xd, wd, red, out=guard.empty((g.n_dst, F)),
                                      argmax=guard.empty((g.n_dst, F), torch.int32) if red == tiga.MAX else None, ws=ws)
        guard.check()
        out2, am2 = tiga.tiga_apply_csr(g, xd, wd, red)
        torch.cuda.synchronize()
        assert torch.equal(out, out2), "forward must be reproducible run to run"
        if red == tiga.SUM:
            assert rel_err(host(out), y, A) <= SUM_TOL
        else:
            assert np.array_equal(host(out), y.astype(np.float32)), "max outputs must be bit exact"
            assert np.array_equal(host(am).astype(np.int64), arg), "argmax must be bit exact"
            assert torch.equal(am, am2)
            # the same reducer with 64-bit edge positions: same values, same positions, wider array
            ws64 = guard.workspace(tiga.tiga_csr_workspace_bytes(g, F, tiga.F16 if xd.dtype == torch.float16 else tiga.F32, tiga.MAX64))
            out64, am64 = tiga.tiga_apply_csr(g, xd, wd, tiga.MAX64, out=guard.empty((g.n_dst, F)),
                                              argmax=guard.empty((g.n_dst, F), torch.int64), ws=ws64)
            guard.check()
            assert am64.dtype == torch.int64 and torch.equal(out64, out) and torch.equal(am64, am.long())
            res["arg64"] = am64
        res[red] = (out, am)
    return g, xd, wd, res


def _check_backward(tiga, rowptr, col, x, w, gy, g, xd, wd, res):
    gyd = dev(gy, torch)
    ref = oracle.csr_backward_sum(rowptr, col, x, w, gy)
    guard = Guard(torch)
    gx, gw = tiga.tiga_apply_csr_backward(g, xd, wd, gyd, tiga.SUM, grad_x=guard.empty((g.n_src, x.shape[1])),
                                          grad_w=guard.empty((g.n_edges,)))
    guard.check()
    assert rel_err(host(gx), ref["gx"], ref["Ax"]) <= GRAD_TOL
    assert rel_err(host(gw), ref["gw"], ref["Aw"]) <= GRAD_TOL
    only_x, none_w = tiga.tiga_apply_csr_backward(g, xd, wd, gyd, tiga.SUM, want_w=False)
    assert none_w is None and rel_err(host(only_x), ref["gx"], ref["Ax"]) <= GRAD_TOL
    if 1 in res:
        am = res[1][1]
        _, _, arg = oracle.csr_forward(rowptr, col, x, w, oracle.MAX)
        refm = oracle.csr_backward_max(rowptr, col, x, w, gy, arg)
        gx, gw = tiga.tiga_apply_csr_backward(g, xd, wd, gyd, tiga.MAX, argmax=am, grad_x=guard.empty((g.n_src, x.shape[1])),
                                              grad_w=guard.empty((g.n_edges,)))
        guard.check()
        assert rel_err(host(gx), refm["gx"], refm["Ax"]) <= GRAD_TOL
        assert rel_err(host(gw), refm["gw"], refm["Aw"]) <= GRAD_TOL
        gx, gw = tiga.tiga_apply_csr_backward(g, xd, wd, gyd, tiga.MAX64, argmax=res["arg64"], grad_x=guard.empty((g.n_src, x.shape[1])),
                                              grad_w=guard.empty((g.n_edges,)))
        guard.check()
        assert rel_err(host(gx), refm["gx"], refm["Ax"]) <= GRAD_TOL
        assert rel_err(host(gw), refm["gw"], refm["Aw"]) <= GRAD_TOL


def _random_graph(seed, n_dst, n_src, max_deg, F, p_empty=0.3):
    g = gen.rng(seed, 700)
    deg = g.integers(0, max_deg + 1, size=n_dst)
    deg[g.random(n_dst) < p_empty] = 0
    rowptr = np.concatenate([[0], np.cumsum(deg)]).astype(np.int64)
    E = int(rowptr[-1])
    col = g.integers(0, n_src, size=E).astype(np.int32)
    x = g.standard_normal((n_src, F)).astype(np.float32)
    w = ((g.integers(0, 2**24 - 1, size=E) + 1) * 2.0**-24).astype(np.float32)
    gy = g.standard_normal((n_dst, F)).astype(np.float32)
    return rowptr, col, x, w, gy


def test_printed_worked_example(tiga):
    gd = read_golden("csr_worked_example.txt")
    rowptr = np.array(gd["rowptr"], np.int64)
    col = np.array(gd["col"], np.int32)
    x = np.repeat(np.array(gd["x"], np.float32)[:, None], 4, axis=1)
    w = np.array(gd["w"], np.float32)
    g, xd, wd, res = _check_forward(tiga, rowptr, col, x, w)
    assert host(res[0][0])[:, 0].tolist() == gd["y"]
    gx, gw = tiga.tiga_apply_csr_backward(g, xd, wd, torch.ones((3, 4), device="cuda"), tiga.SUM)
    assert host(gx)[:, 0].tolist() == gd["dx"]
    assert host(gw).tolist() == [4 * v for v in gd["dw"]]      # four identical feature columns


@pytest.mark.parametrize("F", [4, 8, 12, 16, 32, 64, 100, 128, 160, 256, 512])
def test_random_graphs_all_widths(tiga, F):
    rowptr, col, x, w, gy = _random_graph(F, n_dst=3000, n_src=1000, max_deg=40, F=F)
    g, xd, wd, res = _check_forward(tiga, rowptr, col, x, w)
    _check_backward(tiga, rowptr, col, x, w, gy, g, xd, wd, res)


def test_unit_weights_and_duplicates(tiga):
    rowptr, col, x, _, gy = _random_graph(77, n_dst=500, n_src=5, max_deg=30, F=16)   # 5 sources: many duplicates and ties
    g, xd, wd, res = _check_forward(tiga, rowptr, col, x, None)
    _check_backward(tiga, rowptr, col, x, None, gy, g, xd, wd, res)
    # integer-valued features make ties frequent: the lowest edge position must win
    xi = gen.small_int_features(5, 16, 3)
    _check_forward(tiga, rowptr, col, xi, None)


def test_degenerate_shapes(tiga):
    F = 8
    x = gen.normal_features(7, F, 1)
    # no edges at all; one row; one huge row between empty ones; last row heavy
    for rowptr in ([0, 0, 0, 0, 0], [0, 0], [0, 3], [0, 0, 30000, 30000], [0, 5, 5, 9000]):
        rowptr = np.array(rowptr, np.int64)
        E = int(rowptr[-1])
        col = gen.rng(E, 5).integers(0, 7, size=E).astype(np.int32)
        w = gen.edge_weights(E, 2) if E else np.zeros(0, np.float32)
        g, xd, wd, res = _check_forward(tiga, rowptr, col, x, w if E else None)
        gy = gen.normal_features(len(rowptr) - 1, F, 2, 32)
        _check_backward(tiga, rowptr, col, x, w if E else None, gy, g, xd, wd, res)
    # a long run of empty rows (more rows than one tile holds) around a few edges
    rowptr = np.zeros(10001, np.int64)
    rowptr[5000:] = 3
    rowptr[9000:] = 7
    col = np.array([0, 1, 2, 3, 4, 5, 6], np.int32)
    _check_forward(tiga, rowptr, col, x, gen.edge_weights(7, 3))


def test_heavy_rows_span_many_tiles(tiga):
    rowptr, col = gen.rmat_csr(14, 16 << 14, seed=3)
    n = 1 << 14
    assert np.diff(rowptr).max() > 2 * 2048
    x = gen.normal_features(n, 64, 3)
    w = gen.edge_weights(16 << 14, 3)
    gy = gen.normal_features(n, 64, 3, 32)
    g, xd, wd, res = _check_forward(tiga, rowptr, col, x, w)
    _check_backward(tiga, rowptr, col, x, w, gy, g, xd, wd, res)


def test_fp16_features_backward(tiga):
    """Backward with an fp16 feature table: the oracle sees the same (exactly representable) values."""
    for seed, n_dst, n_src, max_deg, F in [(31, 700, 300, 40, 8), (32, 300, 900, 70, 64), (33, 50, 20, 3000, 16)]:
        rowptr, col, x, w, gy = _random_graph(seed, n_dst, n_src, max_deg, F)
        x16 = x.astype(np.float16)
        xr = x16.astype(np.float32)
        g = _relation(tiga, rowptr, col, n_src)
        xd, wd, gyd = dev(x16, torch), dev(w, torch), dev(gy, torch)
        ref = oracle.csr_backward_sum(rowptr, col, xr, w, gy)
        guard = Guard(torch)
        gx, gw = tiga.tiga_apply_csr_backward(g, xd, wd, gyd, tiga.SUM, grad_x=guard.empty((n_src, F)), grad_w=guard.empty((g.n_edges,)))
        guard.check()
        assert gx.dtype == torch.float32
        assert rel_err(host(gx), ref["gx"], ref["Ax"]) <= GRAD_TOL
        assert rel_err(host(gw), ref["gw"], ref["Aw"]) <= GRAD_TOL
        _, _, arg = oracle.csr_forward(rowptr, col, xr, w, oracle.MAX)
        refm = oracle.csr_backward_max(rowptr, col, xr, w, gy, arg)
        y, am = tiga.tiga_apply_csr(g, xd, wd, tiga.MAX)
        assert np.array_equal(host(am), arg)
        gx, gw = tiga.tiga_apply_csr_backward(g, xd, wd, gyd, tiga.MAX, argmax=am, grad_x=guard.empty((n_src, F)),
                                              grad_w=guard.empty((g.n_edges,)))
        guard.check()
        assert rel_err(host(gx), refm["gx"], refm["Ax"]) <= GRAD_TOL
        assert rel_err(host(gw), refm["gw"], refm["Aw"]) <= GRAD_TOL


def test_max_backward_with_a_gradient_table_larger_than_l2(tiga):
    """The max backward has two forms, picked by the size of the feature-gradient table (128 MB): this
    relation has few edges but 600,000 sources of 64 features, so the four-features-per-thread form
    runs, with fp32 and fp16 features, 32-bit and 64-bit edge positions."""
    n_dst, n_src, F = 3000, 600_000, 64
    rowptr, col, x, w, gy = _random_graph(91, n_dst, n_src, 40, F)
    g = _relation(tiga, rowptr, col, n_src)
    wd, gyd = dev(w, torch), dev(gy, torch)
    for xt in (x, x.astype(np.float16)):
        xr = xt.astype(np.float32)
        xd = dev(xt, torch)
        _, _, arg = oracle.csr_forward(rowptr, col, xr, w, oracle.MAX)
        ref = oracle.csr_backward_max(rowptr, col, xr, w, gy, arg)
        for red, dt in ((tiga.MAX, torch.int32), (tiga.MAX64, torch.int64)):
            _, am = tiga.tiga_apply_csr(g, xd, wd, red)
            assert am.dtype == dt and np.array_equal(host(am).astype(np.int64), arg)
            guard = Guard(torch)
            gx, gw = tiga.tiga_apply_csr_backward(g, xd, wd, gyd, red, argmax=am, grad_x=guard.empty((n_src, F)),
                                                  grad_w=guard.empty((g.n_edges,)))
            guard.check()
            assert rel_err(host(gx), ref["gx"], ref["Ax"]) <= GRAD_TOL
            assert rel_err(host(gw), ref["gw"], ref["Aw"]) <= GRAD_TOL


def test_hex_mesh_degrees(tiga):
    L = 24
    rowptr, col = gen.hex_mesh_csr(L)
    ones = np.ones((L ** 3, 16), np.float32)
    g = _relation(tiga, rowptr, col, L ** 3)
    out, _ = tiga.tiga_apply_csr(g, dev(ones, torch), None, tiga.SUM)
    deg = np.diff(rowptr).astype(np.float32)
    assert np.array_equal(host(out), np.repeat(deg[:, None], 16, axis=1))
    assert deg.max() == read_golden("hex_mesh_counts.txt")["interior_degree"][0]


def test_periodic_closed_form_is_bit_exact(tiga):
    n, F = 1 << 16, 32
    offs = [1, 2, 3, 5, 8, 13, 21, 34, -1, -2, -3, -5, -8, -13, -21, -34]
    rowptr, col = gen.periodic_offset_csr(n, offs)
    x = gen.small_int_features(n, F, 4)
    w = gen.small_int_weights(16 * n, 4)
    g = _relation(tiga, rowptr, col, n)
    out, _ = tiga.tiga_apply_csr(g, dev(x, torch), dev(w, torch), tiga.SUM)
    ref = np.zeros((n, F))
    for k, o in enumerate(offs):
        ref += w[k::16, None].astype(np.float64) * np.roll(x.astype(np.float64), -o, axis=0)
    assert np.array_equal(host(out).astype(np.float64), ref)


def test_fp16_features_int64_rowptr(tiga):
    c = gen.config("cfg4", scale=15)
    assert c["x"].dtype == np.float16 and c["rowptr"].dtype == np.int64
    _check_forward(tiga, c["rowptr"], c["col"], c["x"], None, index64=True)
    for F in (16, 64, 264):
        x = gen.normal_features(1 << 15, F, 8, dtype=np.float16)
        w = gen.edge_weights(c["E"], 8)
        _check_forward(tiga, c["rowptr"], c["col"], x, w, index64=True)


def test_degree_histogram_is_bit_exact(tiga):
    for scale, index64 in ((12, False), (16, True)):
        rowptr, col = gen.rmat_csr(scale, 16 << scale, seed=9)
        g = _relation(tiga, rowptr, col, 1 << scale, index64)
        for nbins in (4096, 8, 1):
            hist, mx = tiga.tiga_csr_degree_histogram(g, nbins)
            ref, rmx = oracle.degree_histogram(rowptr, nbins)
            assert np.array_equal(host(hist), ref) and int(host(mx)[0]) == rmx
        hist, _ = tiga.tiga_csr_degree_histogram(g, 8192)
        h = host(hist)
        if h[-1] == 0:
            assert int(np.sum(np.arange(8192) * h)) == int(rowptr[-1])     # degree sums equal E


def test_full_validation_finds_malformed_relations(tiga):
    rowptr, col = gen.rmat_csr(10, 16 << 10, seed=1)
    n = 1 << 10
    tiga.tiga_validate_csr(_relation(tiga, rowptr, col, n), 1)
    bad = rowptr.copy(); bad[100], bad[101] = bad[101] + 5, bad[100]          # not monotone
    cases = [(bad, col, n)]
    bad = rowptr.copy(); bad[0] = 1
    cases.append((bad, col, n))                                                # does not start at 0
    bad = rowptr.copy(); bad[-1] -= 1
    cases.append((bad, col, n))                                                # endpoint != E
    badc = col.copy(); badc[17] = n
    cases.append((rowptr, badc, n))                                            # source out of range
    badc = col.copy(); badc[5] = -1
    cases.append((rowptr, badc, n))
    for rp, cc, ns in cases:
        with pytest.raises(tiga.TigaError) as ei:
            tiga.tiga_validate_csr(_relation(tiga, rp, cc, ns), 1)
        assert ei.value.status == 5
    torch.cuda.synchronize()


def test_cfg1_full_size(tiga):
    """R-MAT scale 20, 16.8M edges, F=64: every output element against the oracle."""
    c = gen.config("cfg1")
    g, xd, wd, res = _check_forward(tiga, c["rowptr"], c["col"], c["x"], c["w"])
    _check_backward(tiga, c["rowptr"], c["col"], c["x"], c["w"], c["gy"], g, xd, wd, res)
    hist, mx = tiga.tiga_csr_degree_histogram(g, 4096)
    ref, rmx = oracle.degree_histogram(c["rowptr"], 4096)
    assert np.array_equal(host(hist), ref) and int(host(mx)[0]) == rmx


def test_cfg4_full_size(tiga):
    """R-MAT scale 26, 2^30 edges, int64 rowptr, F=8 fp16 features, unit weights, fp32 output:
    every output element against the oracle, and the degree histogram bit-exactly."""
    c = gen.config("cfg4")
    assert c["E"] == 1 << 30 and c["rowptr"].dtype == np.int64
    g = _relation(tiga, c["rowptr"], c["col"], c["n"], index64=True)
    xd = dev(c["x"], torch)
    out, _ = tiga.tiga_apply_csr(g, xd, None, tiga.SUM)
    hist, mx = tiga.tiga_csr_degree_histogram(g, 4096)
    torch.cuda.synchronize()
    out = host(out)
    ref, rmx = oracle.degree_histogram(c["rowptr"], 4096)
    assert np.array_equal(host(hist), ref) and int(host(mx)[0]) == rmx
    y, A, _ = oracle.csr_forward(c["rowptr"], c["col"], c["x"], None, oracle.SUM)
    assert rel_err(out, y, A) <= SUM_TOL
    # the same forward through the hot-source plan: bit-identical
    plan = tiga.tiga_csr_plan_build(g, row_bytes=16)
    assert plan.hot_edges > 0.8 * c["E"]
    planned, _ = tiga.tiga_apply_csr_planned(plan, xd)
    torch.cuda.synchronize()
    assert np.array_equal(host(planned), out)


def _sample_rows_check(tiga, rowptr_h, cold, wd, x, rows, out, arg64, gy=None, gw=None, reducer="sum"):
    """Oracle check of a sample of rows of a relation too large for the oracle as a whole: the rows'
    edges are copied to the host and form a small relation of their own."""
    deg = (rowptr_h[rows + 1] - rowptr_h[rows]).astype(np.int64)
    rp = np.concatenate([[0], np.cumsum(deg)]).astype(np.int64)
    col = np.concatenate([host(cold[int(rowptr_h[r]):int(rowptr_h[r + 1])]) for r in rows]).astype(np.int32)
    w = None if wd is None else np.concatenate([host(wd[int(rowptr_h[r]):int(rowptr_h[r + 1])]) for r in rows]).astype(np.float32)
    rows_t = torch.from_numpy(rows).cuda()
    if reducer == "sum":
        y, A, _ = oracle.csr_forward(rp, col, x, w, oracle.SUM)
        assert rel_err(host(out[rows_t]), y, A) <= SUM_TOL
        if gw is not None:
            ref = oracle.csr_backward_sum(rp, col, x, w, host(gy[rows_t]))
            got = np.concatenate([host(gw[int(rowptr_h[r]):int(rowptr_h[r + 1])]) for r in rows])
            assert rel_err(got, ref["gw"], ref["Aw"]) <= GRAD_TOL
        return
    y, _, arg = oracle.csr_forward(rp, col, x, w, oracle.MAX)
    assert np.array_equal(host(out[rows_t]), y.astype(np.float32))
    shift = (rowptr_h[rows] - rp[:-1])[:, None]                    # sample position -> position in the full relation
    assert np.array_equal(host(arg64[rows_t]), np.where(arg >= 0, arg + shift, -1))
    if gw is not None:
        ref = oracle.csr_backward_max(rp, col, x, w, host(gy[rows_t]), arg)
        got = np.concatenate([host(gw[int(rowptr_h[r]):int(rowptr_h[r + 1])]) for r in rows])
        assert rel_err(got, ref["gw"], ref["Aw"]) <= GRAD_TOL


@pytest.mark.parametrize("F", [4, 16])
def test_relation_with_more_than_2_31_edges(tiga, F):
    """2^31 edges and more: 64-bit row offsets, 64-bit edge positions in argmax (TIGA_MAX64; the
    32-bit reducer refuses), narrow (F = 4) and wide (F = 16) feature rows.  Sampled rows — the first
    and last, the rows around edge 2^31, the longest — are checked completely against the oracle."""
    n_dst, n_src = (1 << 20) + (1 << 15), 4096
    rs = gen.rng(41, 900)
    deg = rs.integers(0, 4099, size=n_dst).astype(np.int64)
    deg[rs.random(n_dst) < 0.02] = 0
    deg[[5, 77_777, n_dst - 1]] = [20_000, 150_000, 9_000]
    rowptr = np.concatenate([[0], np.cumsum(deg)]).astype(np.int64)
    E = int(rowptr[-1])
    assert E > (1 << 31) + (1 << 20)
    gt = torch.Generator(device="cuda").manual_seed(4242)
    cold = torch.randint(0, n_src, (E,), dtype=torch.int32, device="cuda", generator=gt)
    wd = None
    if F == 16:
        wd = (torch.randint(0, (1 << 24) - 1, (E,), dtype=torch.int32, device="cuda", generator=gt) + 1).float() * 2.0 ** -24
    x = gen.normal_features(n_src, F, 9)
    gy_h = gen.normal_features(n_dst, F, 10)
    xd, gy = dev(x, torch), dev(gy_h, torch)
    g = tiga.CsrRelation(dev(rowptr, torch), cold, n_src)
    cross = int(np.searchsorted(rowptr, 1 << 31, side="right") - 1)       # the row that holds edge 2^31
    rows = np.unique(np.concatenate([[0, 1, 5, 77_777, n_dst - 2, n_dst - 1, cross - 1, cross, cross + 1],
                                     rs.integers(0, n_dst, size=120), np.flatnonzero(deg == 0)[:3]])).astype(np.int64)

    with pytest.raises(tiga.TigaError) as e:
        tiga.tiga_apply_csr(g, xd, wd, tiga.MAX)
    assert e.value.status == 2
    y, _ = tiga.tiga_apply_csr(g, xd, wd, tiga.SUM)
    gx, gw = tiga.tiga_apply_csr_backward(g, xd, wd, gy, tiga.SUM)
    _sample_rows_check(tiga, rowptr, cold, wd, x, rows, y, None, gy, gw, "sum")
    # a source's gradient row gathers over all of its edges, wherever they are
    rp_d = g.rowptr
    for j in (0, 1234, n_src - 1):
        e_j = torch.nonzero(cold == j).flatten()
        r_j = torch.searchsorted(rp_d, e_j, right=True) - 1
        wj = torch.ones_like(e_j, dtype=torch.float64) if wd is None else wd[e_j].double()
        ref = (wj[:, None] * gy[r_j].double()).sum(0)
        mag = (wj[:, None] * gy[r_j].double().abs()).sum(0)
        assert float(((gx[j].double() - ref).abs() / mag).max()) <= GRAD_TOL
    del gw, gx, y
    ym, am = tiga.tiga_apply_csr(g, xd, wd, tiga.MAX64)
    assert am.dtype == torch.int64 and int(am.max()) >= (1 << 31)
    gx, gw = tiga.tiga_apply_csr_backward(g, xd, wd, gy, tiga.MAX64, argmax=am)
    _sample_rows_check(tiga, rowptr, cold, wd, x, rows, ym, am, gy, gw, "max")
    # all of the max cotangents, routed through the selected edges (float64 on the device)
    valid = am >= 0
    e_sel = am[valid]
    f_idx = torch.arange(F, device="cuda").expand(n_dst, F)[valid]
    wsel = torch.ones_like(e_sel, dtype=torch.float64) if wd is None else wd[e_sel].double()
    contrib = wsel * gy[valid].double()
    ref = torch.zeros((n_src, F), dtype=torch.float64, device="cuda").index_put_((cold[e_sel].long(), f_idx), contrib, accumulate=True)
    mag = torch.zeros((n_src, F), dtype=torch.float64, device="cuda").index_put_((cold[e_sel].long(), f_idx), contrib.abs(), accumulate=True)
    assert float(((gx.double() - ref).abs() / mag.clamp_min(1e-300)).max()) <= GRAD_TOL


def test_row_gather_probe_runs_and_checks_its_arguments(tiga):
    """The benchmark's measuring probe (a library of its own, not part of the product ABI)."""
    from paper_2609_24802_b200 import bench_probe
    table = torch.randn((4096, 64), device="cuda")
    idx = torch.randint(0, 4096, (100_000,), device="cuda", dtype=torch.int32)
    sink = torch.zeros(1, device="cuda")
    bench_probe.row_gather(table, idx, sink)
    torch.cuda.synchronize()
    assert torch.isfinite(sink).all()
    with pytest.raises(ValueError, match="status 1"):
        bench_probe.row_gather(torch.randn((16, 3), device="cuda"), idx[:4] % 16, sink)      # 12-byte rows
    with pytest.raises(ValueError, match="status 2"):
        bench_probe.row_gather(torch.randn((16, 12), device="cuda"), idx[:4] % 16, sink)     # 48-byte rows: not a power of two
