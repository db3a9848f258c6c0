"""Cases for the checked build of the library (libtiga_checked.so: every gathered index is range-checked
on the device, violations set a status word and the access goes to element 0).  Run as a script in a
process of its own with TIGA_CHECKED=1 (tests/test_gpu_checked.py does that): the library is chosen
when the binding is imported.

Part 1: well-formed inputs through the main entry points; results match the oracle and the status
word stays 0.  Part 2: relations whose index arrays hold a few out-of-range entries; the status word
names the violation, nothing faults, and the result equals the oracle's for the same relation with the
bad entries pointing at element 0 (which is where the checked build sends them)."""
import os
import sys

import numpy as np
import torch

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(HERE))
sys.path.insert(0, HERE)

import gen  # noqa: E402
import oracle  # noqa: E402
from parity import GRAD_TOL, SUM_TOL, dev, host, rel_err  # noqa: E402
from paper_2609_24802_b200 import api as T  # noqa: E402


def random_graph(seed, n_dst, n_src, max_deg, F):
    g = gen.rng(seed, 700)
    deg = g.integers(0, max_deg + 1, size=n_dst)
    deg[g.random(n_dst) < 0.3] = 0
    deg[3] = 9000                                   # one row for the chunked / multi-tile paths
    rowptr = np.concatenate([[0], np.cumsum(deg)]).astype(np.int64)
    E = int(rowptr[-1])
    col = g.integers(0, n_src, size=E).astype(np.int32)
    x = g.standard_normal((n_src, F)).astype(np.float32)
    w = ((g.integers(0, 2**24 - 1, size=E) + 1) * 2.0**-24).astype(np.float32)
    gy = g.standard_normal((n_dst, F)).astype(np.float32)
    return rowptr, col, x, w, gy


def csr_case(rowptr, col_dev, col_ref, x, w, gy, n_src, expect):
    """Forward sum / max and both backwards with `col_dev` on the device, compared with the oracle on
    `col_ref`; afterwards the status word must equal `expect`."""
    g = T.CsrRelation(dev(rowptr.astype(np.int32), torch), dev(col_dev, torch), n_src)
    xd, wd, gyd = dev(x, torch), dev(w, torch), dev(gy, torch)
    y, A, _ = oracle.csr_forward(rowptr, col_ref, x, w, oracle.SUM)
    out, _ = T.tiga_apply_csr(g, xd, wd, T.SUM)
    assert rel_err(host(out), y, A) <= SUM_TOL
    ym, _, arg = oracle.csr_forward(rowptr, col_ref, x, w, oracle.MAX)
    outm, am = T.tiga_apply_csr(g, xd, wd, T.MAX)
    assert np.array_equal(host(outm), ym.astype(np.float32)) and np.array_equal(host(am).astype(np.int64), arg)
    ref = oracle.csr_backward_sum(rowptr, col_ref, x, w, gy)
    gx, gw = T.tiga_apply_csr_backward(g, xd, wd, gyd, T.SUM)
    assert rel_err(host(gx), ref["gx"], ref["Ax"]) <= GRAD_TOL and rel_err(host(gw), ref["gw"], ref["Aw"]) <= GRAD_TOL
    refm = oracle.csr_backward_max(rowptr, col_ref, x, w, gy, arg)
    gx, gw = T.tiga_apply_csr_backward(g, xd, wd, gyd, T.MAX, argmax=am)
    assert rel_err(host(gx), refm["gx"], refm["Ax"]) <= GRAD_TOL and rel_err(host(gw), refm["gw"], refm["Aw"]) <= GRAD_TOL
    st = T.checked_status()
    assert st == expect, f"status word {st}, expected {expect}"
    return g, am


def main():
    assert T.is_checked_build(), "run with TIGA_CHECKED=1"
    assert T.checked_status() == 0

    # ---- part 1: well-formed inputs, wide and narrow feature rows, fp32 and fp16
    for F, dtype in ((64, np.float32), (8, np.float32), (8, np.float16), (32, np.float32)):
        rowptr, col, x, w, gy = random_graph(50 + F, 600, 300, 40, F)
        if dtype == np.float16:
            x = x.astype(np.float16)
            xr = x.astype(np.float32)
            g = T.CsrRelation(dev(rowptr, torch), dev(col, torch), 300)
            y, A, _ = oracle.csr_forward(rowptr, col, xr, None, oracle.SUM)
            out, _ = T.tiga_apply_csr(g, dev(x, torch), None, T.SUM)
            assert rel_err(host(out), y, A) <= SUM_TOL
            plan = T.tiga_csr_plan_build(g, max_hot_rows=40)
            planned, _ = T.tiga_apply_csr_planned(plan, dev(x, torch))
            assert torch.equal(planned, out)
            assert T.checked_status() == 0
        else:
            csr_case(rowptr, col, col, x, w, gy, 300, 0)
    n = 3000
    pos = gen.uniform_points(n, 61)
    feat = gen.normal_features(n, 16, 61, 31)
    gyr = gen.normal_features(n, 16, 61, 32)
    r = gen.radius_for_expected_neighbours(n, 12.0)
    ones = np.ones(3, np.float32)
    y, A, cnt = oracle.radius_forward(pos, feat, r, ones, [1, 1, 1], T.MSG_GAUSS, p0=float(r) / 2, use_cells=True)
    out, count, ws = T.tiga_apply_radius(dev(pos, torch), dev(feat, torch), r, ones, [1, 1, 1], T.MSG_GAUSS, p0=float(r) / 2,
                                         count=torch.empty(n, dtype=torch.int32, device="cuda"))
    assert np.array_equal(host(count), cnt) and rel_err(host(out), y, A) <= SUM_TOL
    ref = oracle.radius_backward_gauss(pos, feat, gyr, r, ones, [1, 1, 1], float(r) / 2, use_cells=True)
    gx, gp = T.tiga_apply_radius_backward(dev(pos, torch), dev(feat, torch), dev(gyr, torch), r, ones, [1, 1, 1], float(r) / 2)
    assert rel_err(host(gx), ref["gx"], ref["Agx"]) <= GRAD_TOL and rel_err(host(gp), ref["gp"], ref["Agp"]) <= GRAD_TOL
    c = gen.config("cfg3", m=10)
    yl, Al, cl = oracle.radius_forward(c["pos"], None, c["r"], c["box"], c["periodic"], T.MSG_LJ, p0=1.0, p1=1.0, use_cells=True)
    outl, countl, _ = T.tiga_apply_radius(dev(c["pos"], torch), None, c["r"], c["box"], c["periodic"], T.MSG_LJ, p0=1.0, p1=1.0,
                                          count=torch.empty(len(c["pos"]), dtype=torch.int32, device="cuda"))
    assert np.array_equal(host(countl), cl) and rel_err(host(outl), yl, Al) <= SUM_TOL
    params = gen.mlp_params(8, 16, 4, 7)
    xm, gm = gen.normal_features(n, 8, 62, 31), gen.normal_features(n, 4, 62, 32)
    ym, Am, cm = oracle.radius_mlp_forward(pos, xm, r, ones, [1, 1, 1], *params, use_cells=True)
    P = [dev(a, torch) for a in params]
    outm, countm, wsm = T.tiga_apply_radius_mlp(dev(pos, torch), dev(xm, torch), r, ones, [1, 1, 1], *P,
                                                count=torch.empty(n, dtype=torch.int32, device="cuda"))
    assert np.array_equal(host(countm), cm) and rel_err(host(outm), ym, Am) <= SUM_TOL
    T.tiga_apply_radius_mlp_backward(dev(pos, torch), dev(xm, torch), dev(gm, torch), r, ones, [1, 1, 1], *P)
    idx, rd2, yk, Ak = oracle.knn(pos, xm, 16)
    outk, nbr, d2, _ = T.tiga_apply_knn(dev(pos, torch), dev(xm, torch), 16, ones)
    assert np.array_equal(host(nbr), idx) and rel_err(host(outk), yk, Ak) <= SUM_TOL
    assert T.checked_status() == 0, "well-formed inputs must not raise the status word"

    # ---- part 2: a few source indices just outside [0, n_src): flagged, redirected to row 0, no fault
    for F in (64, 8):
        rowptr, col, x, w, gy = random_graph(70 + F, 600, 300, 40, F)
        bad = col.copy()
        where = gen.rng(7, 701).choice(len(col), size=25, replace=False)
        bad[where[:15]] = 300                       # one past the last source row
        bad[where[15:]] = -1
        fixed = col.copy()
        fixed[where] = 0
        g, am = csr_case(rowptr, bad, fixed, x, w, gy, 300, 1)
        # an argmax array with positions outside the relation: flagged as edge positions
        am_bad = am.clone()
        am_bad[5, 0] = g.n_edges + 3
        T.tiga_apply_csr_backward(g, dev(x, torch), dev(w, torch), dev(gy, torch), T.MAX, argmax=am_bad)
        st = T.checked_status()
        assert st & 2, f"status word {st}: an out-of-range edge position must set bit 2"
    torch.cuda.synchronize()
    print("checked build: all cases passed")


if __name__ == "__main__":
    main()
