"""Pins for the edge-network part of the oracle (paper Appendix A): an explicit gather -> MLP ->
index_add evaluation with torch autograd in float64 on an independently built edge list, plus
structural invariants."""
import numpy as np
import pytest

import gen
import oracle

torch = pytest.importorskip("torch")


def _setup(n, seed, periodic, Fin=8, H=16, Fout=4, r=0.25):
    pos = gen.uniform_points(n, seed)
    x = gen.normal_features(n, Fin, seed, 31)
    gy = gen.normal_features(n, Fout, seed, 32)
    g = gen.rng(seed, 71)
    W1 = (g.standard_normal((H, 3 + Fin)) * 0.5).astype(np.float32)
    b1 = (g.standard_normal(H) * 0.2).astype(np.float32)
    W2 = (g.standard_normal((Fout, H)) * 0.5).astype(np.float32)
    b2 = (g.standard_normal(Fout) * 0.2).astype(np.float32)
    return pos, x, gy, (W1, b1, W2, b2), np.ones(3, np.float32), np.full(3, int(periodic), np.int32), np.float32(r)


def _torch_reference(pos, x, gy, params, box, per, r):
    """Edges by an all-pairs numpy search; message and reduction by torch ops; gradients by autograd."""
    p64 = pos.astype(np.float64)
    D = p64[None, :, :] - p64[:, None, :]              # D[i, j] = p_j - p_i
    for d in range(3):
        if per[d]:
            D[:, :, d] -= float(box[d]) * np.round(D[:, :, d] / float(box[d]))
    M = (D ** 2).sum(-1) <= float(r) ** 2
    np.fill_diagonal(M, False)
    rows, cols = np.nonzero(M)
    shift = torch.from_numpy(D[rows, cols] - (p64[cols] - p64[rows]))      # periodic image offsets (constants)
    P = torch.tensor(p64, requires_grad=True)
    X = torch.tensor(x.astype(np.float64), requires_grad=True)
    W1, b1, W2, b2 = [torch.tensor(a.astype(np.float64), requires_grad=True) for a in params]
    ri, ci = torch.from_numpy(rows), torch.from_numpy(cols)
    delta = P[ci] - P[ri] + shift
    hid = torch.relu(torch.cat((delta, X[ci]), dim=-1) @ W1.T + b1)
    msg = hid @ W2.T + b2
    y = torch.zeros((len(pos), W2.shape[0]), dtype=torch.float64).index_add(0, ri, msg)
    loss = (y * torch.from_numpy(gy.astype(np.float64))).sum()
    grads = torch.autograd.grad(loss, (X, P, W1, b1, W2, b2))
    return y.detach().numpy(), [g.numpy() for g in grads], M.sum(1)


@pytest.mark.parametrize("periodic", [0, 1])
def test_forward_and_all_gradients_match_torch_autograd(periodic):
    pos, x, gy, params, box, per, r = _setup(150, 5, periodic)
    y, A, cnt = oracle.radius_mlp_forward(pos, x, r, box, per, *params)
    yt, gt, ct = _torch_reference(pos, x, gy, params, box, per, r)
    assert np.array_equal(cnt, ct)
    assert np.max(np.abs(y - yt) / (A + 1e-300)) < 1e-12
    b = oracle.radius_mlp_backward(pos, x, gy, r, box, per, *params)
    for name, ref in zip(("gx", "gp", "gW1", "gb1", "gW2", "gb2"), gt):
        assert np.max(np.abs(b[name] - ref) / (b["A" + name] + 1e-300)) < 1e-11, name
    # translation invariance: position gradients sum to zero
    assert np.max(np.abs(b["gp"].sum(0))) < 1e-11 * b["Agp"].sum()
    # the final bias sits inside the sum: d(loss)/d(b2) = sum_i count_i * ybar_i
    assert np.allclose(b["gb2"], (cnt[:, None] * gy.astype(np.float64)).sum(0), rtol=1e-12)


def test_no_neighbours_gives_zero_and_widths(periodic=0):
    pos, x, gy, params, box, per, r = _setup(40, 9, 0, Fin=5, H=8, Fout=3, r=0.01)
    y, A, cnt = oracle.radius_mlp_forward(pos, x, r, box, per, *params)
    assert cnt.sum() == 0 and np.all(y == 0) and np.all(A == 0)
    pos, x, gy, params, box, per, r = _setup(90, 10, 1, Fin=5, H=32, Fout=3, r=0.3)
    y, A, cnt = oracle.radius_mlp_forward(pos, x, r, box, per, *params)
    yc, Ac, cc = oracle.radius_mlp_forward(pos, x, r, box, per, *params, use_cells=True)
    assert np.array_equal(y, yc) and np.array_equal(cnt, cc)
    yt, gt, _ = _torch_reference(pos, x, gy, params, box, per, r)
    assert np.max(np.abs(y - yt) / (A + 1e-300)) < 1e-12
    b = oracle.radius_mlp_backward(pos, x, gy, r, box, per, *params, use_cells=True)
    for name, ref in zip(("gx", "gp", "gW1", "gb1", "gW2", "gb2"), gt):
        assert np.max(np.abs(b[name] - ref) / (b["A" + name] + 1e-300)) < 1e-11, name
