"""Pins for the online-softmax oracle: dense causal attention from a library softmax, library
log-sum-exp per row, the paper's state-combine rule, closed forms and degenerate rows.  No GPU."""
import numpy as np
import pytest

import oracle

torch = pytest.importorskip("torch")


def random_csr(rng, n_dst, n_src, max_deg, empty=0.2):
    deg = rng.integers(1, max_deg + 1, n_dst)
    deg[rng.random(n_dst) < empty] = 0
    rowptr = np.concatenate([[0], np.cumsum(deg)]).astype(np.int64)
    col = rng.integers(0, n_src, rowptr[-1]).astype(np.int32)
    return rowptr, col


def test_causal_attention_example():
    # the appendix' check: 65 tokens, head width 64, triangular relation with the diagonal
    n, D = 65, 64
    g = torch.Generator().manual_seed(7)
    q, k, v = (torch.randn(n, D, generator=g, dtype=torch.float64) for _ in range(3))
    rowptr = np.cumsum([0] + [i + 1 for i in range(n)]).astype(np.int64)
    col = np.concatenate([np.arange(i + 1) for i in range(n)]).astype(np.int32)
    scores = (q @ k.T) * D ** -0.5
    future = torch.triu(torch.ones(n, n, dtype=torch.bool), 1)
    ref = scores.masked_fill(future, -torch.inf).softmax(-1) @ v
    y, A, lse = oracle.csr_attention(rowptr, col, q.numpy(), k.numpy(), v.numpy(), D ** -0.5)
    assert np.allclose(y, ref.numpy(), rtol=1e-12, atol=1e-13)
    assert np.allclose(lse, torch.logsumexp(scores.masked_fill(future, -torch.inf), -1).numpy(), rtol=1e-12)
    assert np.allclose(y[0], v[0].numpy())                          # token zero reads only itself


def test_rows_against_library_logsumexp():
    from scipy.special import logsumexp, softmax
    rng = np.random.default_rng(3)
    n_dst, n_src, D = 200, 150, 8
    rowptr, col = random_csr(rng, n_dst, n_src, 40)
    q, k, v = rng.standard_normal((n_dst, D)), rng.standard_normal((n_src, D)), rng.standard_normal((n_src, D))
    y, A, lse = oracle.csr_attention(rowptr, col, q, k, v, 0.7)
    for i in range(n_dst):
        c = col[rowptr[i]:rowptr[i + 1]]
        if len(c) == 0:
            assert np.all(y[i] == 0) and np.all(A[i] == 0) and lse[i] == -np.inf
            continue
        s = 0.7 * (k[c] @ q[i])
        p = softmax(s)
        assert np.allclose(y[i], p @ v[c], rtol=1e-12, atol=1e-14)
        assert np.allclose(A[i], p @ np.abs(v[c]), rtol=1e-12)
        assert np.isclose(lse[i], logsumexp(s), rtol=1e-13)


def test_combine_rule_of_the_streaming_state():
    # a row split in two parts: the states (m, l, o) of the parts combine to the state of the whole
    rng = np.random.default_rng(4)
    D, n_src = 4, 50
    k, v = rng.standard_normal((n_src, D)), rng.standard_normal((n_src, D))
    q = rng.standard_normal((1, D))
    c = rng.integers(0, n_src, 30).astype(np.int32)
    whole = oracle.csr_attention(np.array([0, 30]), c, q, k, v, 1.3)
    parts = oracle.csr_attention(np.array([0, 11, 30]), c, np.repeat(q, 2, 0), k, v, 1.3)
    (ya, yb), (ma, mb) = parts[0], parts[2]                        # finalised row = state (lse, 1, y)
    m = max(ma, mb)
    l = np.exp(ma - m) + np.exp(mb - m)
    o = np.exp(ma - m) * ya + np.exp(mb - m) * yb
    assert np.allclose(o / l, whole[0][0], rtol=1e-12)
    assert np.isclose(m + np.log(l), whole[2][0], rtol=1e-13)


def test_closed_forms():
    rng = np.random.default_rng(5)
    D = 4
    v = rng.standard_normal((6, D))
    k = np.tile(rng.standard_normal((1, D)), (6, 1))               # equal keys: the mean of the values
    q = rng.standard_normal((2, D))
    y, _, lse = oracle.csr_attention(np.array([0, 6, 7]), np.array([0, 1, 2, 3, 4, 5, 3], np.int32), q, k, v, 0.5)
    assert np.allclose(y[0], v.mean(0), rtol=1e-13)
    assert np.array_equal(y[1], v[3])                               # a single edge returns its value exactly
    assert np.isclose(lse[0], 0.5 * k[0] @ q[0] + np.log(6.0))
    # a repeated edge is a separate message: it doubles that source's weight
    k2 = rng.standard_normal((3, D))
    y2, _, _ = oracle.csr_attention(np.array([0, 4]), np.array([0, 1, 1, 2], np.int32), q[:1], k2, v[:3], 1.0)
    w = np.exp(k2 @ q[0]) * np.array([1.0, 2.0, 1.0])
    assert np.allclose(y2[0], (w / w.sum()) @ v[:3], rtol=1e-12)
    # adding to every key a vector orthogonal to nothing in particular shifts all scores of a row
    # by the same amount: the result does not change
    shift = rng.standard_normal(D)
    y3, _, _ = oracle.csr_attention(np.array([0, 4]), np.array([0, 1, 1, 2], np.int32), q[:1], k2 + shift, v[:3], 1.0)
    assert np.allclose(y3, y2, rtol=1e-12)


def test_large_scores_do_not_overflow():
    q = np.array([[100.0, 0.0]])
    k = np.array([[10.0, 0.0], [9.0, 0.0], [-10.0, 0.0]])
    v = np.array([[1.0, 0.0], [0.0, 1.0], [5.0, 5.0]])
    y, _, lse = oracle.csr_attention(np.array([0, 3]), np.array([0, 1, 2], np.int32), q, k, v, 1.0)
    e = np.exp(-100.0)
    assert np.allclose(y[0], [1.0 / (1.0 + e), e / (1.0 + e)], rtol=1e-12, atol=0.0)
    assert np.isclose(lse[0], 1000.0 + np.log1p(e))
