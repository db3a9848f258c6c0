"""GPU parity of the online-softmax reducer over a stored relation (paper Section 5, attention
appendix) against the fp64 oracle: outputs within 1e-5 of the sum of absolute contributions,
log-sum-exp within 1e-5 absolute + relative."""
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


def _check(tiga, rowptr, col, n_src, q, k, v, scale, rowptr_dtype=np.int32, tol=SUM_TOL):
    g = tiga.CsrRelation(dev(rowptr.astype(rowptr_dtype), torch), dev(col, torch), n_src)
    guard = Guard(torch)
    out, lse, _ = tiga.tiga_apply_csr_attention(g, dev(q, torch), dev(k, torch), dev(v, torch), scale,
                                                out=guard.empty(q.shape), lse=guard.empty((q.shape[0],)),
                                                ws=guard.workspace(tiga.tiga_csr_attention_workspace_bytes(g, q.shape[1])))
    guard.check()
    y, A, ref_lse = oracle.csr_attention(rowptr, col, q, k, v, np.float32(scale))
    err = rel_err(host(out), y, A)
    if tol > SUM_TOL:
        print(f"online softmax: largest normalised error {err:.3e} (widened tolerance {tol:.3e}, plain {SUM_TOL:.0e})")
    assert err <= tol
    got = host(lse).astype(np.float64)
    empty = np.isneginf(ref_lse)
    assert np.array_equal(np.isneginf(got), empty)
    assert np.all(np.abs(got[~empty] - ref_lse[~empty]) <= max(tol, 1e-5) * (1.0 + np.abs(ref_lse[~empty])))
    out2, _, _ = tiga.tiga_apply_csr_attention(g, dev(q, torch), dev(k, torch), dev(v, torch), scale, want_lse=False)
    assert torch.equal(out, out2), "no atomics: reruns must be bit identical"
    return out


def _qkv(n_dst, n_src, D, seed):
    return (gen.normal_features(n_dst, D, seed, 31), gen.normal_features(n_src, D, seed, 32),
            gen.normal_features(n_src, D, seed, 33))


def test_causal_attention_example(tiga):
    # the appendix' check: 65 tokens (a partial tile), head width 64, triangular relation with the diagonal
    n, D = 65, 64
    rowptr = np.cumsum([0] + [i + 1 for i in range(n)]).astype(np.int64)
    col = np.concatenate([np.arange(i + 1) for i in range(n)]).astype(np.int32)
    q, k, v = _qkv(n, n, D, 7)
    out = _check(tiga, rowptr, col, n, q, k, v, D ** -0.5)
    assert np.allclose(host(out)[0], v[0], rtol=1e-6, atol=1e-7)      # token zero reads only itself


@pytest.mark.parametrize("D", [4, 8, 16, 24, 32, 64, 100, 128])
def test_widths_on_a_skewed_graph(tiga, D):
    c = gen.config("cfg1", 11, scale=12, F=4)                          # R-MAT: empty rows, one very long row
    q, k, v = _qkv(c["n"], c["n"], D, 12)
    _check(tiga, c["rowptr"], c["col"], c["n"], q, k, v, D ** -0.5)


def test_long_causal_sequence_spans_many_tiles(tiga):
    n, D = 1500, 32                                                    # rows of up to 1500 edges: carry-outs across tiles
    rowptr = np.cumsum([0] + [i + 1 for i in range(n)]).astype(np.int64)
    col = np.concatenate([np.arange(i + 1) for i in range(n)]).astype(np.int32)
    q, k, v = _qkv(n, n, D, 13)
    _check(tiga, rowptr, col, n, q, k, v, D ** -0.5, rowptr_dtype=np.int64)


def test_one_row_longer_than_many_tiles_and_empty_tail(tiga):
    n_src, D = 3000, 16
    g = gen.rng(14, 1)
    col = g.integers(0, n_src, 20000).astype(np.int32)
    rowptr = np.array([0, 0, 20000, 20000, 20000], np.int64)          # empty, huge, empty, empty
    q, k, v = _qkv(4, n_src, D, 14)
    _check(tiga, rowptr, col, n_src, q, k, v, 0.25)


def test_large_scores_stay_finite(tiga):
    c = gen.config("cfg1", 15, scale=10, F=4)
    q, k, v = _qkv(c["n"], c["n"], 32, 15)
    q, k = q * 6.0, k * 6.0                                            # scores of several hundred
    # an fp32 score carries a rounding error of up to about D * 2^-24 * sum_d |q_d k_d|; the softmax
    # turns an absolute score error into a relative weight error, so the bound scales with the scores
    bound = 4.0 * 2.0 ** -24 * float((np.abs(q).max(0) * np.abs(k).max(0)).sum())
    out = _check(tiga, c["rowptr"], c["col"], c["n"], q, k, v, 1.0, tol=SUM_TOL + bound)
    assert torch.isfinite(out).all()


def test_empty_relation_and_bad_arguments(tiga):
    q, k, v = _qkv(10, 10, 8, 16)
    rowptr = np.zeros(11, np.int64)
    out = _check(tiga, rowptr, np.zeros(0, np.int32), 10, q, k, v, 1.0)
    assert torch.all(out == 0)
    g = tiga.CsrRelation(dev(rowptr.astype(np.int32), torch), dev(np.zeros(0, np.int32), torch), 10)
    for D, status in ((6, 1), (132, 2)):
        x = torch.zeros((10, D), device="cuda")
        with pytest.raises(tiga.TigaError) as e:
            tiga.tiga_apply_csr_attention(g, x, x, x, 1.0, ws=torch.empty(1 << 16, dtype=torch.uint8, device="cuda"))
        assert e.value.status == status


def test_graph_attention_at_benchmark_size(tiga):
    # the benchmark's stored relation (R-MAT scale 20, 16.8M edges) with head width 64
    c = gen.config("cfg1", gen.DEFAULT_SEED)
    q, k, v = _qkv(c["n"], c["n"], 64, 17)
    _check(tiga, c["rowptr"], c["col"], c["n"], q, k, v, 0.125)
