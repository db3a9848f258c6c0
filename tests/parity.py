"""Helpers shared by the GPU parity tests (comparison metric, host<->device marshalling)."""
import numpy as np

SUM_TOL = 1e-5      # forward sums: |gpu - oracle| <= SUM_TOL * sum of |contributions|
GRAD_TOL = 1e-4     # gradients, same normalisation


def rel_err(got, ref, A):
    """Largest error normalised by the sum of absolute contributions; entries whose
    normaliser is zero (empty rows, points without neighbours) must be exactly zero."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    A = np.asarray(A, dtype=np.float64)
    zero = A == 0
    assert np.all(got[zero] == 0.0), "entries without contributions must be exactly 0"
    if np.all(zero):
        return 0.0
    return float(np.max(np.abs(got[~zero] - ref[~zero]) / A[~zero]))


def dev(a, torch, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def host(t):
    return t.detach().cpu().numpy()
