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


class Guard:
    """Stand-in for a memory checker: every output and workspace handed to the library is carved out
    of a larger buffer.  The bands on both sides are filled with 0xA5 and must be untouched after
    the call; output interiors start as NaN (floats) or 0xA5A5A5A5 (integers) and must be
    overwritten in full, which proves that every row is written (empty ones included) and nothing
    outside is.  Workspaces get bands only: their contents are scratch."""

    BAND = 4096

    def __init__(self, torch):
        self.torch = torch
        self.items = []

    def _carve(self, nbytes):
        t = self.torch
        raw = t.full((2 * self.BAND + (nbytes + 255) // 256 * 256,), 0xA5, dtype=t.uint8, device="cuda")
        return raw

    def empty(self, shape, dtype=None):
        """An output tensor of this shape inside guard bands, poisoned."""
        t = self.torch
        dtype = t.float32 if dtype is None else dtype
        shape = tuple(int(s) for s in (shape if isinstance(shape, (tuple, list)) else (shape,)))
        n = 1
        for s in shape:
            n *= s
        esz = t.empty(0, dtype=dtype).element_size()
        raw = self._carve(n * esz)
        view = raw[self.BAND:self.BAND + n * esz].view(dtype).view(shape)
        if dtype.is_floating_point:
            view.fill_(float("nan"))
        self.items.append((raw, n * esz, view, "out"))
        return view

    def workspace(self, nbytes):
        nbytes = max(int(nbytes), 256)
        raw = self._carve(nbytes)
        view = raw[self.BAND:self.BAND + nbytes]
        self.items.append((raw, nbytes, view, "ws"))
        return view

    def check(self, allow_untouched=()):
        """Bands intact; every output element overwritten.  `allow_untouched`: outputs (tensors) that a
        call legitimately leaves alone."""
        t = self.torch
        t.cuda.synchronize()
        skip = {v.data_ptr() for v in allow_untouched}
        for raw, nbytes, view, kind in self.items:
            assert bool((raw[:self.BAND] == 0xA5).all()), "the library wrote in front of a buffer"
            assert bool((raw[self.BAND + nbytes:] == 0xA5).all()), "the library wrote behind a buffer"
            if kind != "out" or view.data_ptr() in skip or view.numel() == 0:
                continue
            if view.dtype.is_floating_point:
                assert not bool(t.isnan(view).any()), "an output element was not written (still NaN)"
            elif view.element_size() == 4:
                assert not bool((view.view(t.int32) == -1515870811).any()), "an output element was not written"
            elif view.element_size() == 8:
                assert not bool((view.view(t.int64) == -6510615555426900571).any()), "an output element was not written"
        self.items = []
