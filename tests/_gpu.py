"""Helpers for the GPU parity tests: device upload, guard bands, oracle comparison."""
import numpy as np
import torch

import oracle
import pf_workloads as wl

TOL = {wl.BF16: 1e-2, wl.F32: 1e-4}   # Frobenius-relative, per output tensor
TDT = {wl.BF16: torch.bfloat16, wl.F32: torch.float32}
GUARD = 64


def dev(a, dtype):
    return wl.to_torch(a, dtype).cuda()


def host(t, dtype):
    return wl.from_torch(t, dtype)


class Guarded:
    """An output tensor carved out of a larger sentinel-filled buffer, so that any write
    outside the tensor (before, after, or into row padding) is detected."""

    def __init__(self, shape, dtype, ld=None):
        rows = int(np.prod(shape[:-1]))
        cols = int(shape[-1])
        self.ld = cols if ld is None else ld
        self.rows, self.cols, self.shape = rows, cols, tuple(shape)
        n = rows * self.ld
        self.buf = torch.full((n + 2 * GUARD,), -7.0, dtype=TDT[dtype], device="cuda")
        self.t = self.buf[GUARD:GUARD + n].view(rows, self.ld)[:, :cols]
        if ld is None:
            self.t = self.t.reshape(self.shape)

    def check(self):
        b = self.buf.float().cpu()
        assert torch.all(b[:GUARD] == -7.0) and torch.all(b[-GUARD:] == -7.0), "guard band overwritten"
        if self.ld != self.cols:
            pad = b[GUARD:GUARD + self.rows * self.ld].view(self.rows, self.ld)[:, self.cols:]
            assert torch.all(pad == -7.0), "row padding overwritten"


def assert_close(got_t, want64, dtype, what, tol=None, abs_ref64=None):
    """Frobenius-relative error against the oracle.  For outputs of a handful of elements the
    Frobenius norm of the exact result can itself be a near-cancelled sum, so relative error is
    unbounded for any rounding of the m x r intermediate; such tiny outputs may instead be
    measured against `abs_ref64`, the oracle evaluated on the absolute values of the inputs
    (the magnitude of the summands)."""
    tol = tol or TOL[dtype]
    got = host(got_t.contiguous(), dtype)
    err = oracle.rel_err(got, want64)
    if err > tol and abs_ref64 is not None and np.asarray(want64).size < 256:
        diff = float(np.linalg.norm(oracle.widen(got).reshape(-1) - np.asarray(want64).reshape(-1)))
        err_abs = diff / max(float(np.linalg.norm(abs_ref64)), 1e-300)
        assert err_abs <= tol, f"{what}: err vs summand magnitude {err_abs:.3e} (rel {err:.3e})"
        return err_abs
    assert err <= tol, f"{what}: rel err {err:.3e}"
    return err
