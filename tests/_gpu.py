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


# Every (case, tensor) that took the cancellation rule below, in the order met.
ESCAPES = []
CANCELLED = 0.05      # a result counts as cancelled when ||exact|| < CANCELLED * ||summand magnitudes||


def assert_close(got_t, want64, dtype, what, tol=None, abs_ref64=None):
    """Frobenius-relative error against the oracle, at the stated tolerance.

    One refinement, for bf16 only and only for outputs of fewer than 256 elements: such an output
    can be a single near-cancelled sum, for which no rounding of the m x r intermediate to bf16
    gives a bounded relative error.  When the exact result is demonstrably cancelled
    (||exact||_F < 0.05 ||summand magnitudes||_F, `abs_ref64` being the oracle evaluated on the
    absolute values of the inputs) the error is measured against the summand magnitudes instead,
    and the case is recorded in ESCAPES.  fp32 never takes this route: nothing there is rounded
    to bf16, so a miss of 1e-4 is a defect."""
    tol = tol or TOL[dtype]
    got = host(got_t.contiguous(), dtype)
    err = oracle.rel_err(got, want64)
    if (err > tol and dtype == wl.BF16 and abs_ref64 is not None and np.asarray(want64).size < 256):
        ref_norm = float(np.linalg.norm(np.asarray(want64)))
        abs_norm = float(np.linalg.norm(abs_ref64))
        if ref_norm < CANCELLED * abs_norm:
            diff = float(np.linalg.norm(oracle.widen(got).reshape(-1) - np.asarray(want64).reshape(-1)))
            err_abs = diff / max(abs_norm, 1e-300)
            ESCAPES.append((what, err, ref_norm / max(abs_norm, 1e-300), err_abs))
            assert err_abs <= tol, f"{what}: err vs summand magnitude {err_abs:.3e} (rel {err:.3e})"
            return err_abs
    assert err <= tol, f"{what}: rel err {err:.3e}"
    return err


def assert_blocks_close(got_t, want64, dtype, what, br=128, bc=128, tol=None):
    """The same bound per block: the maximum over br x bc blocks (of the tensor flattened to
    [rows, last dimension]) of the block's Frobenius-relative error must stay within the
    tolerance, so a wrong edge strip or a mis-clipped tile cannot hide in the whole-tensor norm."""
    tol = tol or TOL[dtype]
    got = oracle.widen(host(got_t.contiguous(), dtype))
    want = np.asarray(want64, dtype=np.float64)
    got = got.reshape(-1, got.shape[-1])
    want = want.reshape(-1, want.shape[-1])
    assert got.shape == want.shape, (what, got.shape, want.shape)
    R, C = want.shape
    pr, pc = (-R) % br, (-C) % bc
    d2 = np.pad((got - want) ** 2, ((0, pr), (0, pc)))
    w2 = np.pad(want ** 2, ((0, pr), (0, pc)))
    nb_r, nb_c = d2.shape[0] // br, d2.shape[1] // bc
    num = d2.reshape(nb_r, br, nb_c, bc).sum(axis=(1, 3))
    den = w2.reshape(nb_r, br, nb_c, bc).sum(axis=(1, 3))
    rel = np.sqrt(num / np.maximum(den, 1e-300))
    worst = np.unravel_index(int(np.argmax(rel)), rel.shape)
    assert rel[worst] <= tol, f"{what}: block {worst} of {rel.shape} has rel err {rel[worst]:.3e}"
    return float(rel[worst])
