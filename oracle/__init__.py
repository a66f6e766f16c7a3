"""fp64 CPU oracle for low-rank pre-factorized layers -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It shares no code with the CUDA library and never imports it.  The arithmetic
lives in ``pf_oracle.c`` (plain loops in double precision, one per definition); this file
only widens stored inputs to fp64 exactly, marshals numpy arrays and defines the
comparison metric.

Functions (paper passages they follow are cited in ``pf_oracle.c``):

    linear_fwd(x, U, V)              -> y, T            y = (x U) V^T
    linear_bwd(x, U, V, dY)          -> dX, dU, dV      chain rule on the above
    linear_grouped_fwd / _bwd(x, U, V[, dY])            the same for G factor pairs (shared or own x)
    conv_fwd(x, U, V, stride, pad)   -> y, T            k x k conv to r channels, then 1 x 1
    conv_bwd(x, U, V, dY, stride, pad) -> dX, dU, dV
    pack(list_of_arrays)             -> flat, offsets   flat gradient buffer
    unpack(flat, numels)             -> arrays, offsets its inverse

Parity pins (tests/test_oracle_*.py): hand-computed tiny cases, the dense identity
(xU)V^T = x(UV^T), special cases that reduce to a textbook matrix product or a library
correlation, the dense chain rule, central finite differences, an independent
im2col route for the convolution, Table 1 parameter counts and pure-Python brute force.
The paper prints no numeric layer output, so no output value is pinned by its text.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libpf_oracle.so")
_SRC = os.path.join(_HERE, "pf_oracle.c")
_lib = None


def build(force: bool = False) -> str:
    """Compile pf_oracle.c with gcc (OpenMP) into libpf_oracle.so next to it."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", tmp, _SRC])
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_SO)
        L, D, I = ctypes.c_long, ctypes.c_void_p, ctypes.c_int
        lib.pf_oracle_threads.restype = I
        lib.pf_oracle_linear_fwd.argtypes = [D, D, D, L, L, L, L, D, D]
        lib.pf_oracle_linear_bwd.argtypes = [D, D, D, D, D, L, L, L, L, D, D, D, D]
        lib.pf_oracle_conv_fwd.argtypes = [D, D, D] + [L] * 10 + [D, D]
        lib.pf_oracle_conv_bwd.argtypes = [D, D, D, D, D] + [L] * 10 + [D, D, D, D]
        lib.pf_oracle_pack.argtypes = [D, D, I, I, D, D]
        for f in ("linear_fwd", "linear_bwd", "conv_fwd", "conv_bwd", "pack"):
            getattr(lib, "pf_oracle_" + f).restype = None
        _lib = lib
    return _lib


def threads() -> int:
    return int(_load().pf_oracle_threads())


def widen(a) -> np.ndarray:
    """Stored values -> float64, exactly.  uint16 arrays are bf16 bit patterns."""
    a = np.asarray(a)
    if a.dtype == np.uint16:
        a = np.ascontiguousarray(a)          # fancy-indexed slices may not be C-ordered
        return np.ascontiguousarray((a.astype(np.uint32) << np.uint32(16)).view(np.float32),
                                    dtype=np.float64)
    return np.ascontiguousarray(a, dtype=np.float64)


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def linear_fwd(x, U, V):
    x, U, V = widen(x), widen(U), widen(V)
    m, k = x.shape
    k2, r = U.shape
    n, r2 = V.shape
    assert k == k2 and r == r2
    T = np.empty((m, r))
    y = np.empty((m, n))
    _load().pf_oracle_linear_fwd(_p(x), _p(U), _p(V), m, k, n, r, _p(T), _p(y))
    return y, T


def linear_fwd_act(x, U, V, bias=None, relu=False):
    """y = act((x U) V^T + bias), the factorized layer followed by its (unfactorized) bias and, for the
    first half of the feed-forward block, max(0, .) (Section 2.4: FFN(x) = max(0, x W1 + b1) W2 + b2 with
    W = U V^T; Section 2.1: biases stay as they are).  Returns (y, T) with T = x U."""
    y, T = linear_fwd(x, U, V)
    if bias is not None:
        b = widen(bias)
        assert b.shape == (y.shape[1],)
        y = y + b[None, :]
    if relu:
        y = np.maximum(y, 0.0)
    return y, T


def bias_act_bwd(y, dY, relu=True):
    """Backward of y = act(z + bias) (Section 2.4's max(0, x W1 + b1)): dZ = dY where y > 0 (else 0) for
    max(0, .), dZ = dY for the identity; dbias = column sums of dZ (plain sums over the rows)."""
    y, dY = widen(y), widen(dY)
    dZ = np.where(y > 0, dY, 0.0) if relu else dY.copy()
    return dZ, dZ.sum(axis=0)


def linear_bwd(x, U, V, dY):
    x, U, V, dY = widen(x), widen(U), widen(V), widen(dY)
    m, k = x.shape
    n, r = V.shape
    assert U.shape == (k, r) and dY.shape == (m, n)
    _, T = linear_fwd(x, U, V)
    G = np.empty((m, r))
    dX = np.empty((m, k))
    dU = np.empty((k, r))
    dV = np.empty((n, r))
    _load().pf_oracle_linear_bwd(_p(x), _p(U), _p(V), _p(dY), _p(T), m, k, n, r,
                                 _p(G), _p(dX), _p(dU), _p(dV))
    return dX, dU, dV


def linear_grouped_fwd(x, U, V):
    """Grouped layer (Section 2.3, per-gate LSTM factors; Section 2.4, attention projections):
    y[g] = (x[g] U[g]) V[g]^T for every group g, each through linear_fwd.  x is [G, m, k], or
    [m, k] when all groups read the same input."""
    G = len(U)
    out = [linear_fwd(x if np.ndim(x) == 2 else x[g], U[g], V[g]) for g in range(G)]
    return np.stack([o[0] for o in out]), np.stack([o[1] for o in out])


def linear_grouped_bwd(x, U, V, dY):
    """Gradients of the grouped layer, group by group through linear_bwd.  An input shared by all
    groups collects the gradient of every group that reads it: dX = sum over g of dX[g]."""
    G = len(U)
    shared = np.ndim(x) == 2
    out = [linear_bwd(x if shared else x[g], U[g], V[g], dY[g]) for g in range(G)]
    dX = np.sum([o[0] for o in out], axis=0) if shared else np.stack([o[0] for o in out])
    return dX, np.stack([o[1] for o in out]), np.stack([o[2] for o in out])


def conv_out_hw(H, W, kh, kw, stride, pad):
    return (H + 2 * pad - kh) // stride + 1, (W + 2 * pad - kw) // stride + 1


def conv_fwd(x, U, V, stride=1, pad=1):
    x, U, V = widen(x), widen(U), widen(V)
    N, H, W, C = x.shape
    kh, kw, C2, R = U.shape
    O, R2 = V.shape
    assert C == C2 and R == R2
    Ho, Wo = conv_out_hw(H, W, kh, kw, stride, pad)
    T = np.empty((N, Ho, Wo, R))
    y = np.empty((N, Ho, Wo, O))
    _load().pf_oracle_conv_fwd(_p(x), _p(U), _p(V), N, H, W, C, R, O, kh, kw, stride, pad,
                               _p(T), _p(y))
    return y, T


def conv_bwd(x, U, V, dY, stride=1, pad=1):
    x, U, V, dY = widen(x), widen(U), widen(V), widen(dY)
    N, H, W, C = x.shape
    kh, kw, _, R = U.shape
    O = V.shape[0]
    Ho, Wo = conv_out_hw(H, W, kh, kw, stride, pad)
    assert dY.shape == (N, Ho, Wo, O)
    _, T = conv_fwd(x, U, V, stride, pad)
    dT = np.empty((N, Ho, Wo, R))
    dX = np.empty((N, H, W, C))
    dU = np.empty((kh, kw, C, R))
    dV = np.empty((O, R))
    _load().pf_oracle_conv_bwd(_p(x), _p(U), _p(V), _p(dY), _p(T), N, H, W, C, R, O,
                               kh, kw, stride, pad, _p(dT), _p(dX), _p(dU), _p(dV))
    return dX, dU, dV


def pack(grads):
    """Flat gradient buffer: values copied bit for bit, in list order, tightly."""
    grads = [np.ascontiguousarray(g).reshape(-1) for g in grads]
    count = len(grads)
    dt = grads[0].dtype if count else np.dtype(np.uint16)
    assert all(g.dtype == dt for g in grads)
    numels = np.array([g.size for g in grads], dtype=np.int64)
    total = int(numels.sum())
    flat = np.empty(total, dtype=dt)
    offsets = np.zeros(count + 1, dtype=np.int64)
    ptrs = (ctypes.c_void_p * max(count, 1))(*[g.ctypes.data for g in grads])
    _load().pf_oracle_pack(ctypes.cast(ptrs, ctypes.c_void_p), _p(numels), count,
                           dt.itemsize, _p(flat), _p(offsets))
    return flat, offsets


def unpack(flat, numels):
    """The inverse of pack (Section 4.1, after the all-reduce): tensor i is the slice of the flat
    buffer at the prefix-sum offset of numels.  Returns (list of arrays, offsets)."""
    flat = np.asarray(flat)
    offsets = np.zeros(len(numels) + 1, dtype=np.int64)
    out = []
    for i, cnt in enumerate(numels):
        offsets[i + 1] = offsets[i] + int(cnt)
        out.append(np.array([flat[e] for e in range(offsets[i], offsets[i + 1])], dtype=flat.dtype))
    return out, offsets


def rel_err(z, z_ref) -> float:
    """Frobenius-norm-relative error  ||z - z_ref||_F / max(||z_ref||_F, tiny)  in fp64."""
    z = widen(z).reshape(-1)
    z_ref = np.asarray(z_ref, dtype=np.float64).reshape(-1)
    assert z.shape == z_ref.shape, (z.shape, z_ref.shape)
    den = max(float(np.linalg.norm(z_ref)), 1e-300)
    return float(np.linalg.norm(z - z_ref)) / den
