"""Pins for the fp64 oracle of the factorized convolution (Section 2.2, Appendix B
"Convolution layer"): thin k x k convolution U into r channels, then 1 x 1 convolution V^T.

Checked against: a hand-computed example, an independent im2col + matrix-product route
(the unrolled-matrix view of Section 2.2), library correlations (scipy, torch conv2d in
fp64 with autograd), special cases, finite differences and pure-Python brute force.
"""
import os

import numpy as np
import pytest

import oracle
from _util import read_golden, rng_int


def test_hand_case(golden_dir):
    g = read_golden(os.path.join(golden_dir, "conv_hand_case.txt"))
    y, T = oracle.conv_fwd(g["x"], g["U"], g["V"], 1, 1)
    dX, dU, dV = oracle.conv_bwd(g["x"], g["U"], g["V"], g["dY"], 1, 1)
    for got, want in ((y, "y"), (T, "T"), (dX, "dX"), (dU, "dU"), (dV, "dV")):
        np.testing.assert_array_equal(got, g[want])


def _im2col(x, kh, kw, st, pad):
    """Unrolled patches [N*Ho*Wo, kh*kw*C], rows ordered (tap-major, channel fastest)."""
    N, H, W, C = x.shape
    xp = np.zeros((N, H + 2 * pad, W + 2 * pad, C))
    xp[:, pad:pad + H, pad:pad + W] = x
    Ho = (H + 2 * pad - kh) // st + 1
    Wo = (W + 2 * pad - kw) // st + 1
    cols = np.zeros((N, Ho, Wo, kh, kw, C))
    for a in range(kh):
        for b in range(kw):
            cols[:, :, :, a, b, :] = xp[:, a:a + st * Ho:st, b:b + st * Wo:st, :]
    return cols.reshape(N * Ho * Wo, kh * kw * C), (N, Ho, Wo)


CASES = [  # N,H,W,C,R,O,kh,kw,st,pad
    (1, 3, 3, 1, 1, 1, 3, 3, 1, 1),
    (2, 5, 4, 3, 2, 3, 3, 3, 1, 1),
    (1, 6, 5, 2, 3, 2, 3, 3, 2, 1),
    (2, 4, 4, 2, 2, 3, 1, 1, 1, 0),
    (1, 5, 5, 2, 2, 2, 3, 3, 1, 0),
    (1, 7, 6, 2, 2, 2, 5, 5, 2, 2),
]


@pytest.mark.parametrize("case", CASES)
def test_fwd_equals_unrolled_matrix_route(case):
    """Section 2.2: the convolution is a matrix product with the unrolled (c_in k^2) x r
    matrix, followed by the r x c_out projection; so it must equal the linear oracle on
    im2col patches."""
    N, H, W, C, R, O, kh, kw, st, pad = case
    x, U, V = rng_int(1, (N, H, W, C)), rng_int(2, (kh, kw, C, R)), rng_int(3, (O, R))
    y, T = oracle.conv_fwd(x, U, V, st, pad)
    cols, (n_, ho, wo) = _im2col(x, kh, kw, st, pad)
    y2, T2 = oracle.linear_fwd(cols, U.reshape(kh * kw * C, R), V)
    np.testing.assert_array_equal(y, y2.reshape(n_, ho, wo, O))
    np.testing.assert_array_equal(T, T2.reshape(n_, ho, wo, R))


@pytest.mark.parametrize("case", CASES)
def test_fwd_bwd_against_torch_conv2d_fp64(case):
    """Library pin: two chained torch conv2d calls (cross-correlation) in fp64 and their
    autograd gradients."""
    torch = pytest.importorskip("torch")
    import torch.nn.functional as F
    N, H, W, C, R, O, kh, kw, st, pad = case
    rng = np.random.default_rng(5)
    x, U, V = rng.normal(size=(N, H, W, C)), rng.normal(size=(kh, kw, C, R)), rng.normal(size=(O, R))
    Ho, Wo = oracle.conv_out_hw(H, W, kh, kw, st, pad)
    dY = rng.normal(size=(N, Ho, Wo, O))
    tx = torch.tensor(x).permute(0, 3, 1, 2).contiguous().requires_grad_(True)   # NCHW
    tU = torch.tensor(U).permute(3, 2, 0, 1).contiguous().requires_grad_(True)   # [R,C,kh,kw]
    tV = torch.tensor(V).reshape(O, R, 1, 1).clone().requires_grad_(True)
    tT = F.conv2d(tx, tU, stride=st, padding=pad)
    ty = F.conv2d(tT, tV)
    ty.backward(torch.tensor(dY).permute(0, 3, 1, 2).contiguous())
    y, T = oracle.conv_fwd(x, U, V, st, pad)
    dX, dU, dV = oracle.conv_bwd(x, U, V, dY, st, pad)
    assert oracle.rel_err(y, ty.detach().permute(0, 2, 3, 1).numpy()) < 1e-13
    assert oracle.rel_err(T, tT.detach().permute(0, 2, 3, 1).numpy()) < 1e-13
    assert oracle.rel_err(dX, tx.grad.permute(0, 2, 3, 1).numpy()) < 1e-13
    assert oracle.rel_err(dU, tU.grad.permute(2, 3, 1, 0).numpy()) < 1e-13
    assert oracle.rel_err(dV, tV.grad.reshape(O, R).numpy()) < 1e-13


def test_1x1_conv_is_the_linear_layer():
    N, H, W, C, R, O = 2, 3, 4, 5, 2, 6
    x, U, V = rng_int(7, (N, H, W, C)), rng_int(8, (1, 1, C, R)), rng_int(9, (O, R))
    dY = rng_int(10, (N, H, W, O))
    y, _ = oracle.conv_fwd(x, U, V, 1, 0)
    yl, _ = oracle.linear_fwd(x.reshape(-1, C), U.reshape(C, R), V)
    np.testing.assert_array_equal(y.reshape(-1, O), yl)
    dX, dU, dV = oracle.conv_bwd(x, U, V, dY, 1, 0)
    dXl, dUl, dVl = oracle.linear_bwd(x.reshape(-1, C), U.reshape(C, R), V, dY.reshape(-1, O))
    np.testing.assert_array_equal(dX.reshape(-1, C), dXl)
    np.testing.assert_array_equal(dU.reshape(C, R), dUl)
    np.testing.assert_array_equal(dV, dVl)


def test_identity_projection_is_plain_correlation_scipy():
    """V = I (R = O): the layer is a plain multi-channel cross-correlation."""
    sig = pytest.importorskip("scipy.signal")
    N, H, W, C, R = 1, 6, 5, 2, 3
    x, U = rng_int(11, (N, H, W, C)), rng_int(12, (3, 3, C, R))
    y, _ = oracle.conv_fwd(x, U, np.eye(R), 1, 1)
    for j in range(R):
        want = sum(sig.correlate2d(x[0, :, :, c], U[:, :, c, j], mode="same") for c in range(C))
        np.testing.assert_array_equal(y[0, :, :, j], want)


def test_delta_kernel_passes_input_through():
    N, H, W, C = 2, 4, 5, 3
    x = rng_int(13, (N, H, W, C))
    U = np.zeros((3, 3, C, C))
    for c in range(C):
        U[1, 1, c, c] = 1.0
    V = rng_int(14, (4, C))
    y, T = oracle.conv_fwd(x, U, V, 1, 1)
    np.testing.assert_array_equal(T, x)
    np.testing.assert_array_equal(y, x @ V.T)


def test_shifted_delta_kernel_is_cross_correlation_not_flipped():
    """U[0,0] = 1 must read the upper-left neighbour (no kernel flip)."""
    x = rng_int(15, (1, 4, 4, 1))
    U = np.zeros((3, 3, 1, 1))
    U[0, 0, 0, 0] = 1.0
    _, T = oracle.conv_fwd(x, U, np.ones((1, 1)), 1, 1)
    want = np.zeros((4, 4))
    want[1:, 1:] = x[0, :-1, :-1, 0]
    np.testing.assert_array_equal(T[0, :, :, 0], want)


def test_dense_kernel_identity():
    """W[a,b,c,o] = sum_j U[a,b,c,j] V[o,j]: the factorized pair equals one dense conv."""
    N, H, W, C, R, O = 1, 5, 4, 2, 2, 3
    x, U, V = rng_int(16, (N, H, W, C)), rng_int(17, (3, 3, C, R)), rng_int(18, (O, R))
    Wd = np.einsum("abcj,oj->abco", U, V)
    y, _ = oracle.conv_fwd(x, U, V, 1, 1)
    yd, _ = oracle.conv_fwd(x, Wd, np.eye(O), 1, 1)
    np.testing.assert_array_equal(y, yd)


def test_fwd_brute_force_python_loops_stride2():
    N, H, W, C, R, O, st, pad = 1, 5, 6, 2, 2, 2, 2, 1
    x, U, V = rng_int(19, (N, H, W, C)), rng_int(20, (3, 3, C, R)), rng_int(21, (O, R))
    Ho, Wo = (H + 2 * pad - 3) // st + 1, (W + 2 * pad - 3) // st + 1
    want = np.zeros((N, Ho, Wo, O))
    for ho in range(Ho):
        for wo in range(Wo):
            for o in range(O):
                for j in range(R):
                    for a in range(3):
                        for b in range(3):
                            h, w = ho * st - pad + a, wo * st - pad + b
                            if 0 <= h < H and 0 <= w < W:
                                for c in range(C):
                                    want[0, ho, wo, o] += x[0, h, w, c] * U[a, b, c, j] * V[o, j]
    y, _ = oracle.conv_fwd(x, U, V, st, pad)
    assert y.shape == want.shape
    np.testing.assert_array_equal(y, want)


@pytest.mark.parametrize("st,pad", [(1, 1), (2, 1)])
def test_bwd_finite_differences_including_borders(st, pad):
    rng = np.random.default_rng(8)
    N, H, W, C, R, O = 2, 5, 4, 3, 2, 3
    x, U, V = rng.normal(size=(N, H, W, C)), rng.normal(size=(3, 3, C, R)), rng.normal(size=(O, R))
    Ho, Wo = oracle.conv_out_hw(H, W, 3, 3, st, pad)
    dY = rng.normal(size=(N, Ho, Wo, O))
    dX, dU, dV = oracle.conv_bwd(x, U, V, dY, st, pad)

    def loss(x_, U_, V_):
        return float(np.sum(dY * oracle.conv_fwd(x_, U_, V_, st, pad)[0]))

    h = 1e-6
    for arr, grad, idx in ((x, dX, 0), (U, dU, 1), (V, dV, 2)):
        fd = np.zeros_like(arr)
        for pos in np.ndindex(arr.shape):
            args = [x.copy(), U.copy(), V.copy()]
            args[idx][pos] += h
            up = loss(*args)
            args[idx][pos] -= 2 * h
            dn = loss(*args)
            fd[pos] = (up - dn) / (2 * h)
        assert oracle.rel_err(grad, fd) < 1e-7


def test_bwd_rank_column_and_image_slicing():
    """dU/dV columns depend only on the matching factor columns; dX of an image only on
    that image: the sampling used by full-size parity checks."""
    N, H, W, C, R, O = 3, 4, 4, 2, 4, 3
    x, U, V = rng_int(22, (N, H, W, C)), rng_int(23, (3, 3, C, R)), rng_int(24, (O, R))
    dY = rng_int(25, (N, H, W, O))
    dX, dU, dV = oracle.conv_bwd(x, U, V, dY)
    J = [0, 2]
    _, dUj, dVj = oracle.conv_bwd(x, U[..., J], V[:, J], dY)
    np.testing.assert_array_equal(dUj, dU[..., J])
    np.testing.assert_array_equal(dVj, dV[:, J])
    dX1, _, _ = oracle.conv_bwd(x[1:2], U, V, dY[1:2])
    np.testing.assert_array_equal(dX1[0], dX[1])
