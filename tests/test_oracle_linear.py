"""Pins for the fp64 oracle of the factorized FC layer (Section 2.1, Appendix B "FC layer").

None of these re-type the oracle's own loops: they check it against a hand-computed
example, the dense identity, textbook special cases, the dense chain rule, finite
differences and pure-Python brute force of the index definition.
"""
import os

import numpy as np
import pytest

import oracle
from _util import read_golden, rng_int


def test_hand_case(golden_dir):
    g = read_golden(os.path.join(golden_dir, "linear_hand_case.txt"))
    y, T = oracle.linear_fwd(g["x"], g["U"], g["V"])
    dX, dU, dV = oracle.linear_bwd(g["x"], g["U"], g["V"], g["dY"])
    for got, want in ((y, "y"), (T, "T"), (dX, "dX"), (dU, "dU"), (dV, "dV")):
        np.testing.assert_array_equal(got, g[want])


@pytest.mark.parametrize("m,k,n,r", [(1, 1, 1, 1), (5, 7, 3, 2), (4, 3, 9, 5), (13, 6, 2, 11)])
def test_fwd_dense_identity(m, k, n, r):
    """(xU)V^T = x(UV^T): W ~ U V^T is the whole point of Section 2.1."""
    x, U, V = rng_int(1, (m, k)), rng_int(2, (k, r)), rng_int(3, (n, r))
    y, T = oracle.linear_fwd(x, U, V)
    np.testing.assert_array_equal(y, x @ (U @ V.T))
    np.testing.assert_array_equal(T, x @ U)


def test_fwd_dense_identity_real_values():
    rng = np.random.default_rng(0)
    x, U, V = rng.normal(size=(17, 23)), rng.normal(size=(23, 5)), rng.normal(size=(11, 5))
    y, _ = oracle.linear_fwd(x, U, V)
    assert oracle.rel_err(y, x @ (U @ V.T)) < 1e-13


def test_fwd_identity_factor_is_plain_matmul():
    """r = k and U = I reduces the layer to the textbook product x V^T."""
    x, V = rng_int(4, (6, 5)), rng_int(5, (8, 5))
    y, T = oracle.linear_fwd(x, np.eye(5), V)
    np.testing.assert_array_equal(y, x @ V.T)
    np.testing.assert_array_equal(T, x)


def test_fwd_brute_force_python_loops():
    m, k, n, r = 3, 4, 5, 2
    x, U, V = rng_int(6, (m, k)), rng_int(7, (k, r)), rng_int(8, (n, r))
    want = np.zeros((m, n))
    for i in range(m):
        for o in range(n):
            for j in range(r):
                for c in range(k):
                    want[i, o] += x[i, c] * U[c, j] * V[o, j]
    y, _ = oracle.linear_fwd(x, U, V)
    np.testing.assert_array_equal(y, want)


@pytest.mark.parametrize("m,k,n,r", [(5, 7, 3, 2), (4, 3, 9, 5), (2, 6, 6, 8)])
def test_bwd_dense_chain_rule(m, k, n, r):
    """Dense layer y = xW, W = UV^T: dW = x^T dY, dX = dY W^T, then dU = dW V, dV = dW^T U."""
    x, U, V, dY = (rng_int(10, (m, k)), rng_int(11, (k, r)), rng_int(12, (n, r)),
                   rng_int(13, (m, n)))
    dX, dU, dV = oracle.linear_bwd(x, U, V, dY)
    W = U @ V.T
    dW = x.T @ dY
    np.testing.assert_array_equal(dX, dY @ W.T)
    np.testing.assert_array_equal(dU, dW @ V)
    np.testing.assert_array_equal(dV, dW.T @ U)


def test_bwd_finite_differences():
    """L = sum(dY * y); central differences in every entry of x, U, V."""
    rng = np.random.default_rng(3)
    m, k, n, r = 4, 5, 6, 3
    x, U, V, dY = (rng.normal(size=(m, k)), rng.normal(size=(k, r)), rng.normal(size=(n, r)),
                   rng.normal(size=(m, n)))
    dX, dU, dV = oracle.linear_bwd(x, U, V, dY)

    def loss(x_, U_, V_):
        return float(np.sum(dY * oracle.linear_fwd(x_, U_, V_)[0]))

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


def test_bwd_is_plain_sum_over_rows_no_mean():
    """Stacking the same batch twice doubles dU and dV (no 1/m anywhere)."""
    x, U, V, dY = rng_int(20, (3, 4)), rng_int(21, (4, 2)), rng_int(22, (5, 2)), rng_int(23, (3, 5))
    _, dU1, dV1 = oracle.linear_bwd(x, U, V, dY)
    _, dU2, dV2 = oracle.linear_bwd(np.vstack([x, x]), U, V, np.vstack([dY, dY]))
    np.testing.assert_array_equal(dU2, 2 * dU1)
    np.testing.assert_array_equal(dV2, 2 * dV1)


def test_rank_column_slicing_gives_matching_gradient_columns():
    """dU[:, J] and dV[:, J] only depend on columns J of U and V: this is what lets
    full-size parity checks sample the factor gradients."""
    x, U, V, dY = rng_int(30, (6, 5)), rng_int(31, (5, 4)), rng_int(32, (7, 4)), rng_int(33, (6, 7))
    _, dU, dV = oracle.linear_bwd(x, U, V, dY)
    J = [1, 3]
    _, dUj, dVj = oracle.linear_bwd(x, U[:, J], V[:, J], dY)
    np.testing.assert_array_equal(dUj, dU[:, J])
    np.testing.assert_array_equal(dVj, dV[:, J])


def test_widen_bf16_bits_exact():
    bits = np.array([0x3F80, 0xBF80, 0x4000, 0x3F00, 0x0000, 0x3FC0], dtype=np.uint16)
    np.testing.assert_array_equal(oracle.widen(bits), [1.0, -1.0, 2.0, 0.5, 0.0, 1.5])


def test_rel_err_metric():
    a = np.array([3.0, 4.0])
    assert oracle.rel_err(a, a) == 0.0
    assert abs(oracle.rel_err(a + np.array([0.3, 0.4]), a) - 0.1) < 1e-15


def test_widen_returns_c_contiguous_for_sliced_bit_patterns():
    """Column-sliced bf16 bit patterns (as used for sampled parity) must be marshalled in C order."""
    import pf_workloads as wl
    U = wl.round_to(np.arange(24, dtype=np.float64).reshape(2, 3, 4), wl.BF16)
    w = oracle.widen(U[..., [0, 2]])
    assert w.flags["C_CONTIGUOUS"]
    np.testing.assert_array_equal(w, np.arange(24.0).reshape(2, 3, 4)[..., [0, 2]])


# ---------------------------------------------------------------------------------------------
# grouped layer (per-gate LSTM factors of Section 2.3, attention projections of Section 2.4)
def test_grouped_shared_input_equals_one_dense_layer_with_concatenated_weights():
    """G factor pairs reading one x are the dense layer x [W_1 | ... | W_G] with W_g = U_g V_g^T
    (the way the four gates of an LSTM are usually stored): outputs are its column blocks, and the
    input gradient is dY_cat W_cat^T, i.e. the SUM over the groups.  Integers: exact."""
    G, m, k, n, r = 3, 5, 4, 6, 2
    x = rng_int(1, (m, k)); U = rng_int(2, (G, k, r)); V = rng_int(3, (G, n, r)); dY = rng_int(4, (G, m, n))
    y, T = oracle.linear_grouped_fwd(x, U, V)
    W_cat = np.concatenate([U[g] @ V[g].T for g in range(G)], axis=1)          # k x (G n)
    np.testing.assert_array_equal(np.concatenate(list(y), axis=1), x @ W_cat)
    np.testing.assert_array_equal(T, np.stack([x @ U[g] for g in range(G)]))
    dX, dU, dV = oracle.linear_grouped_bwd(x, U, V, dY)
    dY_cat = np.concatenate(list(dY), axis=1)
    np.testing.assert_array_equal(dX, dY_cat @ W_cat.T)
    dW_cat = x.T @ dY_cat                                                        # dense weight gradient
    for g in range(G):
        dW = dW_cat[:, g * n:(g + 1) * n]
        np.testing.assert_array_equal(dU[g], dW @ V[g])
        np.testing.assert_array_equal(dV[g], dW.T @ U[g])


def test_grouped_own_inputs_is_a_block_diagonal_layer():
    """Groups with their own x are one layer on the concatenated input with a block-diagonal weight:
    nothing mixes between groups, dX stays per group."""
    G, m, k, n, r = 2, 4, 3, 5, 2
    x = rng_int(5, (G, m, k)); U = rng_int(6, (G, k, r)); V = rng_int(7, (G, n, r)); dY = rng_int(8, (G, m, n))
    W = np.zeros((G * k, G * n))
    for g in range(G):
        W[g * k:(g + 1) * k, g * n:(g + 1) * n] = U[g] @ V[g].T
    x_cat = np.concatenate(list(x), axis=1)
    y, _ = oracle.linear_grouped_fwd(x, U, V)
    np.testing.assert_array_equal(np.concatenate(list(y), axis=1), x_cat @ W)
    dX, dU, dV = oracle.linear_grouped_bwd(x, U, V, dY)
    np.testing.assert_array_equal(np.concatenate(list(dX), axis=1), np.concatenate(list(dY), axis=1) @ W.T)
    for g in range(G):   # a group alone gives the same factor gradients
        _, dU1, dV1 = oracle.linear_bwd(x[g], U[g], V[g], dY[g])
        np.testing.assert_array_equal(dU[g], dU1)
        np.testing.assert_array_equal(dV[g], dV1)


def test_grouped_parameter_count_matches_the_lstm_table():
    """Per-gate factorization of one LSTM layer: 8 factor pairs of 1500 x 375 / 375 x 1500 (Table 1:
    4dr + 12hr parameters with d = h = 1500, r = 375)."""
    d = h = 1500
    r = 375
    assert 8 * r * (d + h) == 4 * d * r + 12 * h * r


# ---- bias and activation after the factorized layer (Section 2.4: FFN(x) = max(0, x W1 + b1) W2 + b2)

def test_bias_relu_hand_example():
    """x = [1, -2], U = [[1], [1]] (T = -1), V = [[2], [-3]] gives (xU)V^T = [-2, 3]; with bias
    [0.5, 0.5] that is [-1.5, 3.5], and max(0, .) leaves [0, 3.5]."""
    x = np.array([[1.0, -2.0]], dtype=np.float32)
    U = np.array([[1.0], [1.0]], dtype=np.float32)
    V = np.array([[2.0], [-3.0]], dtype=np.float32)
    b = np.array([0.5, 0.5], dtype=np.float32)
    y, T = oracle.linear_fwd_act(x, U, V, b, relu=True)
    np.testing.assert_array_equal(T, [[-1.0]])
    np.testing.assert_array_equal(y, [[0.0, 3.5]])
    y, _ = oracle.linear_fwd_act(x, U, V, b, relu=False)
    np.testing.assert_array_equal(y, [[-1.5, 3.5]])
    y, _ = oracle.linear_fwd_act(x, U, V, None, relu=True)
    np.testing.assert_array_equal(y, [[0.0, 3.0]])


@pytest.mark.parametrize("m,k,n,r", [(5, 7, 6, 3), (9, 4, 11, 4)])
def test_bias_relu_equals_the_dense_ffn_half(m, k, n, r):
    """max(0, x W + b) with the dense W = U V^T formed first (the other association order), in
    integers so that both orders are exact; and the whole block FFN(x) = max(0, x W1 + b1) W2 + b2."""
    x, U, V = rng_int(1, (m, k)), rng_int(2, (k, r)), rng_int(3, (n, r))
    b = rng_int(4, (n,))
    W = U.astype(np.float64) @ V.astype(np.float64).T
    want = np.maximum(x.astype(np.float64) @ W + b, 0.0)
    got, _ = oracle.linear_fwd_act(x, U, V, b, relu=True)
    np.testing.assert_array_equal(got, want)
    assert (got == 0).any() and (got > 0).any()          # the case exercises both branches
    # second half of the block on top of it (no activation), against the dense formula
    U2, V2, b2 = rng_int(5, (n, r)), rng_int(6, (k, r)), rng_int(7, (k,))
    h = got.astype(np.float32)
    ffn, _ = oracle.linear_fwd_act(h, U2, V2, b2, relu=False)
    W2 = U2.astype(np.float64) @ V2.astype(np.float64).T
    np.testing.assert_array_equal(ffn, want @ W2 + b2)


def test_bias_relu_properties():
    rng = np.random.default_rng(11)
    x, U, V = (rng.standard_normal(s).astype(np.float32) for s in ((6, 5), (5, 3), (4, 3)))
    b = rng.standard_normal(4).astype(np.float32)
    y0, T0 = oracle.linear_fwd(x, U, V)
    y1, T1 = oracle.linear_fwd_act(x, U, V, None, relu=False)
    np.testing.assert_array_equal(y0, y1)                 # no bias, no activation: the plain layer
    np.testing.assert_array_equal(T0, T1)
    yb, _ = oracle.linear_fwd_act(x, U, V, b, relu=False)
    np.testing.assert_allclose(yb - y0, np.broadcast_to(b.astype(np.float64), y0.shape), rtol=0, atol=1e-12)
    yr, _ = oracle.linear_fwd_act(x, U, V, b, relu=True)
    assert (yr >= 0).all()
    np.testing.assert_array_equal(yr, np.where(yb > 0, yb, 0.0))
    # positive homogeneity of max(0, .): scaling x and the bias by 4 (exact in binary) scales y by 4
    y4, _ = oracle.linear_fwd_act(4 * x, U, V, 4 * b, relu=True)
    np.testing.assert_array_equal(y4, 4 * yr)


def test_bias_act_bwd_hand_example_and_autograd():
    """y = max(0, z + b) with y = [[0, 2], [3, 0]] and dY = [[5, 7], [11, 13]]: dZ keeps dY where
    y > 0 -> [[0, 7], [11, 0]], dbias = column sums [11, 7].  And fp64 autograd of relu(z + b)."""
    y = np.array([[0.0, 2.0], [3.0, 0.0]], dtype=np.float32)
    dY = np.array([[5.0, 7.0], [11.0, 13.0]], dtype=np.float32)
    dZ, db = oracle.bias_act_bwd(y, dY, relu=True)
    np.testing.assert_array_equal(dZ, [[0.0, 7.0], [11.0, 0.0]])
    np.testing.assert_array_equal(db, [11.0, 7.0])
    dZ, db = oracle.bias_act_bwd(y, dY, relu=False)
    np.testing.assert_array_equal(dZ, dY)
    np.testing.assert_array_equal(db, [16.0, 20.0])
    import torch
    rng = np.random.default_rng(5)
    z = torch.tensor(rng.standard_normal((9, 6)), dtype=torch.float64, requires_grad=True)
    b = torch.tensor(rng.standard_normal(6), dtype=torch.float64, requires_grad=True)
    g = rng.standard_normal((9, 6))
    out = torch.relu(z + b)
    out.backward(torch.tensor(g))
    dZ, db = oracle.bias_act_bwd(out.detach().numpy().astype(np.float32), g.astype(np.float32), relu=True)
    np.testing.assert_allclose(dZ, z.grad.numpy(), rtol=0, atol=1e-6)
    np.testing.assert_allclose(db, b.grad.numpy(), rtol=0, atol=1e-5)
