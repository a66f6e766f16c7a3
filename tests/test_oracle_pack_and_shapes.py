"""Pins for the flat gradient buffer (Section 4.1 "Implementation details and
optimizations") and for the factor shapes used as workloads (Table 1 closed forms,
Table 2 totals, appendix architecture tables)."""
import os

import numpy as np
import pytest

import oracle
import pf_workloads as wl
from _util import read_counts


def _brute_pack(grads):
    out, offs = [], [0]
    for g in grads:
        for v in g.reshape(-1):
            out.append(v)
        offs.append(offs[-1] + g.size)
    return np.array(out, dtype=grads[0].dtype), np.array(offs, dtype=np.int64)


@pytest.mark.parametrize("numels", [[1], [3, 5], [7, 0, 2, 1], [16, 1, 15, 33, 2]])
@pytest.mark.parametrize("dt", [np.uint16, np.float32])
def test_pack_brute_force_and_invariants(numels, dt):
    rng = np.random.default_rng(1)
    grads = [rng.integers(0, 60000, size=n).astype(dt) for n in numels]
    flat, offs = oracle.pack(grads)
    want, woffs = _brute_pack(grads)
    assert flat.dtype == dt and flat.tobytes() == want.tobytes()
    np.testing.assert_array_equal(offs, woffs)
    assert offs[0] == 0 and offs[-1] == sum(numels) and np.all(np.diff(offs) >= 0)
    for i, g in enumerate(grads):                       # unpack is the inverse
        np.testing.assert_array_equal(flat[offs[i]:offs[i + 1]], g)


def test_pack_empty_list():
    flat, offs = oracle.pack([])
    assert flat.size == 0 and list(offs) == [0]


def test_table1_closed_forms_match_workload_shapes(golden_dir):
    g = read_counts(os.path.join(golden_dir, "paper_counts.txt"))
    lin, conv = wl.linear_cases(), wl.conv_cases()
    # Factorized FC: r(m+n) parameters (Table 1).  FFN: 10 p d r (Table 1) at pd=512, r=128.
    pd, r = g["ffn_pd"], g["ffn_r"]
    up, down = lin["C2a"], lin["C2b"]
    assert (up.k, up.n, up.r, down.k, down.n, down.r) == (pd, 4 * pd, r, 4 * pd, pd, r)
    ffn_params = up.r * (up.k + up.n) + down.r * (down.k + down.n)
    assert ffn_params == 10 * pd * r == 655360
    # Factorized conv: c_in r k^2 + r c_out (Table 1), ResNet-18 conv4_x and VGG conv10.
    cu, cv = g["resnet18_conv4_u"], g["resnet18_conv4_v"]
    c4 = conv["C4"]
    assert (c4.C, c4.R, c4.kh, c4.kw) == cu and (c4.R, c4.O) == cv[:2]
    assert c4.C * c4.R * 9 + c4.R * c4.O == 147456 + 16384 == 163840
    vu, vv = g["vgg_conv_u"], g["vgg_conv_v"]
    assert vu[0] * vu[1] * vu[2] * vu[3] + vv[0] * vv[1] == 655360
    # Pack total of the C4 factor gradients equals the closed form.
    _, offs = oracle.pack([np.zeros(c4.kh * c4.kw * c4.C * c4.R, np.uint16),
                           np.zeros(c4.O * c4.R, np.uint16)])
    assert offs[-1] == 163840


def test_lstm_saving_confirms_per_gate_factor_shapes(golden_dir):
    """Table 2's parameter saving equals layers x (4(dh+h^2) - (4dr+12hr)) (Table 1)."""
    g = read_counts(os.path.join(golden_dir, "paper_counts.txt"))
    d, h, r, L = g["lstm_d"], g["lstm_h"], g["lstm_r"], g["lstm_layers"]
    saving = g["lstm_params_vanilla"] - g["lstm_params_lowrank"]
    assert saving == L * (4 * (d * h + h * h) - (4 * d * r + 12 * h * r)) == 18000000
    c3 = wl.linear_cases()["C3i"]
    assert (c3.k, c3.n, c3.r) == (d, 4 * h, r)


def test_generator_is_deterministic_and_rounded_once():
    a = wl.LinearCase("t", 5, 7, 3, 2, wl.BF16, 9).generate()
    b = wl.LinearCase("t", 5, 7, 3, 2, wl.BF16, 9).generate()
    for kx in a:
        assert a[kx].dtype == np.uint16 and np.array_equal(a[kx], b[kx])
    # bf16 RNE: 1 + 2^-8 is a tie and rounds to even (1.0); 1 + 3*2^-9 rounds up
    r = wl.round_to(np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -9, -2.5]), wl.BF16)
    np.testing.assert_array_equal(oracle.widen(r), [1.0, 1.0 + 2.0 ** -7, -2.5])
    # one rounding, not two: just above / below a bf16 tie by less than fp32 can hold (going
    # through fp32 first would land on the tie and then on the even neighbour)
    eps = 2.0 ** -40
    r = wl.round_to(np.array([1.0 + 2.0 ** -8 + eps, 1.0 + 3 * 2.0 ** -8 - eps,
                              -(1.0 + 2.0 ** -8 + eps), -(1.0 + 3 * 2.0 ** -8 - eps)]), wl.BF16)
    np.testing.assert_array_equal(oracle.widen(r), [1.0 + 2.0 ** -7, 1.0 + 2.0 ** -7,
                                                    -(1.0 + 2.0 ** -7), -(1.0 + 2.0 ** -7)])
    # agreement with an exact rational rounding on random values
    from fractions import Fraction
    vals = wl.normal(77, 0, (300,))
    got = oracle.widen(wl.round_to(vals, wl.BF16))
    for v, g in zip(vals, got):
        e = int(np.floor(np.log2(abs(v))))
        ulp = Fraction(2) ** (e - 7)
        q = Fraction(v) / ulp
        lo = q.numerator // q.denominator
        frac = q - lo
        n = lo + (1 if frac > Fraction(1, 2) or (frac == Fraction(1, 2) and lo % 2) else 0)
        assert Fraction(g) == n * ulp


def test_generator_distributions():
    z = wl.normal(3, 0, (200000,))
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1.0) < 0.01
    u = wl.uniform(3, 1, (200000,))
    assert u.min() > -1 and u.max() < 1 and abs(u.mean()) < 0.01 and abs(u.std() - 3 ** -0.5) < 0.01
    c = wl.conv_cases()["C4"]
    small = wl.ConvCase("s", 2, 8, 8, c.C, c.R, c.O, wl.F32, c.seed).generate()
    assert small["x"].min() == 0.0 and (small["x"] == 0).mean() > 0.4      # post-ReLU
    assert abs(small["U"].std() - (2.0 / (9 * c.C)) ** 0.5) < 2e-3          # Kaiming fan-in


@pytest.mark.parametrize("numels", [[1], [3, 5], [7, 0, 2, 1], [16, 1, 15, 33, 2]])
@pytest.mark.parametrize("dt", [np.uint16, np.float32])
def test_unpack_is_the_inverse_of_pack(numels, dt):
    rng = np.random.default_rng(2)
    grads = [rng.integers(0, 60000, size=n).astype(dt) for n in numels]
    flat, offs = oracle.pack(grads)
    back, offs2 = oracle.unpack(flat, numels)
    np.testing.assert_array_equal(offs, offs2)
    assert len(back) == len(grads)
    for b, g in zip(back, grads):
        assert b.dtype == dt and b.tobytes() == g.tobytes()
    # and slicing by the prefix sums (the definition) gives the same
    for i, b in enumerate(back):
        np.testing.assert_array_equal(b, flat[offs[i]:offs[i + 1]])
