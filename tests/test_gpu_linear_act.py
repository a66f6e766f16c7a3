"""GPU parity: the factorized linear forward with bias and activation (Section 2.4) vs the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2103_03936_b200 as pf
import pf_workloads as wl
from _gpu import Guarded, assert_blocks_close, assert_close, dev

pytestmark = pytest.mark.gpu


def run_act(case, bias=True, relu=True, stash=True, ld_pad=0):
    d = case.generate()
    dt = case.dtype
    m, k, n, r = case.m, case.k, case.n, case.r
    b_host = wl.round_to(wl.normal(case.seed, 7, (n,), 0.5), dt) if bias else None

    def up(a, cols):
        if not ld_pad:
            return dev(a, dt)
        buf = torch.zeros((a.shape[0], cols + ld_pad), dtype=wl.to_torch(a[:1], dt).dtype, device="cuda")
        buf[:, :cols] = dev(a, dt)
        return buf[:, :cols]

    x, U, V = up(d["x"], k), up(d["U"], r), up(d["V"], r)
    b = dev(b_host, dt) if bias else None
    gy = Guarded((m, n), dt, ld=n + ld_pad if ld_pad else None)
    gT = Guarded((m, r), dt, ld=r + ld_pad if ld_pad else None)
    l0 = pf.pf_launch_count()
    pf.pf_lowrank_linear_fwd_act(x, U, V, bias=b, act=pf.PF_ACT_RELU if relu else pf.PF_ACT_NONE, y=gy.t,
                                 T_stash=gT.t if stash else None)
    launches = pf.pf_launch_count() - l0
    torch.cuda.synchronize()
    y_ref, T_ref = oracle.linear_fwd_act(d["x"], d["U"], d["V"], b_host, relu=relu)
    tag = f"{case.name} {m}x{k}->{n} r{r} {dt} bias={bias} relu={relu} "
    assert_close(gy.t, y_ref, dt, tag + "y")
    if m >= 128 and n >= 128:
        assert_blocks_close(gy.t, y_ref, dt, tag + "y")
    if stash:
        assert_close(gT.t, T_ref, dt, tag + "T")
    if relu:
        assert float(gy.t.float().min()) >= 0.0
        # the activation really cut something, and kept something
        assert (y_ref == 0).mean() > 0.1 and (y_ref > 0).mean() > 0.1
    gy.check()
    gT.check()
    assert pf.pf_last_device_status() == 0
    return launches


@pytest.mark.parametrize("bias,relu", [(True, True), (True, False), (False, True)])
@pytest.mark.parametrize("m,k,n,r", [(2100, 200, 328, 40), (4100, 72, 1000, 136), (2050, 104, 136, 32)])
def test_fused_kernel_epilogue(m, k, n, r, bias, relu):
    """m >= 2048, r <= 192: bias and activation run in the fused kernel's output epilogue (one launch),
    on ragged row tiles and ragged last column tiles (n = 328: 72 valid columns, n = 136: 8)."""
    launches = run_act(wl.LinearCase("act", m, k, n, r, wl.BF16, 31), bias=bias, relu=relu)
    assert launches == 1


def test_fused_kernel_epilogue_persistent_and_ffn_shape():
    """More row tiles than SMs (persistent form of the kernel), and the Transformer FFN up-projection
    at half its batch (the shape the epilogue exists for: max(0, x W1 + b1))."""
    assert run_act(wl.LinearCase("act", 19500, 200, 128, 64, wl.BF16, 32)) == 1
    assert run_act(wl.LinearCase("act", 4096, 512, 2048, 128, wl.BF16, 33), stash=False) == 1


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
@pytest.mark.parametrize("m,k,n,r", [(300, 136, 72, 24), (77, 33, 50, 7), (700, 200, 264, 200)])
def test_unfused_paths(dtype, m, k, n, r):
    """Few rows, odd widths, fp32: the products run unfused (tensor-core or FMA kernels) and bias and
    activation follow in a pass of their own."""
    run_act(wl.LinearCase("act", m, k, n, r, dtype, 34), bias=True, relu=True)
    run_act(wl.LinearCase("act", m, k, n, r, dtype, 35), bias=True, relu=False, stash=False)


def test_padded_pitches_untouched():
    run_act(wl.LinearCase("act", 2100, 72, 136, 24, wl.BF16, 36), ld_pad=8)
    run_act(wl.LinearCase("act", 200, 72, 136, 24, wl.F32, 37), ld_pad=3)


def test_no_bias_no_activation_equals_plain_forward_bitwise():
    c = wl.LinearCase("act", 2100, 200, 328, 40, wl.BF16, 38)
    d = c.generate()
    x, U, V = dev(d["x"], c.dtype), dev(d["U"], c.dtype), dev(d["V"], c.dtype)
    y0 = pf.pf_lowrank_linear_fwd(x, U, V)
    y1 = pf.pf_lowrank_linear_fwd_act(x, U, V)
    assert torch.equal(y0, y1)


def test_bad_arguments():
    c = wl.LinearCase("act", 64, 32, 48, 8, wl.BF16, 39)
    d = c.generate()
    x, U, V = dev(d["x"], c.dtype), dev(d["U"], c.dtype), dev(d["V"], c.dtype)
    with pytest.raises(pf.PfError):
        pf.pf_lowrank_linear_fwd_act(x, U, V, act=7)
    with pytest.raises(ValueError):
        pf.pf_lowrank_linear_fwd_act(x, U, V, bias=torch.zeros(47, dtype=torch.bfloat16, device="cuda"))


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
@pytest.mark.parametrize("relu", [True, False])
@pytest.mark.parametrize("m,n,ld_pad", [(1, 1, 0), (77, 50, 3), (700, 264, 0), (4100, 1000, 8), (20000, 33, 0)])
def test_bias_act_bwd(dtype, relu, m, n, ld_pad):
    """dZ in place over dY (bit-exact: a copy or a zero), dbias = column sums against the oracle;
    guard bands and row padding untouched."""
    y64 = np.maximum(wl.normal(61, 0, (m, n)), 0.0)
    y_h = wl.round_to(y64, dtype)
    g_h = wl.round_to(wl.normal(61, 1, (m, n)), dtype)
    gy = Guarded((m, n), dtype, ld=n + ld_pad if ld_pad else None)
    gd = Guarded((m, n), dtype, ld=n + ld_pad if ld_pad else None)
    gb = Guarded((1, n), dtype)
    gy.t.copy_(dev(y_h, dtype))
    gd.t.copy_(dev(g_h, dtype))
    pf.pf_bias_act_bwd(gy.t, gd.t, act=pf.PF_ACT_RELU if relu else pf.PF_ACT_NONE, dbias=gb.t.view(-1))
    torch.cuda.synchronize()
    dZ_ref, db_ref = oracle.bias_act_bwd(y_h, g_h, relu=relu)
    got = oracle.widen(wl.from_torch(gd.t.contiguous(), dtype))
    np.testing.assert_array_equal(got, dZ_ref)
    assert_close(gb.t.view(-1), db_ref, dtype, f"dbias {m}x{n} {dtype} relu={relu}", tol=1e-2 if dtype == wl.BF16 else 1e-4)
    for g in (gy, gd, gb):
        g.check()
    # without dbias: one launch, no workspace
    gd.t.copy_(dev(g_h, dtype))
    l0 = pf.pf_launch_count()
    assert pf.pf_bias_act_bwd(gy.t, gd.t, act=pf.PF_ACT_RELU if relu else pf.PF_ACT_NONE, want_dbias=False) is None
    assert pf.pf_launch_count() - l0 == 1
    assert pf.pf_last_device_status() == 0
