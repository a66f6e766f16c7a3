"""GPU parity: grouped factorized linear layers (several factor pairs of one shape in one call)
through the C ABI vs the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2103_03936_b200 as pf
import pf_workloads as wl
from _gpu import Guarded, TDT, assert_blocks_close, assert_close, dev

pytestmark = pytest.mark.gpu


def make(G, m, k, n, r, dtype, seed, shared_x):
    """Seeded inputs of G layers: x [G, m, k] (or one [m, k]), U [G, k, r], V [G, n, r], dY [G, m, n]."""
    sig = 1.0 / np.sqrt(k)
    x = wl.round_to(wl.normal(seed, 0, (m, k) if shared_x else (G, m, k)), dtype)
    U = wl.round_to(wl.normal(seed, 1, (G, k, r), sig), dtype)
    V = wl.round_to(wl.normal(seed, 2, (G, n, r), sig), dtype)
    dY = wl.round_to(wl.normal(seed, 3, (G, m, n)), dtype)
    return x, U, V, dY


def padded(a, dtype, ld):
    """Device copy whose rows are ld elements apart (ld >= the row length)."""
    t = dev(a, dtype)
    buf = torch.zeros(t.shape[:-1] + (ld,), dtype=t.dtype, device="cuda")
    buf[..., :t.shape[-1]] = t
    return buf[..., :t.shape[-1]]


def run_grouped(G, m, k, n, r, dtype, seed, shared_x, stash=True, need_dX=True, pad_to=None, blocks=False):
    x_h, U_h, V_h, dY_h = make(G, m, k, n, r, dtype, seed, shared_x)
    if pad_to:   # row pitches rounded up to a multiple of pad_to elements
        up = lambda v: (v + pad_to - 1) // pad_to * pad_to
        x, U, V, dY = padded(x_h, dtype, up(k)), padded(U_h, dtype, up(r)), padded(V_h, dtype, up(r)), padded(dY_h, dtype, up(n))
    else:
        x, U, V, dY = (dev(a, dtype) for a in (x_h, U_h, V_h, dY_h))
    gy = Guarded((G, m, n), dtype)
    if pad_to:   # the stash at a padded pitch too, so that it can be read back as an operand
        gT = Guarded((G * m, r), dtype, ld=(r + pad_to - 1) // pad_to * pad_to)
        T_t = gT.t.unflatten(0, (G, m))
    else:
        gT = Guarded((G, m, r), dtype)
        T_t = gT.t
    before = pf.pf_launch_count()
    pf.pf_lowrank_linear_grouped_fwd(x, U, V, y=gy.t, T_stash=T_t if stash else None)
    launches_fwd = pf.pf_launch_count() - before
    gdX = Guarded((m, k) if shared_x else (G, m, k), dtype)
    gdU, gdV = Guarded((G, k, r), dtype), Guarded((G, n, r), dtype)
    before = pf.pf_launch_count()
    pf.pf_lowrank_linear_grouped_bwd(x, U, V, dY, T_stash=T_t if stash else None, need_dX=need_dX,
                                     dX=gdX.t if need_dX else None, dU=gdU.t, dV=gdV.t)
    launches_bwd = pf.pf_launch_count() - before
    torch.cuda.synchronize()
    y_ref, T_ref = oracle.linear_grouped_fwd(x_h, U_h, V_h)
    dX_ref, dU_ref, dV_ref = oracle.linear_grouped_bwd(x_h, U_h, V_h, dY_h)
    tag = f"G{G} {m}x{k}->{n} r{r} {dtype} {'shared' if shared_x else 'own'} x "
    checks = [("y", gy, y_ref), ("dU", gdU, dU_ref), ("dV", gdV, dV_ref)]
    if stash:
        checks.append(("T", gT, T_ref))
    if need_dX:
        checks.append(("dX", gdX, dX_ref))
    for nm, g, ref in checks:
        got = T_t if nm == "T" else g.t
        # per group: a wrong group cannot hide in the norm over all of them
        if got.dim() == 3:
            for q in range(G):
                assert_close(got[q], ref[q], dtype, f"{tag}{nm}[{q}]")
                if blocks:
                    assert_blocks_close(got[q], ref[q], dtype, f"{tag}{nm}[{q}]")
        else:
            assert_close(got, ref, dtype, tag + nm)
            if blocks:
                assert_blocks_close(got, ref, dtype, tag + nm)
    for g in (gy, gT, gdX, gdU, gdV):
        g.check()
    assert pf.pf_last_device_status() == 0
    return launches_fwd, launches_bwd


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
@pytest.mark.parametrize("shared_x", [False, True])
def test_small_and_ragged_shapes_run_group_by_group(dtype, shared_x):
    """fp32, and bf16 layouts TMA cannot describe, take the ungrouped kernels group by group."""
    run_grouped(3, 37, 20, 29, 5, dtype, 201, shared_x)
    run_grouped(2, 130, 17, 24, 33, dtype, 202, shared_x, stash=False)
    run_grouped(4, 7, 100, 3, 1, dtype, 203, shared_x, need_dX=False)


@pytest.mark.parametrize("shared_x", [False, True])
@pytest.mark.parametrize("G,m,k,n,r", [(4, 300, 136, 264, 40), (3, 1000, 328, 520, 96), (5, 129, 64, 72, 64),
                                       (2, 2500, 200, 136, 136)])
def test_tensor_core_path_two_launches_each_way(G, m, k, n, r, shared_x):
    """bf16 with 16-byte aligned pitches and strides: all groups in two launches forward and two
    backward (three when the intermediate has to be recomputed), ragged row / column / rank tails."""
    lf, lb = run_grouped(G, m, k, n, r, wl.BF16, 210, shared_x)
    assert (lf, lb) == (2, 2)
    lf, lb = run_grouped(G, m, k, n, r, wl.BF16, 211, shared_x, stash=False, need_dX=False)
    assert (lf, lb) == (2, 3)


@pytest.mark.parametrize("pad_to", [None, 8])
def test_lstm_per_gate_shape(pad_to):
    """The eight gate matrices of one factorized LSTM layer (appendix LSTM table: 1500 x 375 and
    375 x 1500 factors per gate), m = 700 rows.  The four input gates share x_t; here all eight
    groups share one input, the worst case for the summed input gradient.  Tight pitches (3000 and
    750 bytes) run group by group; pitches padded to 16 bytes take the two-launch path."""
    lf, lb = run_grouped(8, 700, 1500, 1500, 375, wl.BF16, 220, True, pad_to=pad_to, blocks=True)
    if pad_to:
        assert (lf, lb) == (2, 2)


@pytest.mark.parametrize("shared_x", [True, False])
def test_attention_projection_shape(shared_x):
    """Four 512 -> 512 projections at rank 128 (Section 2.4 / Appendix D) on 8192 tokens."""
    lf, lb = run_grouped(4, 8192, 512, 512, 128, wl.BF16, 230, shared_x, blocks=True)
    assert (lf, lb) == (2, 2)


def test_grouped_backward_is_bit_reproducible():
    G, m, k, n, r = 4, 4096, 256, 320, 64
    x_h, U_h, V_h, dY_h = make(G, m, k, n, r, wl.BF16, 240, False)
    x, U, V, dY = (dev(a, wl.BF16) for a in (x_h, U_h, V_h, dY_h))
    a = pf.pf_lowrank_linear_grouped_bwd(x, U, V, dY)
    b = pf.pf_lowrank_linear_grouped_bwd(x, U, V, dY)
    torch.cuda.synchronize()
    for p, q in zip(a, b):
        assert torch.equal(p, q)
    assert pf.pf_last_device_status() == 0


def test_invalid_arguments_are_refused_on_the_host():
    U = torch.zeros((2, 8, 4), dtype=torch.bfloat16, device="cuda")
    V = torch.zeros((2, 6, 4), dtype=torch.bfloat16, device="cuda")
    x = torch.zeros((5, 8), dtype=torch.bfloat16, device="cuda")
    before = pf.pf_launch_count()
    with pytest.raises(pf.PfError) as e:     # workspace too small
        pf.pf_lowrank_linear_grouped_fwd(x, U, V, workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 3
    L = pf.lib()
    y = torch.zeros((2, 5, 6), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    # overlapping factor groups (stride smaller than one matrix)
    st = L.pf_lowrank_linear_grouped_fwd(2, x.data_ptr(), 8, 0, U.data_ptr(), 4, 8, V.data_ptr(), 4, 24, y.data_ptr(), 6, 30,
                                         None, 0, 0, 5, 8, 6, 4, pf.PF_BF16, ws.data_ptr(), ws.numel(), None)
    assert st == 1
    st = L.pf_lowrank_linear_grouped_fwd(0, x.data_ptr(), 8, 0, U.data_ptr(), 4, 32, V.data_ptr(), 4, 24, y.data_ptr(), 6, 30,
                                         None, 0, 0, 5, 8, 6, 4, pf.PF_BF16, ws.data_ptr(), ws.numel(), None)
    assert st == 1
    assert pf.pf_launch_count() == before
