"""GPU parity: factor gradients in fp32 and / or accumulated over micro-batches
(pf_lowrank_linear_bwd_ex) vs the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2103_03936_b200 as pf
import pf_workloads as wl
from _gpu import Guarded, assert_close, dev

pytestmark = pytest.mark.gpu


def _inputs(case):
    d = case.generate()
    return d, tuple(dev(d[k_], case.dtype) for k_ in ("x", "U", "V", "dY"))


def run_f32(case, expect_native=None):
    """fp32 gradients of one call: against the oracle, and against the plain call (the same sums
    rounded once more: rounding the fp32 result to the storage type must reproduce it bit for bit)."""
    d, (x, U, V, dY) = _inputs(case)
    dt = case.dtype
    m, k, n, r = case.m, case.k, case.n, case.r
    _, T = pf.pf_lowrank_linear_fwd(x, U, V, want_stash=True)
    l0 = pf.pf_launch_count()
    dX0, dU0, dV0 = pf.pf_lowrank_linear_bwd(x, U, V, dY, T_stash=T)
    l1 = pf.pf_launch_count()
    gU, gV = Guarded((k, r), wl.F32), Guarded((n, r), wl.F32)
    dX1, _, _ = pf.pf_lowrank_linear_bwd(x, U, V, dY, T_stash=T, dU=gU.t, dV=gV.t, grads_f32=True)
    l2 = pf.pf_launch_count()
    torch.cuda.synchronize()
    dX_ref, dU_ref, dV_ref = oracle.linear_bwd(d["x"], d["U"], d["V"], d["dY"])
    tag = f"{case.name} {m}x{k}->{n} r{r} {dt} fp32 grads "
    assert gU.t.dtype == torch.float32 and gV.t.dtype == torch.float32
    assert_close(gU.t, dU_ref, wl.F32, tag + "dU", tol=1e-2 if dt == wl.BF16 else 1e-4)
    assert_close(gV.t, dV_ref, wl.F32, tag + "dV", tol=1e-2 if dt == wl.BF16 else 1e-4)
    assert torch.equal(gU.t.to(dU0.dtype), dU0) and torch.equal(gV.t.to(dV0.dtype), dV0)
    assert torch.equal(dX0, dX1)
    gU.check()
    gV.check()
    # unrounded sums carry more bits than bf16 holds; gradients that went through a bf16 copy do not
    native = bool((gU.t != gU.t.to(torch.bfloat16).float()).any()) and bool((gV.t != gV.t.to(torch.bfloat16).float()).any())
    if expect_native is not None:
        assert native == expect_native
        if native:
            assert l2 - l1 == l1 - l0 + 1          # the plain call's launches plus one for both matrices
    assert pf.pf_last_device_status() == 0
    return native


def run_accumulate(case, f32, parts=3):
    """The batch cut into micro-batches whose gradients are accumulated: the result is the gradient of
    the whole batch (plain sums over rows), on top of what the matrices held before."""
    d, (x, U, V, dY) = _inputs(case)
    dt = case.dtype
    m, k, n, r = case.m, case.k, case.n, case.r
    gdt = wl.F32 if f32 else dt
    prevU = wl.round_to(wl.normal(case.seed, 8, (k, r), 0.5), gdt)
    prevV = wl.round_to(wl.normal(case.seed, 9, (n, r), 0.5), gdt)
    gU, gV = Guarded((k, r), gdt), Guarded((n, r), gdt)
    gU.t.copy_(dev(prevU, gdt))
    gV.t.copy_(dev(prevV, gdt))
    cuts = [m * i // parts for i in range(parts + 1)]
    for lo, hi in zip(cuts[:-1], cuts[1:]):
        pf.pf_lowrank_linear_bwd(x[lo:hi], U, V, dY[lo:hi], need_dX=False, dU=gU.t, dV=gV.t, accumulate=True,
                                 grads_f32=f32)
    torch.cuda.synchronize()
    _, dU_ref, dV_ref = oracle.linear_bwd(d["x"], d["U"], d["V"], d["dY"])
    tag = f"{case.name} {m}x{k}->{n} r{r} {dt} accumulate f32={f32} "
    tol = 1e-2 if dt == wl.BF16 else 1e-4
    assert_close(gU.t, oracle.widen(prevU) + dU_ref, gdt, tag + "dU", tol=tol)
    assert_close(gV.t, oracle.widen(prevV) + dV_ref, gdt, tag + "dV", tol=tol)
    gU.check()
    gV.check()
    assert pf.pf_last_device_status() == 0


@pytest.mark.parametrize("m,k,n,r", [(2100, 200, 328, 40), (4096, 512, 2048, 128), (2304, 136, 1000, 136)])
def test_fp32_grads_fused_shapes_are_unrounded_sums(m, k, n, r):
    """Many rows, r <= 192: fused dX kernel, then dU and dV as split reductions; the fp32 matrices are
    the sums of their fp32 slices, unrounded (one more launch than the plain call)."""
    run_f32(wl.LinearCase("g32", m, k, n, r, wl.BF16, 51), expect_native=True)


@pytest.mark.parametrize("m,k,n,r", [(700, 1504, 520, 376), (300, 136, 72, 24), (1000, 328, 520, 96)])
def test_fp32_grads_few_rows(m, k, n, r):
    run_f32(wl.LinearCase("g32", m, k, n, r, wl.BF16, 52), expect_native=True)


@pytest.mark.parametrize("dtype,m,k,n,r", [(wl.BF16, 300, 100, 136, 33), (wl.BF16, 40, 24, 16, 8), (wl.F32, 200, 72, 136, 24),
                                           (wl.BF16, 2304, 520, 264, 320)])
def test_fp32_grads_through_the_workspace(dtype, m, k, n, r):
    """Odd pitches, one k-block only, fp32 storage, ranks whose reductions do not split: plain
    gradients first, widened in a second pass."""
    run_f32(wl.LinearCase("g32", m, k, n, r, dtype, 53))


@pytest.mark.parametrize("f32", [False, True])
@pytest.mark.parametrize("dtype,m,k,n,r", [(wl.BF16, 2100, 200, 328, 40), (wl.BF16, 900, 200, 264, 96),
                                           (wl.BF16, 300, 100, 136, 33), (wl.F32, 200, 72, 136, 24)])
def test_accumulation_over_micro_batches(dtype, m, k, n, r, f32):
    run_accumulate(wl.LinearCase("acc", m, k, n, r, dtype, 54), f32=f32)


def test_accumulating_fp32_gradients_beats_accumulating_bf16():
    """Sixteen micro-batches: the fp32 accumulator stays an order of magnitude closer to the exact sum
    than the bf16 one (which rounds after every addition)."""
    case = wl.LinearCase("acc16", 16 * 160, 136, 200, 40, wl.BF16, 55)
    d, (x, U, V, dY) = _inputs(case)
    _, dU_ref, _ = oracle.linear_bwd(d["x"], d["U"], d["V"], d["dY"])
    errs = {}
    for f32 in (False, True):
        gdt = torch.float32 if f32 else torch.bfloat16
        dU = torch.zeros((case.k, case.r), dtype=gdt, device="cuda")
        dV = torch.zeros((case.n, case.r), dtype=gdt, device="cuda")
        for i in range(16):
            pf.pf_lowrank_linear_bwd(x[160 * i:160 * (i + 1)], U, V, dY[160 * i:160 * (i + 1)], need_dX=False,
                                     dU=dU, dV=dV, accumulate=True, grads_f32=f32)
        errs[f32] = oracle.rel_err(dU.float().cpu().numpy().astype(np.float64), dU_ref)
    assert errs[True] < 2e-3 and errs[True] < 0.5 * errs[False], errs


def test_bad_flags_and_types():
    case = wl.LinearCase("bad", 64, 32, 48, 8, wl.BF16, 56)
    _, (x, U, V, dY) = _inputs(case)
    with pytest.raises(ValueError):
        pf.pf_lowrank_linear_bwd(x, U, V, dY, accumulate=True)
    with pytest.raises(ValueError):
        pf.pf_lowrank_linear_bwd(x, U, V, dY, dU=torch.zeros((32, 8), dtype=torch.bfloat16, device="cuda"),
                                 dV=torch.zeros((48, 8), dtype=torch.bfloat16, device="cuda"), grads_f32=True)
    import ctypes
    L = pf.lib()
    z = ctypes.c_void_p(x.data_ptr())
    st = L.pf_lowrank_linear_bwd_ex(z, 32, ctypes.c_void_p(U.data_ptr()), 8, ctypes.c_void_p(V.data_ptr()), 8,
                                    ctypes.c_void_p(dY.data_ptr()), 48, None, 0, None, 0, z, 8, z, 8, 64, 32, 48, 8,
                                    pf.PF_BF16, 4, None, 0, None)
    assert st == 1          # PF_ERR_INVALID_ARG: unknown flag bit
