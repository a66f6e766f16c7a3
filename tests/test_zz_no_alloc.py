"""pf_lowrank_linear_fwd_static: the forward for callers that cannot allocate device memory
(latency-critical hosts where cudaMalloc's implicit synchronisation is forbidden, plug-ins that
receive tensors but no allocator, processes whose device memory is fully committed).  Its scratch
is a fixed array inside the library, so this test checks, through the C ABI, that it returns what
pf_lowrank_linear_fwd returns with a caller-provided workspace, bit for bit, and what the fp64
oracle computes -- on two calls in a row, because the array keeps the previous call's contents --
that free device memory is the same before and after a call (nothing is allocated), and that
problems larger than the array are refused on the host.

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test; it also passes on its own in a fresh process.
"""
import pytest
import torch

import oracle
import paper_2103_03936_b200 as pf
import pf_workloads as wl
from _gpu import TOL, assert_close, dev

pytestmark = pytest.mark.gpu


def _both(case, stash=True):
    """Runs the workspace entry and the static entry on one problem; returns both results, the
    oracle's, and the change in free device memory across the static call."""
    d = case.generate()
    x, U, V = (dev(d[k_], case.dtype) for k_ in ("x", "U", "V"))
    tdt = x.dtype
    ref = pf.pf_lowrank_linear_fwd(x, U, V, want_stash=stash)
    y = torch.full((case.m, case.n), -7.0, dtype=tdt, device="cuda")
    T = torch.full((case.m, case.r), -7.0, dtype=tdt, device="cuda") if stash else None
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    pf.pf_lowrank_linear_fwd_static(x, U, V, y=y, T_stash=T)
    torch.cuda.synchronize()
    free1 = torch.cuda.mem_get_info()[0]
    y_or, T_or = oracle.linear_fwd(d["x"], d["U"], d["V"])
    return ((y, T) if stash else (y,)), (ref if stash else (ref,)), ((y_or, T_or) if stash else (y_or,)), free0 - free1


def _first_call_on_this_device():
    """The first call on a device is the set-up call: it looks up the array's device address, and
    with CUDA's lazy module loading that is also the moment the driver materialises the array
    itself (the one time the free-memory figure drops, by the array's size).  Every later call
    must leave free device memory unchanged."""
    x = torch.zeros((8, 16), dtype=torch.bfloat16, device="cuda")
    U = torch.zeros((16, 8), dtype=torch.bfloat16, device="cuda")
    V = torch.zeros((8, 8), dtype=torch.bfloat16, device="cuda")
    pf.pf_lowrank_linear_fwd_static(x, U, V, y=torch.empty((8, 8), dtype=torch.bfloat16, device="cuda"))
    torch.cuda.synchronize()


def _check(case, stash=True):
    _first_call_on_this_device()
    got, ref, orc, used = _both(case, stash)
    for g, r_, o, nm in zip(got, ref, orc, ("y", "T")):
        assert torch.equal(g, r_), f"{case.name} {nm}: the two entry points differ"     # same kernels, same order
        assert_close(g, o, case.dtype, f"{case.name} {nm}", tol=TOL[case.dtype])        # and both match the oracle
    assert used == 0, f"{case.name}: free device memory changed by {used} bytes across the call"


@pytest.mark.parametrize("dtype", [wl.BF16, wl.F32])
def test_static_scratch_forward_matches_workspace_forward_twice_in_a_row(dtype):
    # two different problems back to back: the second call sees the first call's leftovers
    _check(wl.LinearCase("na1", 1000, 328, 520, 96, dtype, 21))
    _check(wl.LinearCase("na2", 300, 100, 130, 33, dtype, 22))      # ragged widths: re-pitched copies
    assert pf.pf_last_device_status() == 0


def test_static_scratch_forward_without_stash_uses_the_array_for_the_intermediate():
    case = wl.LinearCase("na3", 2048, 512, 640, 128, wl.BF16, 23)
    for _ in range(2):
        _check(case, stash=False)


def test_which_benchmark_shapes_fit_the_array():
    """The bound is what the chosen path really uses.  The Transformer-FFN shapes take the fused
    kernel (x U stays on chip, the stash is written directly): they fit.  The LSTM shape fits with
    16-byte row pitches (x U once plus the fp32 slices of the split first product, 7.4 MiB) and is
    refused with the tight pitches of 3000 / 750 bytes, whose re-pitched copies of x, U and V alone
    take 7.7 MiB."""
    _first_call_on_this_device()
    for name in ("C2a", "C2b"):
        c = wl.linear_cases()[name]
        d = c.generate()
        x, U, V = (dev(d[k_], c.dtype) for k_ in ("x", "U", "V"))
        y_ref, T_ref = pf.pf_lowrank_linear_fwd(x, U, V, want_stash=True)
        y, T = torch.empty_like(y_ref), torch.empty_like(T_ref)
        pf.pf_lowrank_linear_fwd_static(x, U, V, y=y, T_stash=T)
        torch.cuda.synchronize()
        assert torch.equal(y, y_ref) and torch.equal(T, T_ref), name
    c = wl.linear_cases()["C3i"]
    d = c.generate()

    def padded(a, cols, ld):
        buf = torch.zeros((a.shape[0], ld), dtype=torch.bfloat16, device="cuda")
        buf[:, :cols] = dev(a, c.dtype)
        return buf[:, :cols]
    x, U, V = padded(d["x"], 1500, 1504), padded(d["U"], 375, 376), padded(d["V"], 375, 376)
    y_ref = pf.pf_lowrank_linear_fwd(x, U, V)
    y = torch.empty_like(y_ref)
    pf.pf_lowrank_linear_fwd_static(x, U, V, y=y)
    torch.cuda.synchronize()
    assert torch.equal(y, y_ref)
    xt, Ut, Vt = (dev(d[k_], c.dtype) for k_ in ("x", "U", "V"))       # tight pitches
    before = pf.pf_launch_count()
    with pytest.raises(pf.PfError) as e:
        pf.pf_lowrank_linear_fwd_static(xt, Ut, Vt, y=y)
    assert e.value.status == 3 and pf.pf_launch_count() == before
    assert pf.pf_last_device_status() == 0


def test_problem_larger_than_the_array_is_refused_before_any_launch():
    assert pf.pf_static_scratch_bytes() == 8 << 20
    m, k, n, r = 2000, 64, 64, 4096           # few rows: unfused products, and x U alone is 16 MB
    assert m * r * 2 > pf.pf_static_scratch_bytes()
    # real buffers of the right sizes: were the call accepted by mistake, it would still stay in bounds
    x = torch.zeros((m, k), dtype=torch.bfloat16, device="cuda")
    U = torch.zeros((k, r), dtype=torch.bfloat16, device="cuda")
    V = torch.zeros((n, r), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((m, n), dtype=torch.bfloat16, device="cuda")
    before = pf.pf_launch_count()
    with pytest.raises(pf.PfError) as e:
        pf.pf_lowrank_linear_fwd_static(x, U, V, y=y)
    assert e.value.status == 3 and pf.pf_launch_count() == before
