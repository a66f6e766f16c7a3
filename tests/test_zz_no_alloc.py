"""pf_lowrank_linear_fwd_static: the forward for callers that cannot allocate device memory
(latency-critical hosts where cudaMalloc's implicit synchronisation is forbidden, plug-ins that
receive tensors but no allocator, processes whose device memory is fully committed).  Its scratch
is a fixed array inside the library, so this test checks, through the C ABI, that it returns what
pf_lowrank_linear_fwd returns with a caller-provided workspace -- on two calls in a row, because
the array keeps the previous call's contents -- and that problems larger than the array are
refused on the host.

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test; it also passes on its own in a fresh process.
"""
import pytest
import torch

import paper_2103_03936_b200 as pf
import pf_workloads as wl
from _gpu import TOL, assert_close, dev

pytestmark = pytest.mark.gpu


def _both(case):
    d = case.generate()
    x, U, V = (dev(d[k_], case.dtype) for k_ in ("x", "U", "V"))
    tdt = x.dtype
    y_ref, T_ref = pf.pf_lowrank_linear_fwd(x, U, V, want_stash=True)
    y = torch.full((case.m, case.n), -7.0, dtype=tdt, device="cuda")
    T = torch.full((case.m, case.r), -7.0, dtype=tdt, device="cuda")
    pf.pf_lowrank_linear_fwd_static(x, U, V, y=y, T_stash=T)
    torch.cuda.synchronize()
    return (y, T), (y_ref, T_ref)


@pytest.mark.parametrize("dtype", [wl.BF16, wl.F32])
def test_static_scratch_forward_matches_workspace_forward_twice_in_a_row(dtype):
    # two different problems back to back: the second call sees the first call's leftovers
    cases = [wl.LinearCase("na1", 1000, 328, 520, 96, dtype, 21),
             wl.LinearCase("na2", 300, 100, 130, 33, dtype, 22)]     # ragged widths: re-pitched copies
    for case in cases:
        (y, T), (y_ref, T_ref) = _both(case)
        assert_close(y, y_ref.double().cpu().numpy(), dtype, "y", tol=TOL[dtype])
        assert_close(T, T_ref.double().cpu().numpy(), dtype, "T", tol=TOL[dtype])
    assert pf.pf_last_device_status() == 0


def test_static_scratch_forward_without_stash_uses_the_array_for_the_intermediate():
    case = wl.LinearCase("na3", 2048, 512, 640, 128, wl.BF16, 23)
    d = case.generate()
    x, U, V = (dev(d[k_], case.dtype) for k_ in ("x", "U", "V"))
    y_ref = pf.pf_lowrank_linear_fwd(x, U, V)
    for _ in range(2):
        y = torch.full((case.m, case.n), -7.0, dtype=x.dtype, device="cuda")
        pf.pf_lowrank_linear_fwd_static(x, U, V, y=y)
        torch.cuda.synchronize()
        assert_close(y, y_ref.double().cpu().numpy(), case.dtype, "y")


def test_problem_larger_than_the_array_is_refused_before_any_launch():
    assert pf.pf_static_scratch_bytes() == 8 << 20
    m, k, n, r = 1 << 20, 64, 64, 64          # needs far more than the array for x U alone
    assert pf.pf_lowrank_linear_workspace(m, k, n, r, pf.PF_BF16, 0) > pf.pf_static_scratch_bytes()
    x = torch.empty((8, k), dtype=torch.bfloat16, device="cuda")       # never dereferenced
    U = torch.empty((k, r), dtype=torch.bfloat16, device="cuda")
    V = torch.empty((n, r), dtype=torch.bfloat16, device="cuda")
    before = pf.pf_launch_count()
    st = pf.lib().pf_lowrank_linear_fwd_static(x.data_ptr(), k, U.data_ptr(), r, V.data_ptr(), r,
                                               x.data_ptr(), n, None, 0, m, k, n, r, pf.PF_BF16, None)
    assert st == 3 and pf.pf_launch_count() == before
