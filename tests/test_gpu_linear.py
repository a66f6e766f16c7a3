"""GPU parity: factorized linear forward/backward through the C ABI vs the fp64 oracle."""
import itertools

import numpy as np
import pytest
import torch

import oracle
import paper_2103_03936_b200 as pf
import pf_workloads as wl
from _gpu import ESCAPES, Guarded, assert_blocks_close, assert_close, dev, host

pytestmark = pytest.mark.gpu


def run_case(case, ld_pad=0, stash=True, need_dX=True, tiny=False, blocks=False):
    d = case.generate()
    dt = case.dtype
    m, k, n, r = case.m, case.k, case.n, case.r

    def up(a, cols):
        if not ld_pad:
            return dev(a, dt)
        buf = torch.zeros((a.shape[0], cols + ld_pad), dtype=wl.to_torch(a[:1], dt).dtype, device="cuda")
        buf[:, :cols] = dev(a, dt)
        return buf[:, :cols]

    x, U, V, dY = up(d["x"], k), up(d["U"], r), up(d["V"], r), up(d["dY"], n)
    gy = Guarded((m, n), dt, ld=n + ld_pad if ld_pad else None)
    gT = Guarded((m, r), dt, ld=r + ld_pad if ld_pad else None)
    out = pf.pf_lowrank_linear_fwd(x, U, V, y=gy.t, T_stash=gT.t if stash else None)
    y_ref, T_ref = oracle.linear_fwd(d["x"], d["U"], d["V"])
    dX_ref, dU_ref, dV_ref = oracle.linear_bwd(d["x"], d["U"], d["V"], d["dY"])
    gdX = Guarded((m, k), dt, ld=k + ld_pad if ld_pad else None)
    gdU = Guarded((k, r), dt, ld=r + ld_pad if ld_pad else None)
    gdV = Guarded((n, r), dt, ld=r + ld_pad if ld_pad else None)
    pf.pf_lowrank_linear_bwd(x, U, V, dY, T_stash=gT.t if stash else None, need_dX=need_dX,
                             dX=gdX.t if need_dX else None, dU=gdU.t, dV=gdV.t)
    torch.cuda.synchronize()
    ab = {}
    if tiny:   # magnitude of the summands, for outputs of a handful of elements
        aw = {k_: np.abs(oracle.widen(v)) for k_, v in d.items()}
        ab["y"], ab["T"] = oracle.linear_fwd(aw["x"], aw["U"], aw["V"])
        ab["dX"], ab["dU"], ab["dV"] = oracle.linear_bwd(aw["x"], aw["U"], aw["V"], aw["dY"])
    tag = f"{case.name} {m}x{k}->{n} r{r} {dt} "
    checks = [("y", gy, y_ref)]
    if stash:
        checks.append(("T", gT, T_ref))
    if need_dX:
        checks.append(("dX", gdX, dX_ref))
    checks += [("dU", gdU, dU_ref), ("dV", gdV, dV_ref)]
    errs = {}
    for nm, g, ref in checks:
        errs[nm] = assert_close(g.t, ref, dt, tag + nm, abs_ref64=ab.get(nm))
        if blocks:   # and no 128 x 128 block of the tensor may miss the same bound
            errs[nm + " worst block"] = assert_blocks_close(g.t, ref, dt, tag + nm)
    for g in (gy, gT, gdX, gdU, gdV):
        g.check()
    assert pf.pf_last_device_status() == 0
    return errs


GRID = [(m, k, n, r) for m, k, n, r in itertools.product((1, 7, 130), (1, 17, 100), (3, 24, 130), (1, 5, 33))]


# Outputs of the bf16 grid that may be measured against the magnitude of their summands (see
# _gpu.assert_close): single near-cancelled sums.  The count is fixed by the seeded inputs.
MAX_CANCELLED_OUTPUTS = 2


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_tiny_exhaustive_grid(dtype):
    first = len(ESCAPES)
    for idx, (m, k, n, r) in enumerate(GRID):
        run_case(wl.LinearCase(f"g{idx}", m, k, n, r, dtype, 100 + idx), tiny=True)
    took = ESCAPES[first:]
    for what, rel, ratio, err_abs in took:
        print(f"cancelled output {what}: rel {rel:.2e}, |exact|/|summands| {ratio:.2e}, err vs summands {err_abs:.2e}")
    assert len(took) <= (MAX_CANCELLED_OUTPUTS if dtype == wl.BF16 else 0), took


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
@pytest.mark.parametrize("m,k,n,r", [(257, 72, 136, 24), (300, 200, 264, 40), (129, 64, 64, 64),
                                     (1000, 328, 520, 96)])
def test_multi_tile_ragged(dtype, m, k, n, r):
    run_case(wl.LinearCase("rag", m, k, n, r, dtype, 7))


@pytest.mark.parametrize("m,k,n,r", [(2100, 200, 328, 40), (2048, 1504, 520, 376), (2500, 136, 72, 200),
                                     (4100, 72, 1000, 130), (2048, 64, 64, 256), (2304, 520, 264, 320),
                                     (2050, 100, 130, 33)])
def test_fused_chain_envelope(m, k, n, r):
    """m >= 2048 with r <= 192 takes the fused two-GEMM kernel (rank paddings 64, 128, 192; ragged
    row tile, ragged k / n tails, with and without stash and dX); the larger ranks of this list run
    as unfused products on the same batch sizes."""
    run_case(wl.LinearCase("chain", m, k, n, r, wl.BF16, 13))
    run_case(wl.LinearCase("chain", m, k, n, r, wl.BF16, 14), stash=False, need_dX=False)


@pytest.mark.parametrize("m,k,n,r", [(19500, 200, 128, 64), (40000, 136, 72, 100)])
def test_fused_chain_more_row_tiles_than_sms(m, k, n, r):
    """More 128-row tiles than SMs: the fused kernel runs as a persistent grid in which a CTA owns
    several tiles (unequal counts, a ragged last tile) and the phases of consecutive tiles overlap;
    forward (one and two output column tiles per row tile) and dX, with and without the stash."""
    run_case(wl.LinearCase("multi", m, k, n, r, wl.BF16, 19))
    run_case(wl.LinearCase("multi", m, k, n, r, wl.BF16, 20), stash=False, need_dX=False)


@pytest.mark.parametrize("m,k,n,r", [(16000, 72, 264, 520), (9000, 200, 520, 392)])
def test_wide_unfused_products_on_cta_pairs(m, k, n, r):
    """Ranks above 384 run as plain products; wide ones with many tiles use the two-CTA MMA kernel:
    a ragged last row pair, ragged column tiles and a ragged k tail, K-major and MN-major B."""
    run_case(wl.LinearCase("pairs", m, k, n, r, wl.BF16, 17))


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_leading_dimensions_and_padding_untouched(dtype):
    run_case(wl.LinearCase("ld", 200, 72, 136, 24, dtype, 8), ld_pad=8)
    run_case(wl.LinearCase("ld", 77, 33, 50, 7, dtype, 9), ld_pad=3)


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_recompute_without_stash_and_no_dX(dtype):
    run_case(wl.LinearCase("ns", 300, 136, 72, 24, dtype, 10), stash=False)
    run_case(wl.LinearCase("nx", 300, 136, 72, 24, dtype, 11), need_dX=False)


def test_config_C1_tiny_fp32():
    run_case(wl.linear_cases()["C1"])


@pytest.mark.parametrize("name", ["C2a", "C2b", "C3i", "C3h"])
def test_configs_full_size(name):
    errs = run_case(wl.linear_cases()[name], blocks=True)
    print(name, errs)


def test_config_C3_padded_pitch():
    """LSTM shape with 16-byte-multiple row pitches (k 1500->1504, r 375->376 elements)."""
    run_case(wl.linear_cases()["C3i"], ld_pad=0)
    c = wl.linear_cases()["C3i"]
    d = c.generate()

    def padded(a, cols, ld):
        buf = torch.zeros((a.shape[0], ld), dtype=torch.bfloat16, device="cuda")
        buf[:, :cols] = dev(a, c.dtype)
        return buf[:, :cols]
    x, U, V, dY = padded(d["x"], 1500, 1504), padded(d["U"], 375, 376), padded(d["V"], 375, 376), dev(d["dY"], c.dtype)
    y, T = pf.pf_lowrank_linear_fwd(x, U, V, want_stash=True)
    dX, dU, dV = pf.pf_lowrank_linear_bwd(x, U, V, dY, T_stash=T)
    y_ref, _ = oracle.linear_fwd(d["x"], d["U"], d["V"])
    dX_ref, dU_ref, dV_ref = oracle.linear_bwd(d["x"], d["U"], d["V"], d["dY"])
    for got, want, nm in ((y, y_ref, "y"), (dX, dX_ref, "dX"), (dU, dU_ref, "dU"), (dV, dV_ref, "dV")):
        assert_close(got, want, c.dtype, nm)


@pytest.fixture(scope="module")
def sweep_inputs():
    c = wl.linear_cases()["C5r16"]
    x = wl.round_to(wl.normal(c.seed, 0, (c.m, c.k)), c.dtype)
    dY = wl.round_to(wl.normal(c.seed, 3, (c.m, c.n)), c.dtype)
    return x, dY, dev(x, c.dtype), dev(dY, c.dtype)


@pytest.mark.parametrize("r", [16, 128, 256, 1024])
def test_rank_sweep_full_size_sampled(sweep_inputs, r):
    """m=16384, k=n=4096: y and dX on sampled rows, dU and dV on sampled rank columns (the
    oracle computes those exactly from sliced inputs), in the configuration the bench times."""
    x_h, dY_h, x, dY = sweep_inputs
    c = wl.linear_cases()[f"C5r{r}"]
    import math
    sig = 1.0 / math.sqrt(c.k)
    U_h = wl.round_to(wl.normal(c.factor_seed, 1, (c.k, r), sig), c.dtype)
    V_h = wl.round_to(wl.normal(c.factor_seed, 2, (c.n, r), sig), c.dtype)
    U, V = dev(U_h, c.dtype), dev(V_h, c.dtype)
    y, T = pf.pf_lowrank_linear_fwd(x, U, V, want_stash=True)
    dX, dU, dV = pf.pf_lowrank_linear_bwd(x, U, V, dY, T_stash=T)
    torch.cuda.synchronize()
    rows = [0, 1, 127, 128, 5000, 8191, 8192, 16383]
    y_ref, T_ref = oracle.linear_fwd(x_h[rows], U_h, V_h)
    dX_ref, _, _ = oracle.linear_bwd(x_h[rows], U_h, V_h, dY_h[rows])
    for got, want, nm in ((y[rows], y_ref, "y rows"), (T[rows], T_ref, "T rows"), (dX[rows], dX_ref, "dX rows")):
        assert_close(got, want, c.dtype, nm)
        assert_blocks_close(got, want, c.dtype, nm)          # 8 sampled rows x 128 columns per block
    J = sorted({0, r // 2, r - 1})
    _, dU_ref, dV_ref = oracle.linear_bwd(x_h, U_h[:, J], V_h[:, J], dY_h)
    for got, want, nm in ((dU[:, J], dU_ref, "dU cols"), (dV[:, J], dV_ref, "dV cols")):
        assert_close(got, want, c.dtype, nm)
        assert_blocks_close(got, want, c.dtype, nm)          # 128 rows x the sampled columns per block
    assert pf.pf_last_device_status() == 0


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_backward_is_bit_reproducible(dtype):
    c = wl.LinearCase("rep", 4096, 256, 320, 64, dtype, 12)
    d = c.generate()
    x, U, V, dY = (dev(d[k_], dtype) for k_ in ("x", "U", "V", "dY"))
    a = pf.pf_lowrank_linear_bwd(x, U, V, dY)
    b = pf.pf_lowrank_linear_bwd(x, U, V, dY)
    torch.cuda.synchronize()
    for p, q in zip(a, b):
        assert torch.equal(p, q)


def test_split_reductions_on_two_streams_do_not_interfere():
    """The slice sums of dU / dV meet at per-tile counters inside the library; launches that are in
    flight at the same time on different streams must use different counter sets."""
    cases = [wl.LinearCase("s0", 4096, 256, 320, 64, wl.BF16, 21), wl.LinearCase("s1", 3000, 384, 256, 128, wl.BF16, 22)]
    ins = []
    for c in cases:
        d = c.generate()
        ins.append(tuple(dev(d[k_], wl.BF16) for k_ in ("x", "U", "V", "dY")))
    ref = [pf.pf_lowrank_linear_bwd(*t) for t in ins]
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    outs = [[], []]
    for it in range(6):
        for i, st in enumerate(streams):
            with torch.cuda.stream(st):
                outs[i].append(pf.pf_lowrank_linear_bwd(*ins[i], stream=st))
    torch.cuda.synchronize()
    for i in range(2):
        for got in outs[i]:
            for p, q in zip(got, ref[i]):
                assert torch.equal(p, q)
    assert pf.pf_last_device_status() == 0


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_empty_batch(dtype):
    tdt = torch.float32 if dtype == wl.F32 else torch.bfloat16
    x = torch.empty((0, 16), dtype=tdt, device="cuda")
    U = torch.ones((16, 4), dtype=tdt, device="cuda")
    V = torch.ones((8, 4), dtype=tdt, device="cuda")
    y = pf.pf_lowrank_linear_fwd(x, U, V)
    assert y.shape == (0, 8)
    dX, dU, dV = pf.pf_lowrank_linear_bwd(x, U, V, torch.empty((0, 8), dtype=tdt, device="cuda"),
                                          dU=torch.full((16, 4), 3.0, dtype=tdt, device="cuda"),
                                          dV=torch.full((8, 4), 3.0, dtype=tdt, device="cuda"))
    torch.cuda.synchronize()
    assert torch.all(dU == 0) and torch.all(dV == 0)


def test_invalid_arguments_raise_not_launch():
    x = torch.zeros((4, 8), dtype=torch.bfloat16, device="cuda")
    U = torch.zeros((8, 2), dtype=torch.bfloat16, device="cuda")
    V = torch.zeros((6, 2), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(pf.PfError) as e:
        pf.pf_lowrank_linear_fwd(x, U, V, workspace=torch.empty(8, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 3
