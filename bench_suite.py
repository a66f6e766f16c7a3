"""Per-configuration timings of the factorized layers (forward, backward, fraction of roofline).

Used by ``bench.py --suite FILE``: every benchmark configuration (tiny fp32, Transformer FFN,
LSTM gates in the tight and in a 16-byte-pitch layout, ResNet-style convolutions with the gradient
pack, and the rank sweep) is timed with CUDA events on rotating buffer sets larger than L2, and
written as one JSON object per line (fwd_us and bwd_us are each call timed alone, fwd_bwd_us is
the pair launched back to back).  Only timing lives here; parity is the tests' job.
"""
from __future__ import annotations

import json
import math

import torch

import pf_workloads as wl
import paper_2103_03936_b200 as pf

L2_BYTES = 126 << 20


def _rand(shape, dtype, scale=1.0, relu=False, ld=None):
    rows = int(math.prod(shape[:-1]))
    cols = shape[-1]
    if ld is None:
        t = torch.randn(shape, device="cuda", dtype=torch.float32) * scale
        if relu:
            t = t.clamp_(min=0)
        return t.to(dtype)
    buf = torch.zeros((rows, ld), device="cuda", dtype=dtype)
    buf[:, :cols] = (torch.randn((rows, cols), device="cuda", dtype=torch.float32) * scale).to(dtype)
    return buf[:, :cols]


def _time(calls_per_set, iters, warmup=3, repeats=5):
    """calls_per_set: list (one per buffer set) of (fwd_call, bwd_call[, extra_call]).

    Every call, and the fwd+bwd pair, is timed on its own as `iters` back-to-back launches that
    rotate through the buffer sets, between two CUDA events (no event between launches, so that
    consecutive kernels overlap the way they do in a training step); median and minimum over
    `repeats` such batches.  The last entry of the result is the fwd+bwd pair."""
    ns = len(calls_per_set)
    ncalls = len(calls_per_set[0])
    for i in range(warmup):
        for c in calls_per_set[i % ns]:
            c()
    torch.cuda.synchronize()
    groups = [(j,) for j in range(ncalls)] + ([(0, 1)] if ncalls >= 2 else [])
    out = []
    for grp in groups:
        ts = []
        for _ in range(repeats):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(iters):
                cs = calls_per_set[i % ns]
                for j in grp:
                    cs[j]()
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) * 1e3 / iters)
        ts.sort()
        out.append({"median_us": ts[len(ts) // 2], "min_us": ts[0]})
    return out


def _library_linear(sets, U, V, iters):
    """The paper's structure on the same GPU, for context: two library matmuls forward and four
    backward through PyTorch (cuBLAS), intermediates in HBM.  Returns (fwd, bwd, fwd+bwd) in us."""
    calls = []
    for (x, dY) in sets:
        m, r, n, k = x.shape[0], U.shape[1], V.shape[0], U.shape[0]
        T = torch.empty((m, r), dtype=x.dtype, device="cuda")
        y = torch.empty((m, n), dtype=x.dtype, device="cuda")
        G = torch.empty((m, r), dtype=x.dtype, device="cuda")
        dX = torch.empty((m, k), dtype=x.dtype, device="cuda")
        dU, dV = torch.empty_like(U), torch.empty_like(V)

        def fwd(x=x, T=T, y=y):
            torch.matmul(x, U, out=T)
            torch.matmul(T, V.t(), out=y)

        def bwd(x=x, dY=dY, T=T, G=G, dX=dX, dU=dU, dV=dV):
            torch.matmul(dY, V, out=G)
            torch.matmul(G, U.t(), out=dX)
            torch.matmul(x.t(), G, out=dU)
            torch.matmul(dY.t(), T, out=dV)

        calls.append((fwd, bwd))
    t = _time(calls, iters)
    return t[0]["median_us"], t[1]["median_us"], t[-1]["median_us"]


def _floors(flops_fwd, bytes_fwd, bytes_bwd, pk):
    f = max(flops_fwd / (pk["bf16_tflops"] * 1e12), bytes_fwd / (pk["hbm_gbs"] * 1e9)) * 1e6
    b = max(2 * flops_fwd / (pk["bf16_tflops"] * 1e12), bytes_bwd / (pk["hbm_gbs"] * 1e9)) * 1e6
    return f, b


def linear_config(name, m, k, n, r, dtype, pk, pad_pitch=False, iters=32, library=True, repeats=5):
    tdt = torch.bfloat16 if dtype == wl.BF16 else torch.float32
    s = 2 if dtype == wl.BF16 else 4
    code = pf.PF_BF16 if dtype == wl.BF16 else pf.PF_F32
    foot = s * (2 * m * k + 2 * m * n + m * r)
    nsets = max(1, min(16, math.ceil(4 * L2_BYTES / foot)))
    ldk = (k + 7) // 8 * 8 if pad_pitch else None
    ldr = (r + 7) // 8 * 8 if pad_pitch else None
    sig = 1.0 / math.sqrt(k)
    U, V = _rand((k, r), tdt, sig, ld=ldr), _rand((n, r), tdt, sig, ld=ldr)
    stream = torch.cuda.current_stream()
    sets = []
    lib_sets = []
    for _ in range(nsets):
        x, dY = _rand((m, k), tdt, ld=ldk), _rand((m, n), tdt)
        lib_sets.append((x, dY))
        y = torch.empty((m, n), dtype=tdt, device="cuda")
        T = _rand((m, r), tdt, ld=ldr)
        dX = _rand((m, k), tdt, ld=ldk)
        dU, dV = _rand((k, r), tdt, ld=ldr), _rand((n, r), tdt, ld=ldr)
        wf = torch.empty(max(256, pf.pf_lowrank_linear_workspace(m, k, n, r, code, 0)), dtype=torch.uint8, device="cuda")
        wb = torch.empty(max(256, pf.pf_lowrank_linear_workspace(m, k, n, r, code, 1)), dtype=torch.uint8, device="cuda")
        f, _ = pf.pf_lowrank_linear_fwd(x, U, V, y=y, T_stash=T, workspace=wf, stream=stream, prepare=True)
        b, _ = pf.pf_lowrank_linear_bwd(x, U, V, dY, T_stash=T, dX=dX, dU=dU, dV=dV, workspace=wb, stream=stream,
                                        prepare=True)
        sets.append((f, b))
    l0 = pf.pf_launch_count()
    for c in sets[0]:
        c()
    launches = pf.pf_launch_count() - l0
    t = _time(sets, iters, repeats=repeats)
    flops_fwd = 2.0 * m * r * (k + n)
    bytes_fwd = s * (m * k + m * n + r * (k + n))
    bytes_bwd = s * (m * n + 2 * m * k + 2 * r * (k + n))
    ff, fb = _floors(flops_fwd, bytes_fwd, bytes_bwd, pk)
    tot = t[-1]["median_us"]
    lib = _library_linear(lib_sets, U, V, iters) if library else (None, None, None)
    return {"config": name, "kind": "linear", "m": m, "k": k, "n": n, "r": r, "dtype": dtype,
            "library_fwd_us": lib[0], "library_bwd_us": lib[1], "library_fwd_bwd_us": lib[2],
            "pitch": "padded to 16 B" if pad_pitch else "tight", "buffer_sets": nsets, "launches_fwd_bwd": launches,
            "fwd_us": t[0]["median_us"], "bwd_us": t[1]["median_us"], "fwd_bwd_us": tot,
            "floor_fwd_us": ff, "floor_bwd_us": fb, "roofline_frac": (ff + fb) / tot,
            "tflops": 3 * flops_fwd / tot / 1e6, "gbs": (bytes_fwd + bytes_bwd) / tot / 1e3}


def act_config(name, m, k, n, r, pk, iters=32, repeats=5):
    """Forward with bias and max(0, .): the fused epilogue beside the plain forward and beside the plain
    forward followed by the bias add and the activation as elementwise passes over y (torch, in place)."""
    tdt = torch.bfloat16
    foot = 2 * (m * k + m * n + m * r)
    nsets = max(1, min(8, math.ceil(4 * L2_BYTES / foot)))
    U, V = _rand((k, r), tdt, k ** -0.5), _rand((n, r), tdt, k ** -0.5)
    b = _rand((n,), tdt, 0.5)
    stream = torch.cuda.current_stream()
    sets = []
    for _ in range(nsets):
        x = _rand((m, k), tdt)
        y = torch.empty((m, n), dtype=tdt, device="cuda")
        T = torch.empty((m, r), dtype=tdt, device="cuda")
        f0, _ = pf.pf_lowrank_linear_fwd(x, U, V, y=y, T_stash=T, stream=stream, prepare=True)
        f1, _ = pf.pf_lowrank_linear_fwd_act(x, U, V, bias=b, act=pf.PF_ACT_RELU, y=y, T_stash=T, stream=stream,
                                             prepare=True)

        def f2(f0=f0, y=y):
            f0()
            y.add_(b).relu_()
        sets.append((f0, f1, f2))
    t = _time(sets, iters, repeats=repeats)[:3]
    bytes_fwd = 2 * (m * k + m * n + m * r + r * (k + n) + n)
    return {"config": name, "kind": "act", "m": m, "k": k, "n": n, "r": r, "dtype": "bf16", "buffer_sets": nsets,
            "plain_fwd_us": t[0]["median_us"], "fused_bias_relu_fwd_us": t[1]["median_us"],
            "plain_fwd_plus_elementwise_us": t[2]["median_us"], "floor_fwd_us": bytes_fwd / pk["hbm_gbs"] / 1e3,
            "roofline_frac": bytes_fwd / pk["hbm_gbs"] / 1e3 / t[1]["median_us"]}


def grouped_config(name, G, m, k, n, r, pk, shared_x, iters=24, repeats=5):
    """G factorized layers of one shape in one call (row pitches padded to 16 bytes), beside the
    same G layers issued one by one through the ungrouped calls."""
    tdt = torch.bfloat16
    up = lambda v: (v + 7) // 8 * 8
    foot = 2 * G * (2 * m * up(k) + 2 * m * up(n) + m * up(r))
    nsets = max(1, min(8, math.ceil(4 * L2_BYTES / foot)))
    sig = 1.0 / math.sqrt(k)

    def t3(g, rows, cols, scale=1.0):
        buf = torch.zeros((g, rows, up(cols)), device="cuda", dtype=tdt)
        buf[..., :cols] = (torch.randn((g, rows, cols), device="cuda") * scale).to(tdt)
        return buf[..., :cols]

    U, V = t3(G, k, r, sig), t3(G, n, r, sig)
    stream = torch.cuda.current_stream()
    sets, singles = [], []
    for _ in range(nsets):
        x = t3(1, m, k)[0] if shared_x else t3(G, m, k)
        dY = t3(G, m, n)
        y, T = t3(G, m, n), t3(G, m, r)
        dX = t3(1, m, k)[0] if shared_x else t3(G, m, k)
        dU, dV = t3(G, k, r), t3(G, n, r)
        code = pf.PF_BF16
        wf = torch.empty(max(256, pf.pf_lowrank_linear_grouped_workspace(G, m, k, n, r, code, 0)), dtype=torch.uint8, device="cuda")
        wb = torch.empty(max(256, pf.pf_lowrank_linear_grouped_workspace(G, m, k, n, r, code, 1)), dtype=torch.uint8, device="cuda")
        f, _ = pf.pf_lowrank_linear_grouped_fwd(x, U, V, y=y, T_stash=T, workspace=wf, stream=stream, prepare=True)
        b, _ = pf.pf_lowrank_linear_grouped_bwd(x, U, V, dY, T_stash=T, dX=dX, dU=dU, dV=dV, workspace=wb, stream=stream,
                                                prepare=True)
        sets.append((f, b))
        # the same layers one call per group (dX of a shared input would still have to be summed)
        w1f = torch.empty(max(256, pf.pf_lowrank_linear_workspace(m, k, n, r, code, 0)), dtype=torch.uint8, device="cuda")
        w1b = torch.empty(max(256, pf.pf_lowrank_linear_workspace(m, k, n, r, code, 1)), dtype=torch.uint8, device="cuda")
        dXg = t3(G, m, k)
        fs = [pf.pf_lowrank_linear_fwd(x if shared_x else x[g], U[g], V[g], y=y[g], T_stash=T[g], workspace=w1f,
                                       stream=stream, prepare=True)[0] for g in range(G)]
        bs = [pf.pf_lowrank_linear_bwd(x if shared_x else x[g], U[g], V[g], dY[g], T_stash=T[g], dX=dXg[g], dU=dU[g],
                                       dV=dV[g], workspace=w1b, stream=stream, prepare=True)[0] for g in range(G)]
        singles.append(((lambda fs=fs: [c() for c in fs]), (lambda bs=bs: [c() for c in bs])))
    l0 = pf.pf_launch_count()
    for c in sets[0]:
        c()
    launches = pf.pf_launch_count() - l0
    t = _time(sets, iters, repeats=repeats)
    t1 = _time(singles, max(2, iters // 4), repeats=repeats)
    flops_fwd = 2.0 * G * m * r * (k + n)
    xg = 1 if shared_x else G
    bytes_fwd = 2 * (xg * m * k + G * m * n + G * r * (k + n))
    bytes_bwd = 2 * (G * m * n + 2 * xg * m * k + 2 * G * r * (k + n))
    ff, fb = _floors(flops_fwd, bytes_fwd, bytes_bwd, pk)
    tot = t[-1]["median_us"]
    return {"config": name, "kind": "grouped linear", "groups": G, "m": m, "k": k, "n": n, "r": r, "dtype": "bf16",
            "shared_x": shared_x, "pitch": "padded to 16 B", "buffer_sets": nsets, "launches_fwd_bwd": launches,
            "fwd_us": t[0]["median_us"], "bwd_us": t[1]["median_us"], "fwd_bwd_us": tot,
            "one_call_per_group_fwd_bwd_us": t1[-1]["median_us"],
            "floor_fwd_us": ff, "floor_bwd_us": fb, "roofline_frac": (ff + fb) / tot,
            "tflops": 3 * flops_fwd / tot / 1e6, "gbs": (bytes_fwd + bytes_bwd) / tot / 1e3}


def conv_config(name, c, pk, iters=20, repeats=5):
    tdt = torch.bfloat16
    M = c.N * c.H * c.W
    foot = 2 * (2 * M * c.C + 2 * M * c.O + M * c.R)
    nsets = max(1, min(8, math.ceil(4 * L2_BYTES / foot)))
    U = _rand((c.kh, c.kw, c.C, c.R), tdt, math.sqrt(2.0 / (c.kh * c.kw * c.C)))
    V = _rand((c.O, c.R), tdt, math.sqrt(2.0 / c.R))
    stream = torch.cuda.current_stream()
    sets = []
    for _ in range(nsets):
        x = _rand((c.N, c.H, c.W, c.C), tdt, relu=True)
        dY = _rand((c.N, c.H, c.W, c.O), tdt)
        y = torch.empty_like(dY)
        T = torch.empty((c.N, c.H, c.W, c.R), dtype=tdt, device="cuda")
        dX, dU, dV = torch.empty_like(x), torch.empty_like(U), torch.empty_like(V)
        args = (c.N, c.H, c.W, c.C, c.R, c.O, c.kh, c.kw, c.stride, c.pad, pf.PF_BF16)
        wf = torch.empty(max(256, pf.pf_lowrank_conv_workspace(*args, 0)), dtype=torch.uint8, device="cuda")
        wb = torch.empty(max(256, pf.pf_lowrank_conv_workspace(*args, 1)), dtype=torch.uint8, device="cuda")
        f, _ = pf.pf_lowrank_conv_fwd(x, U, V, stride=c.stride, pad=c.pad, y=y, T_stash=T, workspace=wf,
                                      stream=stream, prepare=True)
        b, _ = pf.pf_lowrank_conv_bwd(x, U, V, dY, stride=c.stride, pad=c.pad, T_stash=T, dX=dX, dU=dU, dV=dV,
                                      workspace=wb, stream=stream, prepare=True)
        flat = torch.empty(dU.numel() + dV.numel(), dtype=tdt, device="cuda")
        pk_call, _ = pf.pf_pack_factor_grads([dU, dV], flat=flat, stream=stream, prepare=True)
        sets.append((f, b, pk_call))
    l0 = pf.pf_launch_count()
    for cc in sets[0]:
        cc()
    launches = pf.pf_launch_count() - l0
    t = _time(sets, iters, repeats=repeats)
    Keff = c.kh * c.kw * c.C
    flops_fwd = 2.0 * M * c.R * (Keff + c.O)
    bytes_fwd = 2 * (M * c.C + M * c.O + c.R * (Keff + c.O))
    bytes_bwd = 2 * (M * c.O + 2 * M * c.C + 2 * c.R * (Keff + c.O))
    ff, fb = _floors(flops_fwd, bytes_fwd, bytes_bwd, pk)
    tot = t[-1]["median_us"]
    return {"config": name, "kind": "conv", "N": c.N, "H": c.H, "W": c.W, "C": c.C, "R": c.R, "O": c.O,
            "dtype": "bf16", "buffer_sets": nsets, "launches_fwd_bwd_pack": launches,
            "fwd_us": t[0]["median_us"], "bwd_us": t[1]["median_us"], "pack_us": t[2]["median_us"],
            "fwd_bwd_us": tot, "floor_fwd_us": ff, "floor_bwd_us": fb, "roofline_frac": (ff + fb) / tot,
            "tflops": 3 * flops_fwd / tot / 1e6, "gbs": (bytes_fwd + bytes_bwd) / tot / 1e3}


def pack_config(name, numels, pk, iters=30, repeats=5):
    tdt = torch.bfloat16
    grads = [torch.randn(n, device="cuda").to(tdt) for n in numels]
    total = sum(numels)
    nsets = max(1, min(8, math.ceil(2 * L2_BYTES / (4 * total))))
    stream = torch.cuda.current_stream()
    sets = []
    for _ in range(nsets):
        g = [t.clone() for t in grads]
        flat = torch.empty(total, dtype=tdt, device="cuda")
        call, _ = pf.pf_pack_factor_grads(g, flat=flat, stream=stream, prepare=True)
        sets.append((call,))
    t = _time(sets, iters, repeats=repeats)
    us = t[0]["median_us"]
    return {"config": name, "kind": "pack", "tensors": len(numels), "elements": total, "dtype": "bf16",
            "us": us, "gbs": 4.0 * total / us / 1e3, "roofline_frac": (4.0 * total / (pk["hbm_gbs"] * 1e9) * 1e6) / us}


def quick(pk):
    """The configurations the roofline target names, timed with the same back-to-back protocol but few
    repetitions (a few seconds in all), for the benchmark's JSON line: per configuration the forward,
    the backward and the pair in microseconds, the roofline floor and the fraction reached."""
    out = {}

    def keep(r):
        key = r["config"] + (" (16 B pitches)" if r.get("pitch") == "padded to 16 B" else "")
        out[key] = {
            "fwd_us": round(r["fwd_us"], 2), "bwd_us": round(r["bwd_us"], 2), "fwd_bwd_us": round(r["fwd_bwd_us"], 2),
            "floor_us": round(r["floor_fwd_us"] + r["floor_bwd_us"], 2), "roofline_frac": round(r["roofline_frac"], 4),
            "launches": r.get("launches_fwd_bwd", r.get("launches_fwd_bwd_pack"))}
        if "one_call_per_group_fwd_bwd_us" in r:
            out[key]["one_call_per_group_fwd_bwd_us"] = round(r["one_call_per_group_fwd_bwd_us"], 2)

    keep(linear_config("C2a FFN up", 8192, 512, 2048, 128, wl.BF16, pk, iters=24, library=False, repeats=3))
    keep(linear_config("C2b FFN down", 8192, 2048, 512, 128, wl.BF16, pk, iters=24, library=False, repeats=3))
    keep(linear_config("C3 LSTM gates", 700, 1500, 6000, 375, wl.BF16, pk, iters=24, library=False, repeats=3))
    keep(linear_config("C3 LSTM gates", 700, 1500, 6000, 375, wl.BF16, pk, pad_pitch=True, iters=24, library=False, repeats=3))
    keep(grouped_config("LSTM layer per gate (8 x 1500->1500 r375, m=700, shared x)", 8, 700, 1500, 1500, 375, pk, True, iters=12, repeats=3))
    keep(grouped_config("attention projections (4 x 512->512 r128, m=8192)", 4, 8192, 512, 512, 128, pk, False, iters=12, repeats=3))
    for name, c in wl.conv_cases().items():
        keep(conv_config(f"{name} conv", c, pk, iters=8, repeats=3))
    for r in (128, 512):
        keep(linear_config(f"C5 sweep r={r}", 16384, 4096, 4096, r, wl.BF16, pk, iters=6, library=False, repeats=3))
        torch.cuda.empty_cache()
    return out


def run(path, pk, only=None, iters=None, repeats=5, library=True):
    """only: optional substring; configurations whose name lacks it are skipped.  iters / repeats /
    library: fewer back-to-back calls per batch, fewer batches, no library comparison (the short
    form a profiler wraps)."""
    rows = []

    def emit(r):
        if r is None:
            return
        rows.append(r)
        with open(path, "w") as f:
            for rr in rows:
                f.write(json.dumps(rr) + "\n")

    def it(default):
        return default if iters is None else iters

    want = (lambda nm: only is None or only in nm)
    lin = dict(library=library, repeats=repeats)
    if want("C1 tiny fp32"):
        emit(linear_config("C1 tiny fp32", 64, 256, 256, 32, wl.F32, pk, iters=it(32), **lin))
    if want("C2a FFN up"):
        emit(linear_config("C2a FFN up", 8192, 512, 2048, 128, wl.BF16, pk, iters=it(32), **lin))
    if want("C2a FFN up + bias + ReLU"):
        emit(act_config("C2a FFN up + bias + ReLU (forward)", 8192, 512, 2048, 128, pk, iters=it(32), repeats=repeats))
    if want("C2b FFN down"):
        emit(linear_config("C2b FFN down", 8192, 2048, 512, 128, wl.BF16, pk, iters=it(32), **lin))
    if want("C3 LSTM gates tight"):
        emit(linear_config("C3 LSTM gates", 700, 1500, 6000, 375, wl.BF16, pk, iters=it(32), **lin))
    if want("C3 LSTM gates padded"):
        emit(linear_config("C3 LSTM gates", 700, 1500, 6000, 375, wl.BF16, pk, pad_pitch=True, iters=it(32), **lin))
    if want("grouped LSTM per gate"):
        emit(grouped_config("grouped LSTM per gate (8 x 1500->1500 r375, m=700, shared x)", 8, 700, 1500, 1500, 375, pk, True,
                            iters=it(24), repeats=repeats))
    if want("grouped attention projections"):
        emit(grouped_config("grouped attention projections (4 x 512->512 r128, m=8192)", 4, 8192, 512, 512, 128, pk, False,
                            iters=it(24), repeats=repeats))
    for name, c in wl.conv_cases().items():
        if want(f"{name} conv"):
            emit(conv_config(f"{name} conv", c, pk, iters=it(20), repeats=repeats))
    for r in wl.SWEEP_RANKS:
        if want(f"C5 sweep r={r}"):
            emit(linear_config(f"C5 sweep r={r}", 16384, 4096, 4096, r, wl.BF16, pk, iters=it(8), **lin))
            torch.cuda.empty_cache()
    # ResNet-18-sized and Transformer-sized factor-gradient lists (Table 4 / Table 3 parameter counts)
    if want("pack ~3.3M elements"):
        emit(pack_config("pack ~3.3M elements", [147457, 16384, 589821, 65536, 1179653, 131072, 1179648, 131071], pk,
                         iters=it(30), repeats=repeats))
    if want("pack ~26.7M elements"):
        emit(pack_config("pack ~26.7M elements", [65536 + (i % 3) for i in range(100)] + [262144 - (i % 5) for i in range(76)], pk,
                         iters=it(30), repeats=repeats))
    return rows


def main():
    """`python bench_suite.py --only "C4 conv" --iters 2`: time (and thereby launch) one or a few
    configurations by themselves, e.g. as the small command a profiler wraps."""
    import argparse
    import os
    import sys
    ap = argparse.ArgumentParser()
    ap.add_argument("--only", required=True, help="substring of the configuration names to run")
    ap.add_argument("--out", default=os.devnull, help="file for the JSON lines")
    ap.add_argument("--iters", type=int, default=None, help="back-to-back calls per timed batch")
    ap.add_argument("--repeats", type=int, default=5, help="timed batches per call")
    ap.add_argument("--no-library", action="store_true", help="skip the library (cuBLAS) comparison")
    args = ap.parse_args()
    root = os.path.dirname(os.path.abspath(__file__))
    if root not in sys.path:
        sys.path.insert(0, root)
    import bench
    torch.cuda.set_device(0)
    for row in run(args.out, bench.peaks(), only=args.only, iters=args.iters, repeats=args.repeats,
                   library=not args.no_library):
        print(json.dumps(row))


if __name__ == "__main__":
    main()
