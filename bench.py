#!/usr/bin/env python
"""Benchmark of the factorized-layer hot path on B200.

A step is one pass of the whole hot path over one batch of synthetic input shaped like the
Transformer FFN of the paper's Appendix D at rank 1/4: forward of the up-projection
(8192 x 512 -> 2048, r = 128) and of the down-projection (8192 x 2048 -> 512, r = 128), the
backward of both (dX, dU, dV each), and the flat gradient buffer over the four factor
gradients.  All of it runs in this repository's CUDA kernels through the C ABI.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--suite FILE]

Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank runs an independent replica
(the path has no exchange step; the packed buffer is the message a trainer would all-reduce).
`--impl reference` times the fp64 CPU oracle on bounded samples of the same workload.
`--suite FILE` additionally writes per-config timings (LSTM, conv, rank sweep, ...) to FILE.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import pf_workloads as wl  # noqa: E402

METRIC = "factorized-layer fwd+bwd TFLOP/s (and HBM GB/s, fraction of roofline), B200"
WORKLOAD = ("Transformer FFN factorized linear bf16: m=8192 (64x128 tokens), 512->2048 r=128 and "
            "2048->512 r=128, fwd+bwd (dX,dU,dV) + pf_pack_factor_grads of the 4 factor grads")
NSETS = 4  # activation buffer sets rotated between steps so that inputs never sit in L2

# DRAM read + write bytes of one FFN-up forward launch of the dominant kernel, from an ncu capture
# (dram__bytes_read.sum + dram__bytes_write.sum; its summary is kept with the other profile
# summaries); valid while the kernel's sources hash to the value recorded with that capture.
DOMINANT_TRAFFIC_BYTES = 9084928
DOMINANT_SOURCES = ("pf_tc_chain_kernel.cuh", "pf_tc_chain.cu", "pf_tc_prims.cuh", "pf_tc_host.h")
DOMINANT_SHA256 = "741c6958f0d816ad6688e2011454312d007d9ddc7fe2514ff251685c1511015c"


def dominant_traffic():
    import hashlib
    m = hashlib.sha256()
    try:
        for f in DOMINANT_SOURCES:
            with open(os.path.join(ROOT, "paper_2103_03936_b200", "csrc", f), "rb") as fh:
                m.update(fh.read())
    except OSError:
        return None
    return DOMINANT_TRAFFIC_BYTES if m.hexdigest() == DOMINANT_SHA256 else None


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


def linear_flops(c):      # fwd 2mr(k+n) + bwd 4mr(k+n)
    return 6.0 * c.m * c.r * (c.k + c.n)


def linear_bytes(c, stash=True):
    """Algorithmic minimum bytes fwd + bwd: every operand read once, every result written
    once, the m x r intermediates never leaving the chip; a stashed T adds one write+read."""
    s = 2 if c.dtype == wl.BF16 else 4
    fwd = s * (c.m * c.k + c.m * c.n + c.r * (c.k + c.n))
    bwd = s * (c.m * c.n + 2 * c.m * c.k + 2 * c.r * (c.k + c.n))
    return fwd, bwd, (2 * s * c.m * c.r if stash else 0)


def linear_floor_us(c, pk):
    fwd_b, bwd_b, stash_b = linear_bytes(c)
    fl = linear_flops(c)
    f = max(fl / 3 / (pk["bf16_tflops"] * 1e12), fwd_b / (pk["hbm_gbs"] * 1e9))
    b = max(2 * fl / 3 / (pk["bf16_tflops"] * 1e12), bwd_b / (pk["hbm_gbs"] * 1e9))
    return (f + b) * 1e6


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU while the timed region runs."""

    def __init__(self, index: int):
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40,
                 "sw_thermal_slowdown": 0x20, "hw_power_brake_slowdown": 0x80}
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for nm, bit in names.items():
                    if mask & bit:
                        self.reasons.add(nm)
            except Exception:
                pass
            time.sleep(0.005)

    def start(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()

    def stop(self):
        self._stop.set()
        if self._thr is not None:
            self._thr.join()
        med = int(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ----------------------------------------------------------------------------- reference arm
def oracle_step_sample(cases, data, rows):
    import oracle
    for c, d in zip(cases, data):
        x, dY = d["x"][:rows], d["dY"][:rows]
        oracle.linear_fwd(x, d["U"], d["V"])
        oracle.linear_bwd(x, d["U"], d["V"], dY)
    bufs = [np.zeros(c.k * c.r, np.uint16) for c in cases] + [np.zeros(c.n * c.r, np.uint16) for c in cases]
    oracle.pack(bufs)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    cases = [wl.linear_cases()["C2a"], wl.linear_cases()["C2b"]]
    max_rows = 2048
    data = []
    for c in cases:
        small = wl.LinearCase(c.name, max_rows, c.k, c.n, c.r, c.dtype, c.seed)
        data.append({k_: oracle.widen(v) for k_, v in small.generate().items()})
    # calibrate: rows per step such that warmup + steps end within about two minutes
    t0 = time.perf_counter()
    oracle_step_sample(cases, data, 64)
    per_row = (time.perf_counter() - t0) / 64
    budget = 120.0 / max(1, args.steps + args.warmup)
    rows = int(max(16, min(max_rows, budget / max(per_row, 1e-9))))
    for _ in range(args.warmup):
        oracle_step_sample(cases, data, rows)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step_sample(cases, data, rows)
    dt = (time.perf_counter() - t0) / max(1, args.steps)
    flops = sum(6.0 * rows * c.r * (c.k + c.n) for c in cases)
    val = flops / dt / 1e12
    sample = f"first {rows} of 8192 token rows of both FFN layers per step, fwd+bwd+pack, fp64"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": oracle.threads(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ----------------------------------------------------------------------------- our arm
class FfnWorkload:
    def __init__(self, torch, pf, device):
        self.torch, self.pf = torch, pf
        self.cases = [wl.linear_cases()["C2a"], wl.linear_cases()["C2b"]]
        self.host = [c.generate() for c in self.cases]
        stream = torch.cuda.current_stream()
        self.sets = []
        self.calls = []          # per set: list of (name, prepared call)
        self.pinned_in, self.dev_in = [], []
        for s in range(NSETS):
            layer_bufs, calls = [], []
            grads = []
            for c, h in zip(self.cases, self.host):
                x, U, V, dY = (wl.to_torch(h[k_], c.dtype).to(device) for k_ in ("x", "U", "V", "dY"))
                y = torch.empty((c.m, c.n), dtype=torch.bfloat16, device=device)
                T = torch.empty((c.m, c.r), dtype=torch.bfloat16, device=device)
                dX = torch.empty((c.m, c.k), dtype=torch.bfloat16, device=device)
                dU = torch.empty((c.k, c.r), dtype=torch.bfloat16, device=device)
                dV = torch.empty((c.n, c.r), dtype=torch.bfloat16, device=device)
                wsf = torch.empty(max(256, pf.pf_lowrank_linear_workspace(c.m, c.k, c.n, c.r, pf.PF_BF16, 0)),
                                  dtype=torch.uint8, device=device)
                wsb = torch.empty(max(256, pf.pf_lowrank_linear_workspace(c.m, c.k, c.n, c.r, pf.PF_BF16, 1)),
                                  dtype=torch.uint8, device=device)
                fwd, _ = pf.pf_lowrank_linear_fwd(x, U, V, y=y, T_stash=T, workspace=wsf,
                                                  stream=stream, prepare=True)
                bwd, _ = pf.pf_lowrank_linear_bwd(x, U, V, dY, T_stash=T, dX=dX, dU=dU, dV=dV,
                                                  workspace=wsb, stream=stream, prepare=True)
                layer_bufs.append(dict(x=x, U=U, V=V, dY=dY, y=y, T=T, dX=dX, dU=dU, dV=dV))
                calls.append((fwd, bwd))
                grads += [dU, dV]
            flat = torch.empty(sum(g.numel() for g in grads), dtype=torch.bfloat16, device=device)
            pack, _ = pf.pf_pack_factor_grads(grads, flat=flat, stream=stream, prepare=True)
            self.sets.append(dict(layers=layer_bufs, flat=flat))
            self.calls.append([("fwd_up", calls[0][0]), ("fwd_down", calls[1][0]),
                               ("bwd_down", calls[1][1]), ("bwd_up", calls[0][1]), ("pack", pack)])
        # pinned host copies for the end-to-end measurement
        self.pin = [{k_: wl.to_torch(h[k_], c.dtype).pin_memory() for k_ in ("x", "dY")}
                    for c, h in zip(self.cases, self.host)]
        self.flat_host = torch.empty(self.sets[0]["flat"].numel(), dtype=torch.bfloat16).pin_memory()
        self.flops = sum(linear_flops(c) for c in self.cases)
        self.h2d = sum(p["x"].numel() * 2 + p["dY"].numel() * 2 for p in self.pin)
        self.d2h = self.flat_host.numel() * 2

    def step(self, i):
        for _, call in self.calls[i % NSETS]:
            call()

    def step_e2e(self, i):
        s = self.sets[i % NSETS]
        for lay, p in zip(s["layers"], self.pin):
            lay["x"].copy_(p["x"], non_blocking=True)
            lay["dY"].copy_(p["dY"], non_blocking=True)
        for _, call in self.calls[i % NSETS]:
            call()
        self.flat_host.copy_(s["flat"], non_blocking=True)


def max_over_ranks(torch, values, dist, device):
    """Element-wise maximum of a list of floats over all ranks (the values themselves when not
    distributed): a multi-GPU time is the slowest rank's."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def time_region(torch, fn, steps, barrier):
    barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        fn(i)
    e1.record()
    torch.cuda.synchronize()
    barrier()
    return e0.elapsed_time(e1) / 1e3


def cpu_baseline(cases, host):
    """The oracle as it stands, on this machine's host cores, on the full FFN workload."""
    import oracle
    wide = [{k_: oracle.widen(v) for k_, v in h.items()} for h in host]
    reps, total = 0, 0.0
    while reps < 5 and total < 10.0:
        t0 = time.perf_counter()
        for c, d in zip(cases, wide):
            oracle.linear_fwd(d["x"], d["U"], d["V"])
            oracle.linear_bwd(d["x"], d["U"], d["V"], d["dY"])
        oracle.pack([np.zeros(c.k * c.r, np.uint16) for c in cases] +
                    [np.zeros(c.n * c.r, np.uint16) for c in cases])
        total += time.perf_counter() - t0
        reps += 1
    flops = sum(linear_flops(c) for c in cases)
    return {"value": flops * reps / total / 1e12, "unit": "TFLOP/s", "cores": oracle.threads(),
            "kind": "oracle",
            "sample": f"the full FFN workload (all 8192 rows, both layers, fwd+bwd+pack), {reps} repetition(s), fp64"}


def run_ours(args):
    import torch
    import paper_2103_03936_b200 as pf

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback exists)")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_
        dist = dist_
        dist.init_process_group("nccl", device_id=device)

    def barrier():
        if dist is not None:
            dist.barrier()

    pk = peaks()
    w = FfnWorkload(torch, pf, device)
    for i in range(max(args.warmup, 3)):
        w.step(i)
    torch.cuda.synchronize()
    assert pf.pf_last_device_status() == 0

    # --- timed region: K steps
    dom_name = "fwd_up"
    launches0 = pf.pf_launch_count()

    sampler = ClockSampler(local)
    sampler.start()
    secs = time_region(torch, w.step, args.steps, barrier)
    clocks = sampler.stop()
    launches = pf.pf_launch_count() - launches0
    # the dominant kernel on its own: batches of back-to-back launches of the FFN-up forward, rotating
    # over the buffer sets, between two events (no event between launches, so none of their cost)
    fwd_up = [dict(c)[dom_name] for c in w.calls]
    batch, dom_batches = 32, []
    for rep in range(5):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for i in range(batch):
            fwd_up[i % NSETS]()
        b.record()
        torch.cuda.synchronize()
        dom_batches.append(a.elapsed_time(b) * 1e3 / batch)
    dom_us = float(np.median(dom_batches))

    # --- end to end: pinned host inputs in, packed gradients out, every step
    for i in range(3):
        w.step_e2e(i)
    e2e_secs = time_region(torch, w.step_e2e, args.steps, barrier)
    status = pf.pf_last_device_status()
    if status != 0:
        raise SystemExit(f"device status {pf.pf_status_string(status)}")

    secs, e2e_secs = max_over_ranks(torch, [secs, e2e_secs], dist, device)
    per_step = secs / args.steps
    value = world * w.flops / per_step / 1e12
    byts = sum(sum(linear_bytes(c)) for c in w.cases) + 2 * w.d2h
    floor_us = sum(linear_floor_us(c, pk) for c in w.cases)

    c0 = w.cases[0]
    dom_bytes = linear_bytes(c0)[0] + linear_bytes(c0)[2] // 2      # fwd bytes + the T stash write
    roofline = None
    if dom_us:
        ach = dom_bytes / (dom_us * 1e-6) / 1e9
        roofline = {"bound": "hbm", "kernel": "pf_lowrank_linear_fwd (FFN up, 8192x512->2048 r128)",
                    "achieved": ach, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": ach / pk["hbm_gbs"],
                    "traffic": dominant_traffic(), "peak_source": pk["source"], "us_per_launch": dom_us,
                    "timing": f"median of 5 batches of {batch} back-to-back launches on the launching stream, CUDA events around each batch",
                    "algorithmic_bytes_per_launch": dom_bytes}

    out = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": per_step * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD, "cache": f"{NSETS} activation buffer sets rotated (footprint "
                   f"{NSETS * 172} MB > 126 MB L2)", "parallelism": "replicas only" if world > 1 else "1 GPU"},
        "gbs": world * byts / per_step / 1e9,
        "roofline_frac_step": floor_us * 1e-6 / per_step,
        "roofline_floor_us": floor_us,
        "clocks": clocks,
        "e2e": {"value": world * w.flops / (e2e_secs / args.steps) / 1e12, "unit": "TFLOP/s",
                "h2d_bytes_per_step": w.h2d, "d2h_bytes_per_step": w.d2h,
                "ms_per_step": e2e_secs / args.steps * 1e3},
        "gpu_launches": int(launches),
        "roofline": roofline,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(w.cases, w.host)
    if rank == 0:
        import bench_suite as suite
        cases, host = w.cases, w.host
        del w
        torch.cuda.empty_cache()
        if world == 1 and not args.no_configs:
            # the other configurations the roofline target names (LSTM gates, convolutions, rank sweep)
            out["configs"] = suite.quick(pk)
            out["configs_protocol"] = ("per configuration: median over 3 batches of 6-24 back-to-back calls between two "
                                       "CUDA events, buffer sets rotated so that inputs exceed L2; floor = max(FLOPs / "
                                       "bf16 peak, minimum bytes / HBM bandwidth) per pass, of measured peaks")
        if args.suite:
            suite.run(args.suite, pk, only=args.suite_only)
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--suite", default=None, help="also write per-config timings to this file")
    ap.add_argument("--suite-only", default=None, help="substring filter on suite configuration names")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the per-configuration timings")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
