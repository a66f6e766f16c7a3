"""Seeded synthetic inputs shaped like the paper's factorized layers.

This module only *generates data*: a counter-based integer hash gives uniforms,
Box-Muller gives normals, and every value is rounded once (round-to-nearest-even)
to the storage type.  It holds none of the method's arithmetic, so the fp64 oracle
and the CUDA library can both consume exactly the same stored values.

bf16 tensors are carried as ``numpy.uint16`` bit patterns (numpy has no bf16);
fp32 tensors as ``numpy.float32``.

Shapes follow the paper's architecture tables (Transformer FFN factors 512x128 /
128x2048 / 2048x128 / 128x512 in Appendix D; LSTM gate factors 1500x375 in the LSTM
table; ResNet-18 conv_u (256,64,3,3) + conv_v (64,256,1,1)) at the global rank ratio
1/4 of Section 4.  They stand in for CIFAR-10 / ImageNet / WikiText-2 / WMT16
activations, which are not needed: only layer shapes and plausible value
distributions matter to the kernels.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

F32 = "f32"
BF16 = "bf16"

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def _mix64(z: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser on a uint64 array (wrap-around arithmetic)."""
    with np.errstate(over="ignore"):
        z = (z + np.uint64(0x9E3779B97F4A7C15)) & _M64
        z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _M64
        z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _M64
        z = z ^ (z >> np.uint64(31))
    return z


def _uniform01(seed: int, stream: int, lane: int, count: int) -> np.ndarray:
    """count uniforms in the open interval (0,1); element i depends only on
    (seed, stream, lane, i)."""
    key = int(_mix64(np.array([(seed * 0x1000193 + stream) & 0xFFFFFFFFFFFFFFFF],
                              dtype=np.uint64))[0])
    out = np.empty(count, dtype=np.float64)
    chunk = 1 << 22
    for s in range(0, count, chunk):
        e = min(count, s + chunk)
        ctr = np.arange(s, e, dtype=np.uint64) * np.uint64(2) + np.uint64(lane)
        with np.errstate(over="ignore"):
            h = _mix64(ctr ^ np.uint64(key))
            h = _mix64(h + np.uint64(key))
        out[s:e] = ((h >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)
    return out


def uniform(seed: int, stream: int, shape, lo: float = -1.0, hi: float = 1.0) -> np.ndarray:
    n = int(np.prod(shape))
    u = _uniform01(seed, stream, 0, n)
    return (lo + (hi - lo) * u).reshape(shape)


def normal(seed: int, stream: int, shape, sigma: float = 1.0) -> np.ndarray:
    n = int(np.prod(shape))
    u1 = _uniform01(seed, stream, 0, n)
    u2 = _uniform01(seed, stream, 1, n)
    z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * math.pi * u2)
    return (sigma * z).reshape(shape)


def round_to(a64: np.ndarray, dtype: str) -> np.ndarray:
    """Round fp64 values once to the storage type (RNE).

    bf16 is reached in one rounding step: the fp64 value is first narrowed to fp32 with
    round-to-odd (truncate, then set the last bit when anything was cut off), which keeps
    enough information for the final round-to-nearest-even to 8 significand bits to be
    the correctly rounded bf16 of the fp64 value (no double rounding)."""
    a64 = np.ascontiguousarray(a64, dtype=np.float64)
    f32 = a64.astype(np.float32)
    if dtype == F32:
        return f32
    if dtype == BF16:
        back = f32.astype(np.float64)
        inexact = back != a64
        # truncate toward zero where RNE went away from zero, then force the last bit odd
        away = inexact & (np.abs(back) > np.abs(a64))
        bits = f32.view(np.uint32).copy()
        bits[away] -= np.uint32(1)
        bits[inexact] |= np.uint32(1)
        bias = np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1))
        return ((bits + bias) >> np.uint32(16)).astype(np.uint16)
    raise ValueError(dtype)


def to_torch(a: np.ndarray, dtype: str, device="cpu"):
    """Stored values as a torch tensor of the matching dtype (bit-preserving)."""
    import torch
    if dtype == F32:
        t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
    else:
        t = torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)
    return t.to(device) if device != "cpu" else t


def from_torch(t, dtype: str) -> np.ndarray:
    """Inverse of to_torch: stored bit patterns back as numpy."""
    import torch
    t = t.detach().cpu().contiguous()
    if dtype == F32:
        return t.numpy()
    return t.view(torch.int16).numpy().view(np.uint16)


@dataclass
class LinearCase:
    name: str
    m: int
    k: int
    n: int
    r: int
    dtype: str
    seed: int
    x_dist: str = "normal"          # "normal" N(0,1) or "uniform" U(-1,1)
    factor_seed: int | None = None  # factors drawn from another seed (rank sweep)
    note: str = ""

    def generate(self):
        """x[m,k], U[k,r], V[n,r], dY[m,n] in the storage type."""
        fs = self.seed if self.factor_seed is None else self.factor_seed
        sig = 1.0 / math.sqrt(self.k)
        if self.x_dist == "uniform":
            x = uniform(self.seed, 0, (self.m, self.k))
        else:
            x = normal(self.seed, 0, (self.m, self.k))
        U = normal(fs, 1, (self.k, self.r), sig)
        V = normal(fs, 2, (self.n, self.r), sig)
        dY = normal(self.seed, 3, (self.m, self.n))
        return {nm: round_to(a, self.dtype) for nm, a in
                (("x", x), ("U", U), ("V", V), ("dY", dY))}


@dataclass
class ConvCase:
    name: str
    N: int
    H: int
    W: int
    C: int
    R: int
    O: int
    dtype: str
    seed: int
    kh: int = 3
    kw: int = 3
    stride: int = 1
    pad: int = 1
    note: str = ""

    @property
    def Ho(self):
        return (self.H + 2 * self.pad - self.kh) // self.stride + 1

    @property
    def Wo(self):
        return (self.W + 2 * self.pad - self.kw) // self.stride + 1

    def generate(self):
        """x[N,H,W,C] (post-ReLU: clamped at 0), U[kh,kw,C,R], V[O,R] Kaiming-normal
        (fan-in), dY[N,Ho,Wo,O]."""
        x = np.maximum(normal(self.seed, 0, (self.N, self.H, self.W, self.C)), 0.0)
        U = normal(self.seed, 1, (self.kh, self.kw, self.C, self.R),
                   math.sqrt(2.0 / (self.kh * self.kw * self.C)))
        V = normal(self.seed, 2, (self.O, self.R), math.sqrt(2.0 / self.R))
        dY = normal(self.seed, 3, (self.N, self.Ho, self.Wo, self.O))
        return {nm: round_to(a, self.dtype) for nm, a in
                (("x", x), ("U", U), ("V", V), ("dY", dY))}


SWEEP_RANKS = (16, 32, 64, 128, 256, 512, 1024)


def linear_cases() -> dict[str, LinearCase]:
    c = {
        "C1": LinearCase("C1", 64, 256, 256, 32, F32, 0, note="tiny fp32"),
        "C2a": LinearCase("C2a", 8192, 512, 2048, 128, BF16, 1, note="Transformer FFN up"),
        "C2b": LinearCase("C2b", 8192, 2048, 512, 128, BF16, 2, note="Transformer FFN down"),
        "C3i": LinearCase("C3i", 700, 1500, 6000, 375, BF16, 3, x_dist="uniform",
                          note="LSTM gates, input-to-hidden"),
        "C3h": LinearCase("C3h", 700, 1500, 6000, 375, BF16, 4, x_dist="uniform",
                          note="LSTM gates, hidden-to-hidden"),
    }
    for r in SWEEP_RANKS:
        c[f"C5r{r}"] = LinearCase(f"C5r{r}", 16384, 4096, 4096, r, BF16, 6,
                                  factor_seed=6 + int(math.log2(r)), note="rank sweep")
    return c


def conv_cases() -> dict[str, ConvCase]:
    return {
        "C4": ConvCase("C4", 128, 32, 32, 256, 64, 256, BF16, 5, note="ResNet-18 style 3x3"),
        "C5b": ConvCase("C5b", 256, 14, 14, 256, 64, 256, BF16, 7, note="ResNet-50 style 14x14"),
    }


def pack_list(seed: int, numels, dtype: str):
    """A list of 1-D 'gradient' tensors with the given element counts."""
    return [round_to(normal(seed, 10 + i, (int(n),)), dtype) for i, n in enumerate(numels)]
