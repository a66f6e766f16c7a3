"""Helpers shared by the tests (no method arithmetic of the CUDA path or the oracle)."""
import numpy as np


def read_golden(path):
    """Parse 'name d0 d1 ... : v0 v1 ...' lines into float64 arrays."""
    out = {}
    with open(path) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            head, vals = line.split(":")
            parts = head.split()
            shape = tuple(int(p) for p in parts[1:])
            out[parts[0]] = np.array([float(v) for v in vals.split()]).reshape(shape)
    return out


def read_counts(path):
    out = {}
    with open(path) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            key, val = line.split(None, 1)
            val = val.strip()
            out[key] = tuple(int(v) for v in val.split(",")) if "," in val else int(val)
    return out


def rng_int(seed, shape, lo=-3, hi=4):
    """Small-integer test data: products and sums are exact in fp64."""
    return np.random.default_rng(seed).integers(lo, hi, size=shape).astype(np.float64)
