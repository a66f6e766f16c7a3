"""GPU parity: the flat gradient buffer must be bit-exact (offsets and copied values)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2103_03936_b200 as pf
import pf_workloads as wl
from _gpu import dev, host

pytestmark = pytest.mark.gpu


def check_pack(numels, dtype, seed=0, src_shift=None):
    """src_shift[i] elements of misalignment for source i (tensors carved out of a pool)."""
    tensors_h = wl.pack_list(seed, numels, dtype)
    tensors = []
    for i, t in enumerate(tensors_h):
        sh = 0 if src_shift is None else src_shift[i % len(src_shift)]
        pool = torch.zeros(t.size + sh + 8, dtype=wl.to_torch(t[:1], dtype).dtype, device="cuda")
        pool[sh:sh + t.size] = dev(t, dtype)
        tensors.append(pool[sh:sh + t.size])
    total = int(sum(numels))
    tdt = tensors[0].dtype if tensors else torch.bfloat16
    guard = 32
    buf = torch.full((total + 2 * guard,), -7.0, dtype=tdt, device="cuda")
    flat = buf[guard:guard + total]
    _, offs = pf.pf_pack_factor_grads(tensors, flat=flat)
    torch.cuda.synchronize()
    want_flat, want_offs = oracle.pack(tensors_h)
    assert offs == [int(o) for o in want_offs]
    got = host(flat, dtype)
    assert got.tobytes() == want_flat.tobytes()
    assert torch.all(buf[:guard] == -7.0) and torch.all(buf[guard + total:] == -7.0)


@pytest.mark.parametrize("dtype", [wl.BF16, wl.F32])
def test_small_lists_all_alignments(dtype):
    check_pack([1], dtype)
    check_pack([3, 5], dtype)
    check_pack([7, 0, 2, 1], dtype)
    check_pack([16, 1, 15, 33, 2, 64, 129, 5], dtype)
    for shift in range(8):
        check_pack([37, 8, 101, 1, 64, 3], dtype, seed=shift, src_shift=[shift, (3 * shift) % 8, 1])


@pytest.mark.parametrize("dtype", [wl.BF16, wl.F32])
def test_odd_sizes_across_chunks(dtype):
    check_pack([16385, 40001, 3, 100000, 8191, 16384 * 3 + 7], dtype, src_shift=[0, 1, 3, 5, 7])


def test_c4_factor_gradient_list():
    c = wl.conv_cases()["C4"]
    check_pack([c.kh * c.kw * c.C * c.R, c.O * c.R], wl.BF16)


def test_many_tensors_span_several_launches():
    rng = np.random.default_rng(0)
    numels = [int(v) for v in rng.integers(0, 3000, size=1100)]   # more than two launches' worth of tensors
    check_pack(numels, wl.BF16, src_shift=[0, 1, 2, 3])


def test_whole_model_sized_list():
    """A ResNet-18-sized factor-gradient list (about 3.3 M elements, Table 4's parameter
    count of the factorized model), mixed odd sizes."""
    numels = [147456 + 1, 16384, 589824 - 3, 65536, 1179648 + 5, 131072, 1179648, 131071, 5121]
    check_pack(numels, wl.BF16, src_shift=[0, 3])


def test_capacity_error_and_empty_list():
    g = [torch.ones(10, dtype=torch.bfloat16, device="cuda")]
    with pytest.raises(pf.PfError) as e:
        pf.pf_pack_factor_grads(g, flat=torch.empty(9, dtype=torch.bfloat16, device="cuda"))
    assert e.value.status == 3
    flat, offs = pf.pf_pack_factor_grads([])
    assert offs == [0]


def check_unpack(numels, dtype, seed=0, dst_shift=None, flat_shift=0):
    """The inverse copy: bit-exact slices, guard bands around every destination; dst_shift / flat_shift
    misalign the destinations and the flat buffer by elements."""
    tensors_h = wl.pack_list(seed, numels, dtype)
    flat_h, _ = oracle.pack(tensors_h)
    total = int(sum(numels))
    tdt = wl.to_torch(np.zeros(1, dtype=flat_h.dtype if total else np.uint16), dtype).dtype
    pool = torch.zeros(total + flat_shift + 8, dtype=tdt, device="cuda")
    if total:
        pool[flat_shift:flat_shift + total] = dev(flat_h, dtype)
    flat = pool[flat_shift:flat_shift + total]
    guard = 16
    bufs, dsts = [], []
    for i, n in enumerate(numels):
        sh = 0 if dst_shift is None else dst_shift[i % len(dst_shift)]
        b = torch.full((n + sh + 2 * guard,), -7.0, dtype=tdt, device="cuda")
        bufs.append((b, sh))
        dsts.append(b[guard + sh:guard + sh + n])
    offs = pf.pf_unpack_factor_grads(flat, dsts)
    torch.cuda.synchronize()
    want, want_offs = oracle.unpack(flat_h, numels)
    assert offs == [int(o) for o in want_offs]
    for (b, sh), d, w, n in zip(bufs, dsts, want, numels):
        assert host(d, dtype).tobytes() == w.tobytes()
        assert torch.all(b[:guard + sh] == -7.0) and torch.all(b[guard + sh + n:] == -7.0)


@pytest.mark.parametrize("dtype", [wl.BF16, wl.F32])
def test_unpack_small_lists_all_alignments(dtype):
    check_unpack([1], dtype)
    check_unpack([3, 5], dtype)
    check_unpack([7, 0, 2, 1], dtype)
    check_unpack([16, 1, 15, 33, 2, 64, 129, 5], dtype)
    for shift in range(8):
        check_unpack([37, 8, 101, 1, 64, 3], dtype, seed=shift, dst_shift=[shift, (3 * shift) % 8, 1], flat_shift=(5 * shift) % 8)


def test_unpack_round_trip_at_model_scale():
    numels = [147457, 16384, 589821, 65536, 1179653, 131072]
    tensors = [torch.randn(n, device="cuda").to(torch.bfloat16) for n in numels]
    flat, offs = pf.pf_pack_factor_grads(tensors)
    back = [torch.full_like(t, -7.0) for t in tensors]
    offs2 = pf.pf_unpack_factor_grads(flat, back)
    torch.cuda.synchronize()
    assert offs == offs2
    for a, b in zip(tensors, back):
        assert torch.equal(a, b)
    with pytest.raises(pf.PfError) as e:          # a list longer than the flat buffer is refused
        pf.pf_unpack_factor_grads(flat[:100], back)
    assert e.value.status == 3
