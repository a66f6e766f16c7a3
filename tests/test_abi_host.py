"""CPU-only checks of the C-ABI boundary: the library loads, exports every symbol the header
declares, and rejects bad arguments on the host before anything is launched."""
import ctypes
import os
import re

import pytest

import paper_2103_03936_b200 as pf
from paper_2103_03936_b200 import build as pf_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
OK, INVALID, UNSUPPORTED, WORKSPACE = 0, 1, 2, 3
P = 0x7F0000001000  # fake, element- and 256-byte-aligned "device pointer"; never dereferenced


@pytest.fixture(scope="module")
def L():
    pf_build.build()
    return pf.lib()


def test_every_declared_symbol_is_exported(L):
    hdr = open(os.path.join(ROOT, "include", "pf.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"\b(pf_[a-z0-9_]+)\s*\(", hdr))
    assert {"pf_lowrank_linear_fwd", "pf_lowrank_linear_bwd", "pf_lowrank_conv_fwd",
            "pf_lowrank_conv_bwd", "pf_pack_factor_grads"} <= names
    for nm in names:
        assert hasattr(L, nm), nm


def test_version_and_status_strings(L):
    assert pf.pf_version() >= 100
    assert pf.pf_status_string(0) == "PF_OK"
    assert pf.pf_status_string(5) == "PF_ERR_TIMEOUT"
    assert pf.pf_status_string(99) == "PF_ERR_UNKNOWN"


def _lin_fwd(L, **kw):
    a = dict(x=P, ldx=8, U=P, ldu=4, V=P, ldv=4, y=P, ldy=6, T=0, ldt=0, m=5, k=8, n=6, r=4, dtype=1,
             ws=P, wsb=1 << 30, stream=0)
    a.update(kw)
    return L.pf_lowrank_linear_fwd(a["x"], a["ldx"], a["U"], a["ldu"], a["V"], a["ldv"], a["y"],
                                   a["ldy"], a["T"], a["ldt"], a["m"], a["k"], a["n"], a["r"],
                                   a["dtype"], a["ws"], a["wsb"], a["stream"])


def test_linear_fwd_rejects_bad_arguments(L):
    assert _lin_fwd(L, x=0) == INVALID
    assert _lin_fwd(L, U=0) == INVALID
    assert _lin_fwd(L, y=0) == INVALID
    assert _lin_fwd(L, r=0) == INVALID
    assert _lin_fwd(L, k=0) == INVALID
    assert _lin_fwd(L, m=-1) == INVALID
    assert _lin_fwd(L, ldx=7) == INVALID
    assert _lin_fwd(L, ldv=3) == INVALID
    assert _lin_fwd(L, ldy=5) == INVALID
    assert _lin_fwd(L, dtype=7) == INVALID
    assert _lin_fwd(L, x=P + 1) == INVALID            # not element-aligned
    assert _lin_fwd(L, T=P, ldt=3) == INVALID
    assert _lin_fwd(L, ws=0) == WORKSPACE
    assert _lin_fwd(L, ws=P + 16) == WORKSPACE         # not 256-byte aligned
    assert _lin_fwd(L, wsb=8) == WORKSPACE
    assert _lin_fwd(L, m=0) == OK                      # empty problem: no launch


def test_linear_bwd_rejects_bad_arguments(L):
    def call(**kw):
        a = dict(x=P, ldx=8, U=P, ldu=4, V=P, ldv=4, dY=P, lddy=6, T=0, ldt=0, dX=P, lddx=8,
                 dU=P, lddu=4, dV=P, lddv=4, m=5, k=8, n=6, r=4, dtype=0, ws=P, wsb=1 << 30)
        a.update(kw)
        return L.pf_lowrank_linear_bwd(a["x"], a["ldx"], a["U"], a["ldu"], a["V"], a["ldv"],
                                       a["dY"], a["lddy"], a["T"], a["ldt"], a["dX"], a["lddx"],
                                       a["dU"], a["lddu"], a["dV"], a["lddv"], a["m"], a["k"],
                                       a["n"], a["r"], a["dtype"], a["ws"], a["wsb"], 0)
    assert call(dY=0) == INVALID
    assert call(dU=0) == INVALID
    assert call(dV=0) == INVALID
    assert call(lddy=5) == INVALID
    assert call(lddx=7) == INVALID
    assert call(lddu=3) == INVALID
    assert call(dU=P + 2) == INVALID                   # fp32 needs 4-byte alignment
    assert call(wsb=16) == WORKSPACE


def test_workspace_queries(L):
    assert pf.pf_lowrank_linear_workspace(8192, 512, 2048, 128, pf.PF_BF16, 0) > 0
    assert pf.pf_lowrank_linear_workspace(8192, 512, 2048, 128, pf.PF_BF16, 1) >= \
        pf.pf_lowrank_linear_workspace(8192, 512, 2048, 128, pf.PF_BF16, 0)
    assert pf.pf_lowrank_linear_workspace(8, 0, 4, 4, pf.PF_BF16, 0) == 0      # invalid dims
    assert pf.pf_lowrank_conv_workspace(2, 8, 8, 8, 4, 8, 3, 3, 1, 1, pf.PF_BF16, 1) > 0


def _conv_fwd(L, **kw):
    a = dict(x=P, U=P, V=P, y=P, T=0, N=2, H=8, W=8, C=8, R=4, O=8, kh=3, kw=3, stride=1, pad=1,
             dtype=1, ws=P, wsb=1 << 30)
    a.update(kw)
    return L.pf_lowrank_conv_fwd(a["x"], a["U"], a["V"], a["y"], a["T"], a["N"], a["H"], a["W"],
                                 a["C"], a["R"], a["O"], a["kh"], a["kw"], a["stride"], a["pad"],
                                 a["dtype"], a["ws"], a["wsb"], 0)


def test_conv_fwd_rejects_bad_arguments(L):
    assert _conv_fwd(L, x=0) == INVALID
    assert _conv_fwd(L, y=0) == INVALID
    assert _conv_fwd(L, R=0) == INVALID
    assert _conv_fwd(L, pad=-1) == INVALID
    assert _conv_fwd(L, kh=3, kw=1) == UNSUPPORTED
    assert _conv_fwd(L, stride=0) == UNSUPPORTED
    assert _conv_fwd(L, H=1, W=1, pad=0) == INVALID    # kernel larger than padded image
    assert _conv_fwd(L, wsb=0) == WORKSPACE
    assert _conv_fwd(L, N=0) == OK


def test_pack_host_side_contract(L):
    i64 = ctypes.c_int64
    offs = (i64 * 4)()
    ptrs = (ctypes.c_void_p * 3)(P, P + 64, P + 128)
    numels = (i64 * 3)(5, 0, 7)
    # capacity too small: offsets are still the prefix sums, status says so, nothing launched
    st = L.pf_pack_factor_grads(ptrs, numels, 3, 1, P, 11, offs, None, 0, None)
    assert st == WORKSPACE and list(offs) == [0, 5, 5, 12]
    assert L.pf_pack_factor_grads(ptrs, numels, -1, 1, P, 100, offs, None, 0, None) == INVALID
    assert L.pf_pack_factor_grads(None, numels, 3, 1, P, 100, offs, None, 0, None) == INVALID
    assert L.pf_pack_factor_grads(ptrs, numels, 3, 1, P, 100, None, None, 0, None) == INVALID
    assert L.pf_pack_factor_grads(ptrs, numels, 3, 5, P, 100, offs, None, 0, None) == INVALID
    bad = (i64 * 3)(5, -1, 7)
    assert L.pf_pack_factor_grads(ptrs, bad, 3, 1, P, 100, offs, None, 0, None) == INVALID
    odd = (ctypes.c_void_p * 3)(P + 1, P + 64, P + 128)
    assert L.pf_pack_factor_grads(odd, numels, 3, 1, P, 100, offs, None, 0, None) == INVALID
    assert L.pf_pack_factor_grads(ptrs, numels, 3, 1, None, 100, offs, None, 0, None) == INVALID
    # empty list and all-empty tensors are no-ops
    assert L.pf_pack_factor_grads(None, None, 0, 1, None, 0, offs, None, 0, None) == OK
    assert offs[0] == 0
    zeros = (i64 * 3)(0, 0, 0)
    assert L.pf_pack_factor_grads(ptrs, zeros, 3, 1, None, 0, offs, None, 0, None) == OK


def test_binding_raises_when_library_is_missing(monkeypatch, tmp_path):
    """No fallback: a missing library is an ImportError, not a silent slow path."""
    from paper_2103_03936_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(ImportError):
        binding.lib()
