"""ctypes binding over libpf.so: argument marshalling only.

Every function has the name and the semantics of the C entry point it wraps (see
``include/pf.h``).  Tensors are torch CUDA tensors; torch is used for device memory and the
current stream, nothing else.  Outputs and workspaces that the caller does not pass are
allocated here with torch (the C library itself never allocates).
"""
from __future__ import annotations

import ctypes
import os

import torch

PF_F32, PF_BF16 = 0, 1
PF_ACT_NONE, PF_ACT_RELU = 0, 1
PF_GRAD_ACCUMULATE, PF_GRAD_F32 = 1, 2
_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libpf.so")
_lib = None


class PfError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {pf_status_string(status)} ({status})")


def lib() -> ctypes.CDLL:
    """The loaded C library; raises if it has not been built (no fallback path exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2103_03936_b200.build` "
                "(there is no CPU or PyTorch fallback)")
        L = ctypes.CDLL(_LIB_PATH)
        i64, vp, sz, ci = ctypes.c_int64, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
        L.pf_status_string.restype = ctypes.c_char_p
        L.pf_status_string.argtypes = [ci]
        L.pf_version.restype = ci
        L.pf_last_device_status.restype = ci
        L.pf_launch_count.restype = ctypes.c_longlong
        L.pf_lowrank_linear_workspace.restype = sz
        L.pf_lowrank_linear_workspace.argtypes = [i64, i64, i64, i64, ci, ci]
        L.pf_lowrank_linear_fwd.restype = ci
        L.pf_lowrank_linear_fwd.argtypes = [vp, i64, vp, i64, vp, i64, vp, i64, vp, i64,
                                            i64, i64, i64, i64, ci, vp, sz, vp]
        L.pf_lowrank_linear_fwd_act.restype = ci
        L.pf_lowrank_linear_fwd_act.argtypes = [vp, i64, vp, i64, vp, i64, vp, ci, vp, i64, vp, i64,
                                                i64, i64, i64, i64, ci, vp, sz, vp]
        L.pf_bias_act_bwd_workspace.restype = sz
        L.pf_bias_act_bwd_workspace.argtypes = [i64, i64]
        L.pf_bias_act_bwd.restype = ci
        L.pf_bias_act_bwd.argtypes = [vp, i64, vp, i64, vp, i64, i64, ci, ci, vp, sz, vp]
        L.pf_lowrank_linear_fwd_static.restype = ci
        L.pf_lowrank_linear_fwd_static.argtypes = [vp, i64, vp, i64, vp, i64, vp, i64, vp, i64,
                                                   i64, i64, i64, i64, ci, vp]
        L.pf_static_scratch_bytes.restype = sz
        L.pf_lowrank_linear_bwd.restype = ci
        L.pf_lowrank_linear_bwd.argtypes = [vp, i64, vp, i64, vp, i64, vp, i64, vp, i64,
                                            vp, i64, vp, i64, vp, i64,
                                            i64, i64, i64, i64, ci, vp, sz, vp]
        L.pf_lowrank_linear_bwd_ex.restype = ci
        L.pf_lowrank_linear_bwd_ex.argtypes = [vp, i64, vp, i64, vp, i64, vp, i64, vp, i64,
                                               vp, i64, vp, i64, vp, i64, i64, i64, i64, i64, ci, ctypes.c_uint, vp, sz, vp]
        L.pf_lowrank_linear_grouped_workspace.restype = sz
        L.pf_lowrank_linear_grouped_workspace.argtypes = [ci, i64, i64, i64, i64, ci, ci]
        L.pf_lowrank_linear_grouped_fwd.restype = ci
        L.pf_lowrank_linear_grouped_fwd.argtypes = [ci] + [vp, i64, i64] * 5 + [i64, i64, i64, i64, ci, vp, sz, vp]
        L.pf_lowrank_linear_grouped_bwd.restype = ci
        L.pf_lowrank_linear_grouped_bwd.argtypes = [ci] + [vp, i64, i64] * 8 + [i64, i64, i64, i64, ci, vp, sz, vp]
        L.pf_lowrank_conv_workspace.restype = sz
        L.pf_lowrank_conv_workspace.argtypes = [ci] * 12
        L.pf_lowrank_conv_fwd.restype = ci
        L.pf_lowrank_conv_fwd.argtypes = [vp] * 5 + [ci] * 11 + [vp, sz, vp]
        L.pf_lowrank_conv_bwd.restype = ci
        L.pf_lowrank_conv_bwd.argtypes = [vp] * 8 + [ci] * 11 + [vp, sz, vp]
        L.pf_lowrank_conv_bwd_ex.restype = ci
        L.pf_lowrank_conv_bwd_ex.argtypes = [vp] * 8 + [ci] * 11 + [ctypes.c_uint, vp, sz, vp]
        L.pf_pack_factor_grads.restype = ci
        L.pf_pack_factor_grads.argtypes = [vp, vp, ci, ci, vp, i64, vp, vp, sz, vp]
        L.pf_unpack_factor_grads.restype = ci
        L.pf_unpack_factor_grads.argtypes = [vp, i64, vp, vp, ci, ci, vp, vp, sz, vp]
        _lib = L
    return _lib


def pf_status_string(status: int) -> str:
    return lib().pf_status_string(int(status)).decode()


def pf_version() -> int:
    return int(lib().pf_version())


def pf_launch_count() -> int:
    return int(lib().pf_launch_count())


def pf_last_device_status() -> int:
    return int(lib().pf_last_device_status())


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return PF_BF16
    if t.dtype == torch.float32:
        return PF_F32
    raise TypeError(f"unsupported dtype {t.dtype}")


def _check(st: int, where: str):
    if st != 0:
        raise PfError(st, where)


def _ptr(t):
    return ctypes.c_void_p(t.data_ptr()) if t is not None else ctypes.c_void_p(0)


def _mat(t: torch.Tensor, name: str):
    if not t.is_cuda or t.dim() != 2 or (t.shape[1] > 1 and t.stride(1) != 1):
        raise ValueError(f"{name}: need a 2-D CUDA tensor with unit column stride")
    return t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1])


def _stream(stream):
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


class _Prepared:
    """A C call with its arguments marshalled once; keeps the tensors alive."""
    __slots__ = ("fn", "args", "where", "keep")

    def __init__(self, fn, args, where, keep):
        self.fn, self.args, self.where, self.keep = fn, args, where, keep

    def __call__(self):
        st = self.fn(*self.args)
        if st != 0:
            raise PfError(st, self.where)


def _workspace(nbytes: int, device, workspace, stream=None):
    """The caller's workspace, or a fresh one.  A fresh one is handed back to torch's caching
    allocator as soon as the wrapper returns, while the kernels that use it may still be queued:
    that is safe on torch's current stream (the allocator reuses the block in stream order) and is
    made safe on any other stream by recording that stream on the block."""
    if workspace is not None:
        return workspace
    ws = torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)
    if stream is not None and stream != torch.cuda.current_stream(device):
        ws.record_stream(stream)
    return ws


def pf_lowrank_linear_workspace(m, k, n, r, dtype, is_bwd) -> int:
    return int(lib().pf_lowrank_linear_workspace(m, k, n, r, dtype, int(bool(is_bwd))))


def pf_lowrank_linear_fwd(x, U, V, *, y=None, T_stash=None, want_stash=False, workspace=None,
                          stream=None, prepare=False):
    """y = (x U) V^T.  Returns y, or (y, T_stash) when a stash is requested.
    With prepare=True nothing is launched: returns (call, outputs) where call() issues the
    C call with the arguments marshalled once (fixed buffers and stream)."""
    dt = _dtype_code(x)
    m, k = x.shape
    n, r = V.shape
    if U.shape != (k, r):
        raise ValueError("U must be [k, r] and V [n, r]")
    if y is None:
        y = torch.empty((m, n), dtype=x.dtype, device=x.device)
    if T_stash is None and want_stash:
        T_stash = torch.empty((m, r), dtype=x.dtype, device=x.device)
    ws = _workspace(pf_lowrank_linear_workspace(m, k, n, r, dt, 0), x.device, workspace, stream)
    args = (_ptr(x), _mat(x, "x"), _ptr(U), _mat(U, "U"), _ptr(V), _mat(V, "V"), _ptr(y), _mat(y, "y"),
            _ptr(T_stash), _mat(T_stash, "T_stash") if T_stash is not None else 0,
            m, k, n, r, dt, _ptr(ws), ws.numel(), _stream(stream))
    out = (y, T_stash) if T_stash is not None else y
    if prepare:
        return _Prepared(lib().pf_lowrank_linear_fwd, args, "pf_lowrank_linear_fwd", (x, U, V, y, T_stash, ws)), out
    _check(lib().pf_lowrank_linear_fwd(*args), "pf_lowrank_linear_fwd")
    return out


def pf_lowrank_linear_fwd_act(x, U, V, *, bias=None, act=PF_ACT_NONE, y=None, T_stash=None, want_stash=False,
                              workspace=None, stream=None, prepare=False):
    """y = act((x U) V^T + bias); bias [n] in x's dtype or None, act PF_ACT_NONE / PF_ACT_RELU.
    Otherwise as pf_lowrank_linear_fwd."""
    dt = _dtype_code(x)
    m, k = x.shape
    n, r = V.shape
    if U.shape != (k, r):
        raise ValueError("U must be [k, r] and V [n, r]")
    if bias is not None and (bias.shape != (n,) or bias.dtype != x.dtype or not bias.is_contiguous()):
        raise ValueError("bias must be a contiguous [n] tensor of x's dtype")
    if y is None:
        y = torch.empty((m, n), dtype=x.dtype, device=x.device)
    if T_stash is None and want_stash:
        T_stash = torch.empty((m, r), dtype=x.dtype, device=x.device)
    ws = _workspace(pf_lowrank_linear_workspace(m, k, n, r, dt, 0), x.device, workspace, stream)
    args = (_ptr(x), _mat(x, "x"), _ptr(U), _mat(U, "U"), _ptr(V), _mat(V, "V"), _ptr(bias), int(act),
            _ptr(y), _mat(y, "y"), _ptr(T_stash), _mat(T_stash, "T_stash") if T_stash is not None else 0,
            m, k, n, r, dt, _ptr(ws), ws.numel(), _stream(stream))
    out = (y, T_stash) if T_stash is not None else y
    if prepare:
        return _Prepared(lib().pf_lowrank_linear_fwd_act, args, "pf_lowrank_linear_fwd_act",
                         (x, U, V, bias, y, T_stash, ws)), out
    _check(lib().pf_lowrank_linear_fwd_act(*args), "pf_lowrank_linear_fwd_act")
    return out


def pf_bias_act_bwd(y, dY, *, act=PF_ACT_RELU, want_dbias=True, dbias=None, workspace=None, stream=None):
    """Backward of y = act(z + bias): dY [m, n] becomes dZ IN PLACE (zeroed where y <= 0 for PF_ACT_RELU);
    returns dbias [n] (column sums of dZ) or None."""
    dt = _dtype_code(dY)
    m, n = dY.shape
    if dbias is None and want_dbias:
        dbias = torch.empty((n,), dtype=dY.dtype, device=dY.device)
    need = int(lib().pf_bias_act_bwd_workspace(m, n)) if dbias is not None else 0
    ws = _workspace(need, dY.device, workspace, stream)
    st = lib().pf_bias_act_bwd(_ptr(y), _mat(y, "y") if y is not None else 0, _ptr(dY), _mat(dY, "dY"), _ptr(dbias),
                               m, n, int(act), dt, _ptr(ws), ws.numel(), _stream(stream))
    _check(st, "pf_bias_act_bwd")
    return dbias


def pf_static_scratch_bytes() -> int:
    return int(lib().pf_static_scratch_bytes())


def pf_lowrank_linear_fwd_static(x, U, V, *, y, T_stash=None, stream=None):
    """y = (x U) V^T for callers that cannot allocate: the scratch is a fixed array inside the
    library, so the caller passes inputs and outputs only (y is required; nothing is allocated
    here either).  Raises PfError(PF_ERR_WORKSPACE) when the problem does not fit the array.
    Calls on one device share that array: do not let two of them overlap on the GPU."""
    dt = _dtype_code(x)
    m, k = x.shape
    n, r = V.shape
    if U.shape != (k, r):
        raise ValueError("U must be [k, r] and V [n, r]")
    st = lib().pf_lowrank_linear_fwd_static(
        _ptr(x), _mat(x, "x"), _ptr(U), _mat(U, "U"), _ptr(V), _mat(V, "V"), _ptr(y), _mat(y, "y"),
        _ptr(T_stash), _mat(T_stash, "T_stash") if T_stash is not None else 0,
        m, k, n, r, dt, _stream(stream))
    _check(st, "pf_lowrank_linear_fwd_static")
    return (y, T_stash) if T_stash is not None else y


def pf_lowrank_linear_bwd(x, U, V, dY, *, T_stash=None, need_dX=True, dX=None, dU=None, dV=None,
                          accumulate=False, grads_f32=False, workspace=None, stream=None, prepare=False):
    """Returns (dX or None, dU, dV) for upstream gradient dY (prepare: see the forward).
    accumulate: dU and dV (required then) are added to; grads_f32: dU and dV are fp32 tensors."""
    dt = _dtype_code(x)
    m, k = x.shape
    n, r = V.shape
    flags = (PF_GRAD_ACCUMULATE if accumulate else 0) | (PF_GRAD_F32 if grads_f32 else 0)
    gdt = torch.float32 if grads_f32 else x.dtype
    if accumulate and (dU is None or dV is None):
        raise ValueError("accumulate=True needs the dU and dV to add to")
    if dX is None and need_dX:
        dX = torch.empty((m, k), dtype=x.dtype, device=x.device)
    if dU is None:
        dU = torch.empty((k, r), dtype=gdt, device=x.device)
    if dV is None:
        dV = torch.empty((n, r), dtype=gdt, device=x.device)
    if dU.dtype != gdt or dV.dtype != gdt:
        raise ValueError("dU and dV must be float32 with grads_f32=True and of x's dtype otherwise")
    ws = _workspace(pf_lowrank_linear_workspace(m, k, n, r, dt, 1), x.device, workspace, stream)
    args = (_ptr(x), _mat(x, "x"), _ptr(U), _mat(U, "U"), _ptr(V), _mat(V, "V"), _ptr(dY), _mat(dY, "dY"),
            _ptr(T_stash), _mat(T_stash, "T_stash") if T_stash is not None else 0,
            _ptr(dX), _mat(dX, "dX") if dX is not None else 0, _ptr(dU), _mat(dU, "dU"),
            _ptr(dV), _mat(dV, "dV"), m, k, n, r, dt, _ptr(ws), ws.numel(), _stream(stream))
    if flags:
        args = args[:21] + (flags,) + args[21:]
        if prepare:
            return _Prepared(lib().pf_lowrank_linear_bwd_ex, args, "pf_lowrank_linear_bwd_ex",
                             (x, U, V, dY, T_stash, dX, dU, dV, ws)), (dX, dU, dV)
        _check(lib().pf_lowrank_linear_bwd_ex(*args), "pf_lowrank_linear_bwd_ex")
        return dX, dU, dV
    if prepare:
        return _Prepared(lib().pf_lowrank_linear_bwd, args, "pf_lowrank_linear_bwd",
                         (x, U, V, dY, T_stash, dX, dU, dV, ws)), (dX, dU, dV)
    _check(lib().pf_lowrank_linear_bwd(*args), "pf_lowrank_linear_bwd")
    return dX, dU, dV


def pf_lowrank_linear_grouped_workspace(groups, m, k, n, r, dtype, is_bwd) -> int:
    return int(lib().pf_lowrank_linear_grouped_workspace(groups, m, k, n, r, dtype, int(bool(is_bwd))))


def _grp(t: torch.Tensor, name: str, groups: int, may_share: bool = False):
    """(pointer, row pitch, group stride) of a [groups, rows, cols] tensor (unit column stride), or of
    a 2-D [rows, cols] tensor shared by all groups (stride 0) where that is allowed."""
    if t is None:
        return ctypes.c_void_p(0), 0, 0
    if t.dim() == 2 and may_share:
        return _ptr(t), _mat(t, name), 0
    if not t.is_cuda or t.dim() != 3 or t.shape[0] != groups or (t.shape[2] > 1 and t.stride(2) != 1):
        raise ValueError(f"{name}: need a CUDA tensor [groups, rows, cols] with unit column stride")
    ld = t.stride(1) if t.shape[1] > 1 else max(t.stride(1), t.shape[2])
    return _ptr(t), ld, t.stride(0)


def pf_lowrank_linear_grouped_fwd(x, U, V, *, y=None, T_stash=None, want_stash=False, workspace=None,
                                  stream=None, prepare=False):
    """y[g] = (x[g] U[g]) V[g]^T for U [G, k, r], V [G, n, r] and x [G, m, k] or one shared x [m, k].
    Returns y [G, m, n], or (y, T_stash [G, m, r]) when a stash is requested."""
    dt = _dtype_code(U)
    G, k, r = U.shape
    n = V.shape[1]
    m = x.shape[-2]
    if V.shape != (G, n, r) or x.shape[-1] != k:
        raise ValueError("U must be [G, k, r], V [G, n, r], x [G, m, k] or [m, k]")
    if y is None:
        y = torch.empty((G, m, n), dtype=U.dtype, device=U.device)
    if T_stash is None and want_stash:
        T_stash = torch.empty((G, m, r), dtype=U.dtype, device=U.device)
    ws = _workspace(pf_lowrank_linear_grouped_workspace(G, m, k, n, r, dt, 0), U.device, workspace, stream)
    args = (G, *_grp(x, "x", G, True), *_grp(U, "U", G), *_grp(V, "V", G), *_grp(y, "y", G), *_grp(T_stash, "T_stash", G),
            m, k, n, r, dt, _ptr(ws), ws.numel(), _stream(stream))
    out = (y, T_stash) if T_stash is not None else y
    if prepare:
        return _Prepared(lib().pf_lowrank_linear_grouped_fwd, args, "pf_lowrank_linear_grouped_fwd",
                         (x, U, V, y, T_stash, ws)), out
    _check(lib().pf_lowrank_linear_grouped_fwd(*args), "pf_lowrank_linear_grouped_fwd")
    return out


def pf_lowrank_linear_grouped_bwd(x, U, V, dY, *, T_stash=None, need_dX=True, dX=None, dU=None, dV=None,
                                  workspace=None, stream=None, prepare=False):
    """Returns (dX or None, dU [G, k, r], dV [G, n, r]).  dX is [G, m, k] when every group has its own
    x and ONE [m, k] matrix (the sum over the groups) when x [m, k] is shared."""
    dt = _dtype_code(U)
    G, k, r = U.shape
    n = V.shape[1]
    m = x.shape[-2]
    shared = x.dim() == 2
    if dX is None and need_dX:
        dX = torch.empty((m, k) if shared else (G, m, k), dtype=U.dtype, device=U.device)
    if dU is None:
        dU = torch.empty_like(U)
    if dV is None:
        dV = torch.empty_like(V)
    ws = _workspace(pf_lowrank_linear_grouped_workspace(G, m, k, n, r, dt, 1), U.device, workspace, stream)
    args = (G, *_grp(x, "x", G, True), *_grp(U, "U", G), *_grp(V, "V", G), *_grp(dY, "dY", G), *_grp(T_stash, "T_stash", G),
            *_grp(dX, "dX", G, True), *_grp(dU, "dU", G), *_grp(dV, "dV", G),
            m, k, n, r, dt, _ptr(ws), ws.numel(), _stream(stream))
    if prepare:
        return _Prepared(lib().pf_lowrank_linear_grouped_bwd, args, "pf_lowrank_linear_grouped_bwd",
                         (x, U, V, dY, T_stash, dX, dU, dV, ws)), (dX, dU, dV)
    _check(lib().pf_lowrank_linear_grouped_bwd(*args), "pf_lowrank_linear_grouped_bwd")
    return dX, dU, dV


def pf_lowrank_conv_workspace(N, H, W, C, R, O, kh, kw, stride, pad, dtype, is_bwd) -> int:
    return int(lib().pf_lowrank_conv_workspace(N, H, W, C, R, O, kh, kw, stride, pad, dtype,
                                               int(bool(is_bwd))))


def _conv_dims(x, U, V, stride, pad):
    for t, nm in ((x, "x"), (U, "U"), (V, "V")):
        if not t.is_cuda or not t.is_contiguous():
            raise ValueError(f"{nm}: need a contiguous CUDA tensor")
    N, H, W, C = x.shape
    kh, kw, C2, R = U.shape
    O, R2 = V.shape
    if C2 != C or R2 != R:
        raise ValueError("U must be [kh, kw, C, R] and V [O, R]")
    Ho = (H + 2 * pad - kh) // stride + 1
    Wo = (W + 2 * pad - kw) // stride + 1
    return N, H, W, C, R, O, kh, kw, Ho, Wo


def pf_lowrank_conv_fwd(x, U, V, *, stride=1, pad=1, y=None, T_stash=None, want_stash=False,
                        workspace=None, stream=None, prepare=False):
    """NHWC factorized convolution.  Returns y, or (y, T_stash) when a stash is requested."""
    dt = _dtype_code(x)
    N, H, W, C, R, O, kh, kw, Ho, Wo = _conv_dims(x, U, V, stride, pad)
    if y is None:
        y = torch.empty((N, Ho, Wo, O), dtype=x.dtype, device=x.device)
    if T_stash is None and want_stash:
        T_stash = torch.empty((N, Ho, Wo, R), dtype=x.dtype, device=x.device)
    ws = _workspace(pf_lowrank_conv_workspace(N, H, W, C, R, O, kh, kw, stride, pad, dt, 0),
                    x.device, workspace, stream)
    args = (_ptr(x), _ptr(U), _ptr(V), _ptr(y), _ptr(T_stash), N, H, W, C, R, O, kh, kw, stride, pad,
            dt, _ptr(ws), ws.numel(), _stream(stream))
    out = (y, T_stash) if T_stash is not None else y
    if prepare:
        return _Prepared(lib().pf_lowrank_conv_fwd, args, "pf_lowrank_conv_fwd", (x, U, V, y, T_stash, ws)), out
    _check(lib().pf_lowrank_conv_fwd(*args), "pf_lowrank_conv_fwd")
    return out


def pf_lowrank_conv_bwd(x, U, V, dY, *, stride=1, pad=1, T_stash=None, need_dX=True, dX=None,
                        dU=None, dV=None, accumulate=False, grads_f32=False, workspace=None, stream=None,
                        prepare=False):
    """Returns (dX or None, dU, dV) for upstream gradient dY [N, Ho, Wo, O].
    accumulate / grads_f32: as in pf_lowrank_linear_bwd."""
    dt = _dtype_code(x)
    N, H, W, C, R, O, kh, kw, Ho, Wo = _conv_dims(x, U, V, stride, pad)
    if not dY.is_contiguous() or tuple(dY.shape) != (N, Ho, Wo, O):
        raise ValueError("dY must be contiguous [N, Ho, Wo, O]")
    if dX is None and need_dX:
        dX = torch.empty_like(x)
    flags = (PF_GRAD_ACCUMULATE if accumulate else 0) | (PF_GRAD_F32 if grads_f32 else 0)
    gdt = torch.float32 if grads_f32 else x.dtype
    if accumulate and (dU is None or dV is None):
        raise ValueError("accumulate=True needs the dU and dV to add to")
    if dU is None:
        dU = torch.empty(U.shape, dtype=gdt, device=x.device)
    if dV is None:
        dV = torch.empty(V.shape, dtype=gdt, device=x.device)
    if dU.dtype != gdt or dV.dtype != gdt or not dU.is_contiguous() or not dV.is_contiguous():
        raise ValueError("dU and dV must be contiguous, float32 with grads_f32=True and of x's dtype otherwise")
    ws = _workspace(pf_lowrank_conv_workspace(N, H, W, C, R, O, kh, kw, stride, pad, dt, 1),
                    x.device, workspace, stream)
    args = (_ptr(x), _ptr(U), _ptr(V), _ptr(dY), _ptr(T_stash), _ptr(dX), _ptr(dU), _ptr(dV),
            N, H, W, C, R, O, kh, kw, stride, pad, dt, _ptr(ws), ws.numel(), _stream(stream))
    if flags:
        args = args[:19] + (flags,) + args[19:]
        if prepare:
            return _Prepared(lib().pf_lowrank_conv_bwd_ex, args, "pf_lowrank_conv_bwd_ex",
                             (x, U, V, dY, T_stash, dX, dU, dV, ws)), (dX, dU, dV)
        _check(lib().pf_lowrank_conv_bwd_ex(*args), "pf_lowrank_conv_bwd_ex")
        return dX, dU, dV
    if prepare:
        return _Prepared(lib().pf_lowrank_conv_bwd, args, "pf_lowrank_conv_bwd",
                         (x, U, V, dY, T_stash, dX, dU, dV, ws)), (dX, dU, dV)
    _check(lib().pf_lowrank_conv_bwd(*args), "pf_lowrank_conv_bwd")
    return dX, dU, dV


def pf_pack_factor_grads(grads, *, flat=None, stream=None, prepare=False):
    """Copies the tensors of `grads`, in order and tightly, into one flat buffer.
    Returns (flat, offsets) with offsets a python list of count+1 element offsets."""
    count = len(grads)
    if count == 0:
        offs = (ctypes.c_int64 * 1)()
        st = lib().pf_pack_factor_grads(None, None, 0, PF_BF16, _ptr(flat),
                                        flat.numel() if flat is not None else 0, offs, None, 0,
                                        _stream(stream))
        _check(st, "pf_pack_factor_grads")
        return flat, [0]
    dt = _dtype_code(grads[0])
    for g in grads:
        if not g.is_cuda or not g.is_contiguous() or g.dtype != grads[0].dtype:
            raise ValueError("grads: contiguous CUDA tensors of one dtype")
    numels = (ctypes.c_int64 * count)(*[g.numel() for g in grads])
    ptrs = (ctypes.c_void_p * count)(*[g.data_ptr() for g in grads])
    offs = (ctypes.c_int64 * (count + 1))()
    if flat is None:
        flat = torch.empty(sum(g.numel() for g in grads), dtype=grads[0].dtype,
                           device=grads[0].device)
    args = (ptrs, numels, count, dt, _ptr(flat), flat.numel(), offs, None, 0, _stream(stream))
    if prepare:
        return _Prepared(lib().pf_pack_factor_grads, args, "pf_pack_factor_grads",
                         (list(grads), flat)), (flat, offs)
    _check(lib().pf_pack_factor_grads(*args), "pf_pack_factor_grads")
    return flat, list(offs)


def pf_unpack_factor_grads(flat, grads, *, stream=None):
    """The inverse of pf_pack_factor_grads: tensor i of `grads` (contiguous CUDA tensors of flat's
    dtype, overwritten) receives its slice of `flat`.  Returns the list of count+1 element offsets."""
    count = len(grads)
    offs = (ctypes.c_int64 * (count + 1))()
    if count == 0:
        _check(lib().pf_unpack_factor_grads(_ptr(flat), flat.numel(), None, None, 0, _dtype_code(flat), offs, None, 0,
                                            _stream(stream)), "pf_unpack_factor_grads")
        return [0]
    for g in grads:
        if not g.is_cuda or not g.is_contiguous() or g.dtype != flat.dtype:
            raise ValueError("grads: contiguous CUDA tensors of flat's dtype")
    numels = (ctypes.c_int64 * count)(*[g.numel() for g in grads])
    ptrs = (ctypes.c_void_p * count)(*[g.data_ptr() for g in grads])
    _check(lib().pf_unpack_factor_grads(_ptr(flat), flat.numel(), ptrs, numels, count, _dtype_code(flat), offs, None, 0,
                                        _stream(stream)), "pf_unpack_factor_grads")
    return list(offs)
