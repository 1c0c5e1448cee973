"""ctypes binding of the libcott C ABI: argument marshalling only.

Function names and argument order follow ``include/cott.h``.  Tensors are torch CUDA
tensors (contiguous ``[B,H,N,d]``, float32 or bfloat16); outputs and the workspace are
allocated here with torch because the library itself never allocates.
"""
from __future__ import annotations

import contextlib
import ctypes
import functools
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libcott.so")
_lib = None

OP_FWD, OP_BWD, OP_DECODE = 0, 1, 2
F32, BF16 = 0, 1
_SIZE_MAX = ctypes.c_size_t(-1).value


class CottError(RuntimeError):
    """A libcott call returned a non-zero status."""

    def __init__(self, status: int, where: str):
        lib = _load()
        msg = lib.cott_status_string(status).decode()
        cuda = lib.cott_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} ({status})" + (f" [{cuda}]" if status == -4 and cuda else ""))
        self.status = status


class _ScaleParams(ctypes.Structure):
    _fields_ = [("m", ctypes.c_void_p), ("seq_len", ctypes.c_void_p), ("seq_len_scalar", ctypes.c_float)]


def library_path() -> str:
    return _LIB_PATH


def _load():
    """Loads libcott.so; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2409_18747_b200._build` "
            "(libcott has no CPU or PyTorch fallback)")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, ci, cs = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    lib.cott_version.restype = ci
    lib.cott_status_string.restype = ctypes.c_char_p
    lib.cott_status_string.argtypes = [ci]
    lib.cott_last_cuda_error.restype = ctypes.c_char_p
    lib.cott_launch_count.restype = ctypes.c_ulonglong
    lib.cott_profile_enable.restype = ci
    lib.cott_profile_enable.argtypes = [ci]
    lib.cott_profile_read.restype = ci
    lib.cott_profile_read.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ci), ci]
    lib.cott_workspace_bytes.restype = cs
    lib.cott_workspace_bytes.argtypes = [ci, ci, ci, ci, ci, ci, ci]
    lib.cott_query_plan.restype = ci
    lib.cott_query_plan.argtypes = [ci] * 7 + [ctypes.POINTER(ci)] * 3
    lib.cott_workspace_bytes_dkdv.restype = cs
    lib.cott_workspace_bytes_dkdv.argtypes = [ci] * 8
    lib.cott_workspace_bytes_varlen.restype = cs
    lib.cott_workspace_bytes_varlen.argtypes = [ci] * 8
    lib.cott_query_plan_dkdv.restype = ci
    lib.cott_query_plan_dkdv.argtypes = [ci] * 8 + [ctypes.POINTER(ci)] * 4
    lib.cott_fwd_dkdv.restype = ci
    lib.cott_fwd_dkdv.argtypes = [vp] * 6 + [ci] * 7 + [vp, vp, vp, ctypes.POINTER(_ScaleParams), vp, cs, vp]
    lib.cott_bwd_dkdv.restype = ci
    lib.cott_bwd_dkdv.argtypes = [vp] * 8 + [ci] * 7 + [vp] * 5 + [ctypes.POINTER(_ScaleParams), vp, cs, vp]
    lib.cott_decode_step_dkdv.restype = ci
    lib.cott_decode_step_dkdv.argtypes = [vp] * 5 + [ci] * 5 + [ctypes.POINTER(_ScaleParams), vp]
    lib.cott_fwd.restype = ci
    lib.cott_fwd.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci,
                             ctypes.POINTER(_ScaleParams), vp, cs, vp]
    lib.cott_fwd_strided.restype = ci
    lib.cott_fwd_strided.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, vp, vp,
                                     ctypes.POINTER(_ScaleParams), vp, cs, vp]
    lib.cott_bwd_strided.restype = ci
    lib.cott_bwd_strided.argtypes = [vp] * 8 + [ci, ci, ci, ci, ci, ci, vp, vp, vp,
                                                 ctypes.POINTER(_ScaleParams), vp, cs, vp]
    lib.cott_bwd_after_fwd.restype = ci
    lib.cott_bwd_after_fwd.argtypes = [vp] * 8 + [ci, ci, ci, ci, ci, ci, vp, vp, vp,
                                                   ctypes.POINTER(_ScaleParams), vp, vp, cs, vp]
    lib.cott_fwd_varlen.restype = ci
    lib.cott_fwd_varlen.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci,
                                    ctypes.POINTER(_ScaleParams), vp, cs, vp]
    lib.cott_bwd_varlen.restype = ci
    lib.cott_bwd_varlen.argtypes = [vp] * 9 + [ci, ci, ci, ci, ci, ci, ci,
                                                ctypes.POINTER(_ScaleParams), vp, cs, vp]
    lib.cott_fwd_stateful_strided.restype = ci
    lib.cott_fwd_stateful_strided.argtypes = [vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, vp, vp,
                                              ctypes.POINTER(_ScaleParams), vp, cs, vp]
    lib.cott_bwd_stateful.restype = ci
    lib.cott_bwd_stateful.argtypes = [vp] * 11 + [ci] * 6 + [ctypes.POINTER(_ScaleParams), vp, cs, vp]
    lib.cott_bwd_stateful_strided.restype = ci
    lib.cott_bwd_stateful_strided.argtypes = [vp] * 11 + [ci] * 6 + [vp] * 5 + [ctypes.POINTER(_ScaleParams), vp, cs, vp]
    lib.cott_fwd_stateful.restype = ci
    lib.cott_fwd_stateful.argtypes = [vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci,
                                      ctypes.POINTER(_ScaleParams), vp, cs, vp]
    lib.cott_bwd.restype = ci
    lib.cott_bwd.argtypes = [vp] * 8 + [ci, ci, ci, ci, ci, ci, ctypes.POINTER(_ScaleParams), vp, cs, vp]
    lib.cott_decode_step.restype = ci
    lib.cott_decode_step.argtypes = [vp] * 5 + [ci, ci, ci, ci, ctypes.POINTER(_ScaleParams), vp]
    lib.cott_host_step_arena_bytes.restype = cs
    lib.cott_host_step_arena_bytes.argtypes = [ci] * 6
    lib.cott_host_step_slicing.restype = ci
    lib.cott_host_step_slicing.argtypes = [ci, ci, ctypes.POINTER(ci), ctypes.POINTER(ci), ctypes.POINTER(ci)]
    lib.cott_fwd_bwd_host.restype = ci
    lib.cott_fwd_bwd_host.argtypes = [vp] * 11 + [ci] * 6 + [vp, cs, vp]
    lib.cott_fwd_noalloc_max_bytes.restype = cs
    lib.cott_fwd_noalloc.restype = ci
    lib.cott_fwd_noalloc.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ctypes.POINTER(_ScaleParams), vp]
    lib.cott_last_async_status.restype = ci
    lib.cott_last_async_status.argtypes = [vp, vp]
    lib.cott_fwd_noalloc_status.restype = ci
    lib.cott_fwd_noalloc_status.argtypes = [vp]
    lib.cott_shutdown.restype = ci
    lib.cott_set_option.restype = ci
    lib.cott_set_option.argtypes = [ctypes.c_char_p, ctypes.c_longlong]
    lib.cott_get_option.restype = ctypes.c_longlong
    lib.cott_get_option.argtypes = [ctypes.c_char_p]
    _lib = lib
    return lib


def _on_call_stream(fn):
    """Runs a binding call with its ``stream`` argument (if any) as torch's current stream, so
    that every tensor the binding allocates (outputs, workspace) belongs to the stream the
    kernels run on: the caching allocator then cannot hand such a block to work on another
    stream while libcott kernels still use it."""
    @functools.wraps(fn)
    def wrapped(*args, **kwargs):
        stream = kwargs.get("stream")
        ctx = torch.cuda.stream(stream) if stream is not None else contextlib.nullcontext()
        with ctx:
            return fn(*args, **kwargs)
    return wrapped


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"libcott supports float32 and bfloat16 I/O, got {t.dtype}")


def _check_dev(*ts):
    for t in ts:
        if t is None:
            continue
        if not t.is_cuda:
            raise RuntimeError("libcott needs CUDA tensors (there is no CPU path)")
        if not t.is_contiguous():
            raise ValueError("libcott needs contiguous tensors")


class _Strides(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_longlong), ("head", ctypes.c_longlong), ("token", ctypes.c_longlong)]


def _check_rows(*ts):
    """[B,H,N,d] CUDA tensors with contiguous rows; any strides over batch, head and token."""
    for t in ts:
        if not t.is_cuda:
            raise RuntimeError("libcott needs CUDA tensors (there is no CPU path)")
        if t.dim() != 4 or (t.shape[3] > 1 and t.stride(3) != 1):
            raise ValueError("libcott needs [B,H,N,d] tensors whose last dimension is contiguous")


def _strides_of(*ts):
    """ctypes strides shared by the given tensors (None when they are dense [B,H,N,d])."""
    st = tuple(ts[0].stride()[:3])
    for t in ts[1:]:
        if tuple(t.stride()[:3]) != st:
            raise ValueError("tensors of one group (q,k,v / dq,dk,dv) must share their strides")
    if all(t.is_contiguous() for t in ts):
        return None
    return _Strides(st[0], st[1], st[2])


def _ref(s):
    return ctypes.byref(s) if s is not None else None


def _stream_ptr(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return int(s.cuda_stream)


def _scale(m: torch.Tensor, seq_len, scalar: float = 0.0) -> _ScaleParams:
    sp = _ScaleParams()
    sp.m = m.data_ptr()
    sp.seq_len = seq_len.data_ptr() if isinstance(seq_len, torch.Tensor) else None
    sp.seq_len_scalar = float(seq_len) if (seq_len is not None and not isinstance(seq_len, torch.Tensor)) else scalar
    return sp


def fwd_noalloc_status(stream=None) -> int:
    """cott_fwd_noalloc_status: synchronises the stream and returns the status the last
    ``fwd_noalloc`` call left (0, or -5 after a device-side wait gave up)."""
    return int(_load().cott_fwd_noalloc_status(_stream_ptr(stream)))


def shutdown() -> None:
    """cott_shutdown: destroys the streams and events the library created for this thread."""
    rc = _load().cott_shutdown()
    if rc != 0:
        raise CottError(rc, "cott_shutdown")


def set_option(name: str, value: int) -> None:
    """cott_set_option: a process-wide switch for tests and measurements (see ``cott.h``)."""
    rc = _load().cott_set_option(name.encode(), int(value))
    if rc != 0:
        raise CottError(rc, f"cott_set_option({name})")


def get_option(name: str) -> int:
    return int(_load().cott_get_option(name.encode()))


def workspace_bytes(op: int, dt: int, B: int, H: int, N: int, d: int, causal: bool) -> int:
    n = _load().cott_workspace_bytes(op, dt, B, H, N, d, int(bool(causal)))
    if n == _SIZE_MAX:
        raise CottError(-2, "cott_workspace_bytes")
    return int(n)


def query_plan(op: int, dt: int, B: int, H: int, N: int, d: int, causal: bool) -> dict:
    path, group, chunk = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
    rc = _load().cott_query_plan(op, dt, B, H, N, d, int(bool(causal)), ctypes.byref(path),
                                 ctypes.byref(group), ctypes.byref(chunk))
    if rc != 0:
        raise CottError(rc, "cott_query_plan")
    return {"path": path.value, "group": group.value, "chunk": chunk.value}


def workspace_bytes_dkdv(op: int, dt: int, B: int, H: int, N: int, d_k: int, d_v: int, causal: bool) -> int:
    n = _load().cott_workspace_bytes_dkdv(op, dt, B, H, N, d_k, d_v, int(bool(causal)))
    if n == _SIZE_MAX:
        raise CottError(-2, "cott_workspace_bytes_dkdv")
    return int(n)


def query_plan_dkdv(op: int, dt: int, B: int, H: int, N: int, d_k: int, d_v: int, causal: bool) -> dict:
    path, group, chunk, kd = ctypes.c_int(), ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
    rc = _load().cott_query_plan_dkdv(op, dt, B, H, N, d_k, d_v, int(bool(causal)), ctypes.byref(path),
                                      ctypes.byref(group), ctypes.byref(chunk), ctypes.byref(kd))
    if rc != 0:
        raise CottError(rc, "cott_query_plan_dkdv")
    return {"path": path.value, "group": group.value, "chunk": chunk.value, "kernel_d": kd.value}


def _fwd_dkdv(q, k, v, m, seq_len, causal, state_in, return_state, out, workspace, stream):
    """cott_fwd_dkdv: q, k ``[B,H,N,d_k]``, v ``[B,H,N,d_v]``; states ``[B,H,d_k,d_v]``."""
    _check_rows(q, k, v)
    _check_dev(m, state_in, seq_len if isinstance(seq_len, torch.Tensor) else None)
    B, H, N, dk = q.shape
    dv = v.shape[3]
    dt = _dt(q)
    if state_in is not None and (state_in.dtype != torch.float32 or tuple(state_in.shape) != (B, H, dk, dv)):
        raise ValueError("state_in must be float32 [B,H,d_k,d_v]")
    o = torch.empty_like(v) if out is None else out
    _check_rows(o)
    s_qk, s_v, s_o = _strides_of(q, k), _strides_of(v), _strides_of(o)
    state = torch.empty((B, H, dk, dv), dtype=torch.float32, device=q.device) if return_state else None
    need = workspace_bytes_dkdv(OP_FWD, dt, B, H, N, dk, dv, causal)
    ws = torch.empty(max(need, 256), dtype=torch.uint8, device=q.device) if workspace is None else workspace
    sp = _scale(m, seq_len)
    rc = _load().cott_fwd_dkdv(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(),
                               state_in.data_ptr() if state_in is not None else None,
                               state.data_ptr() if state is not None else None, B, H, N, dk, dv,
                               int(bool(causal)), dt, _ref(s_qk), _ref(s_v), _ref(s_o), ctypes.byref(sp),
                               ws.data_ptr(), ws.numel(), _stream_ptr(stream))
    if rc != 0:
        raise CottError(rc, "cott_fwd_dkdv")
    return (o, state) if return_state else o


def _workspace(op, dt, B, H, N, d, causal, device, workspace):
    need = workspace_bytes(op, dt, B, H, N, d, causal)
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=device)
    return workspace, workspace.numel()


def workspace_bytes_varlen(op, dt, B, H, total_tokens, max_seqlen, d, causal=True) -> int:
    """cott_workspace_bytes_varlen: the workspace of a packed batch with room for groups sized by the
    total token count."""
    n = int(_load().cott_workspace_bytes_varlen(op, dt, B, H, int(total_tokens), int(max_seqlen), d, int(bool(causal))))
    if n == _SIZE_MAX:
        raise CottError(-2, "cott_workspace_bytes_varlen")
    return n


def _workspace_varlen(op, dt, B, H, T, max_seqlen, d, causal, device, workspace):
    if workspace is None:
        workspace = torch.empty(max(workspace_bytes_varlen(op, dt, B, H, T, max_seqlen, d, causal), 256),
                                dtype=torch.uint8, device=device)
    return workspace, workspace.numel()


@_on_call_stream
def fwd(q, k, v, m, seq_len=None, causal=True, return_state=False, out=None, workspace=None,
        stream=None):
    """cott_fwd / cott_fwd_strided.  q, k, v: ``[B,H,N,d]`` tensors with contiguous rows and
    common strides -- dense, a ``[B,N,H,d]`` buffer seen through ``permute(0,2,1,3)``, or the
    slices of a fused projection output; no copy is made.  ``seq_len``: None (s_b = N), a float,
    or a float32 ``[B]`` CUDA tensor.  Returns ``o`` (laid out like q when q is dense in
    memory, else dense ``[B,H,N,d]``; or ``out``) or ``(o, state[B,H,d,d] fp32)``."""
    if v.shape[-1] != q.shape[-1]:      # different key and value sizes
        return _fwd_dkdv(q, k, v, m, seq_len, causal, None, return_state, out, workspace, stream)
    _check_rows(q, k, v)
    _check_dev(m, seq_len if isinstance(seq_len, torch.Tensor) else None)
    B, H, N, d = q.shape
    dt = _dt(q)
    o = torch.empty_like(q) if out is None else out
    _check_rows(o)
    s_qkv, s_o = _strides_of(q, k, v), _strides_of(o)
    state = torch.empty((B, H, d, d), dtype=torch.float32, device=q.device) if return_state else None
    ws, ws_bytes = _workspace(OP_FWD, dt, B, H, N, d, causal, q.device, workspace)
    sp = _scale(m, seq_len)
    rc = _load().cott_fwd_strided(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(),
                                  state.data_ptr() if state is not None else None, B, H, N, d,
                                  int(bool(causal)), dt, _ref(s_qkv), _ref(s_o), ctypes.byref(sp),
                                  ws.data_ptr(), ws_bytes, _stream_ptr(stream))
    if rc != 0:
        raise CottError(rc, "cott_fwd_strided")
    return (o, state) if return_state else o


@_on_call_stream
def fwd_stateful(q, k, v, m, seq_len, state_in=None, return_state=True, out=None, workspace=None,
                 stream=None):
    """cott_fwd_stateful: causal forward over one segment of a longer sequence.  ``state_in``
    (fp32 ``[B,H,d,d]`` or None) is the state the previous segment (or a decode step) left;
    ``seq_len`` (a float >= 1 or a float32 ``[B]`` CUDA tensor) is the scaling base of the WHOLE
    sequence and must be the same for all its segments.  Returns ``(o, state)`` or ``o``."""
    _check_rows(q, k, v)
    _check_dev(m, state_in, seq_len if isinstance(seq_len, torch.Tensor) else None)
    if seq_len is None:
        raise ValueError("fwd_stateful needs the scaling base of the whole sequence")
    if v.shape[-1] != q.shape[-1]:      # different key and value sizes
        if state_in is None:
            raise ValueError("with different key and value sizes a segment without a state is a plain fwd call")
        return _fwd_dkdv(q, k, v, m, seq_len, True, state_in, return_state, out, workspace, stream)
    B, H, N, d = q.shape
    dt = _dt(q)
    if state_in is not None and (state_in.dtype != torch.float32 or tuple(state_in.shape) != (B, H, d, d)):
        raise ValueError("state_in must be float32 [B,H,d,d]")
    o = torch.empty_like(q) if out is None else out
    state = torch.empty((B, H, d, d), dtype=torch.float32, device=q.device) if return_state else None
    _check_rows(o)
    s_qkv, s_o = _strides_of(q, k, v), _strides_of(o)
    ws, ws_bytes = _workspace(OP_FWD, dt, B, H, N, d, True, q.device, workspace)
    sp = _scale(m, seq_len)
    rc = _load().cott_fwd_stateful_strided(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(),
                                           state_in.data_ptr() if state_in is not None else None,
                                           state.data_ptr() if state is not None else None, B, H, N, d, dt,
                                           _ref(s_qkv), _ref(s_o), ctypes.byref(sp), ws.data_ptr(), ws_bytes,
                                           _stream_ptr(stream))
    if rc != 0:
        raise CottError(rc, "cott_fwd_stateful_strided")
    return (o, state) if return_state else o


@_on_call_stream
def fwd_noalloc(q, k, v, m, seq_len=None, causal=True, out=None, stream=None):
    """cott_fwd_noalloc: the forward pass on the library's built-in 8 MiB scratch, for callers
    that cannot supply a workspace.  Raises CottError(-3) when the problem needs more."""
    _check_dev(q, k, v, m, seq_len if isinstance(seq_len, torch.Tensor) else None)
    B, H, N, d = q.shape
    o = torch.empty_like(q) if out is None else out
    sp = _scale(m, seq_len)
    rc = _load().cott_fwd_noalloc(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), B, H, N, d,
                                  int(bool(causal)), _dt(q), ctypes.byref(sp), _stream_ptr(stream))
    if rc != 0:
        raise CottError(rc, "cott_fwd_noalloc")
    return o


@_on_call_stream
def bwd(q, k, v, d_o, m, seq_len=None, causal=True, workspace=None, stream=None, out=None, fwd_workspace=None):
    """cott_bwd / cott_bwd_strided; with ``fwd_workspace`` (the workspace tensor the forward call
    on the same q, k, v used, untouched since) cott_bwd_after_fwd, which reuses what that call
    left there.  q, k, v (common strides) and d_o as for ``fwd``; ``out``:
    optional ``(dq, dk, dv)`` tensors with common strides (e.g. the slices of a fused gradient
    buffer), else they are allocated like q.  Returns ``(dq, dk, dv, dm[H] fp32)``."""
    _check_rows(q, k, v, d_o)
    _check_dev(m, seq_len if isinstance(seq_len, torch.Tensor) else None)
    B, H, N, d = q.shape
    dt = _dt(q)
    if v.shape[-1] != d:                # different key and value sizes: cott_bwd_dkdv
        d_v = v.shape[-1]
        dq, dk, dv = (torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)) if out is None else out
        _check_rows(dq, dk, dv)
        dm = torch.empty((H,), dtype=torch.float32, device=q.device)
        need = workspace_bytes_dkdv(OP_BWD, dt, B, H, N, d, d_v, causal)
        ws = torch.empty(max(need, 256), dtype=torch.uint8, device=q.device) if workspace is None else workspace
        sp = _scale(m, seq_len)
        st = [_strides_of(q, k), _strides_of(v), _strides_of(d_o), _strides_of(dq, dk), _strides_of(dv)]
        rc = _load().cott_bwd_dkdv(q.data_ptr(), k.data_ptr(), v.data_ptr(), d_o.data_ptr(), dq.data_ptr(),
                                   dk.data_ptr(), dv.data_ptr(), dm.data_ptr(), B, H, N, d, d_v,
                                   int(bool(causal)), dt, *[_ref(x) for x in st], ctypes.byref(sp),
                                   ws.data_ptr(), ws.numel(), _stream_ptr(stream))
        if rc != 0:
            raise CottError(rc, "cott_bwd_dkdv")
        return dq, dk, dv, dm
    dq, dk, dv = (torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)) if out is None else out
    _check_rows(dq, dk, dv)
    s_qkv, s_do, s_dqkv = _strides_of(q, k, v), _strides_of(d_o), _strides_of(dq, dk, dv)
    dm = torch.empty((H,), dtype=torch.float32, device=q.device)
    ws, ws_bytes = _workspace(OP_BWD, dt, B, H, N, d, causal, q.device, workspace)
    sp = _scale(m, seq_len)
    if fwd_workspace is not None:
        rc = _load().cott_bwd_after_fwd(q.data_ptr(), k.data_ptr(), v.data_ptr(), d_o.data_ptr(),
                                        dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), dm.data_ptr(), B, H, N,
                                        d, int(bool(causal)), dt, _ref(s_qkv), _ref(s_do), _ref(s_dqkv),
                                        ctypes.byref(sp), fwd_workspace.data_ptr(), ws.data_ptr(), ws_bytes,
                                        _stream_ptr(stream))
        if rc != 0:
            raise CottError(rc, "cott_bwd_after_fwd")
        return dq, dk, dv, dm
    rc = _load().cott_bwd_strided(q.data_ptr(), k.data_ptr(), v.data_ptr(), d_o.data_ptr(),
                                  dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), dm.data_ptr(), B, H, N,
                                  d, int(bool(causal)), dt, _ref(s_qkv), _ref(s_do), _ref(s_dqkv),
                                  ctypes.byref(sp), ws.data_ptr(), ws_bytes, _stream_ptr(stream))
    if rc != 0:
        raise CottError(rc, "cott_bwd_strided")
    return dq, dk, dv, dm


def _check_packed(cu_seqlens, *ts):
    if cu_seqlens.dtype != torch.int32 or cu_seqlens.dim() != 1 or cu_seqlens.numel() < 2:
        raise ValueError("cu_seqlens must be an int32 [B+1] CUDA tensor")
    _check_dev(cu_seqlens, *ts)
    for t in ts:
        if t.dim() != 3 or t.shape != ts[0].shape:
            raise ValueError("packed tensors must all be [total_tokens, H, d]")


@_on_call_stream
def fwd_varlen(q, k, v, m, cu_seqlens, max_seqlen, seq_len=None, causal=True, out=None, workspace=None,
               stream=None):
    """cott_fwd_varlen: q, k, v ``[total_tokens, H, d]`` (bf16, d a multiple of 8 up to 128), the sequences of the
    batch back to back; ``cu_seqlens`` int32 ``[B+1]`` CUDA tensor of row offsets.  Returns ``o``."""
    _check_packed(cu_seqlens, q, k, v)
    _check_dev(m, seq_len if isinstance(seq_len, torch.Tensor) else None)
    T, H, d = q.shape
    B = cu_seqlens.numel() - 1
    dt = _dt(q)
    o = torch.empty_like(q) if out is None else out
    ws, ws_bytes = _workspace_varlen(OP_FWD, dt, B, H, T, int(max_seqlen), d, causal, q.device, workspace)
    sp = _scale(m, seq_len)
    rc = _load().cott_fwd_varlen(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(),
                                 cu_seqlens.data_ptr(), B, H, T, int(max_seqlen), d, int(bool(causal)), dt,
                                 ctypes.byref(sp), ws.data_ptr(), ws_bytes, _stream_ptr(stream))
    if rc != 0:
        raise CottError(rc, "cott_fwd_varlen")
    return o


@_on_call_stream
def bwd_varlen(q, k, v, d_o, m, cu_seqlens, max_seqlen, seq_len=None, causal=True, workspace=None,
               stream=None):
    """cott_bwd_varlen.  Returns ``(dq, dk, dv, dm[H] fp32)`` for packed ``[total_tokens, H, d]`` inputs."""
    _check_packed(cu_seqlens, q, k, v, d_o)
    _check_dev(m, seq_len if isinstance(seq_len, torch.Tensor) else None)
    T, H, d = q.shape
    B = cu_seqlens.numel() - 1
    dt = _dt(q)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)
    dm = torch.empty((H,), dtype=torch.float32, device=q.device)
    ws, ws_bytes = _workspace_varlen(OP_BWD, dt, B, H, T, int(max_seqlen), d, causal, q.device, workspace)
    sp = _scale(m, seq_len)
    rc = _load().cott_bwd_varlen(q.data_ptr(), k.data_ptr(), v.data_ptr(), d_o.data_ptr(), dq.data_ptr(),
                                 dk.data_ptr(), dv.data_ptr(), dm.data_ptr(), cu_seqlens.data_ptr(), B, H, T,
                                 int(max_seqlen), d, int(bool(causal)), dt, ctypes.byref(sp), ws.data_ptr(),
                                 ws_bytes, _stream_ptr(stream))
    if rc != 0:
        raise CottError(rc, "cott_bwd_varlen")
    return dq, dk, dv, dm


@_on_call_stream
def bwd_stateful(q, k, v, d_o, m, seq_len, state_in=None, d_state_out=None, return_d_state=True,
                 workspace=None, stream=None, out=None):
    """cott_bwd_stateful: the backward of one segment of a longer causal sequence.  ``state_in``
    (fp32 ``[B,H,d_k,d_v]`` or None = zero) is what ``fwd_stateful`` was given for the segment,
    ``d_state_out`` (same shape, or None = zero) the gradient of the state it handed on (the
    ``d_state_in`` of the next segment's backward); ``seq_len`` as for ``fwd_stateful``; tensors and
    ``out`` as for ``bwd`` (strides are picked up).  Returns ``(dq, dk, dv, d_state_in, dm)``
    (``d_state_in`` is None when not asked for)."""
    _check_rows(q, k, v, d_o)
    _check_dev(m, state_in, d_state_out, seq_len if isinstance(seq_len, torch.Tensor) else None)
    B, H, N, d = q.shape
    d_v = v.shape[-1]
    dt = _dt(q)
    for t in (state_in, d_state_out):
        if t is not None and (t.dtype != torch.float32 or tuple(t.shape) != (B, H, d, d_v) or not t.is_contiguous()):
            raise ValueError("states must be contiguous float32 [B,H,d_k,d_v]")
    dq, dk, dv = (torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)) if out is None else out
    _check_rows(dq, dk, dv)
    same = d == d_v
    st = [_strides_of(q, k, v) if same else _strides_of(q, k), None if same else _strides_of(v), _strides_of(d_o),
          _strides_of(dq, dk, dv) if same else _strides_of(dq, dk), None if same else _strides_of(dv)]
    dm = torch.empty((H,), dtype=torch.float32, device=q.device)
    d_state_in = torch.empty((B, H, d, d_v), dtype=torch.float32, device=q.device) if return_d_state else None
    need = workspace_bytes_dkdv(OP_BWD, dt, B, H, N, d, d_v, True)
    ws = torch.empty(max(need, 256), dtype=torch.uint8, device=q.device) if workspace is None else workspace
    sp = _scale(m, seq_len)
    ptr = lambda t: 0 if t is None else t.data_ptr()
    rc = _load().cott_bwd_stateful_strided(q.data_ptr(), k.data_ptr(), v.data_ptr(), d_o.data_ptr(), ptr(state_in),
                                           ptr(d_state_out), dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), ptr(d_state_in),
                                           dm.data_ptr(), B, H, N, d, d_v, dt, *[_ref(x) for x in st], ctypes.byref(sp),
                                           ws.data_ptr(), ws.numel(), _stream_ptr(stream))
    if rc != 0:
        raise CottError(rc, "cott_bwd_stateful_strided")
    return dq, dk, dv, d_state_in, dm


@_on_call_stream
def decode_step(q, k, v, state, m, seq_len, out=None, stream=None):
    """cott_decode_step.  q,k,v ``[B,H,d]``; ``state`` fp32 ``[B,H,d,d]`` updated in place;
    ``seq_len`` a float (>= 1) or a float32 ``[B]`` CUDA tensor.  Returns ``o [B,H,d]``."""
    _check_dev(q, k, v, state, m, seq_len if isinstance(seq_len, torch.Tensor) else None)
    B, H, d = q.shape
    d_v = v.shape[-1]
    if state.dtype != torch.float32 or tuple(state.shape) != (B, H, d, d_v):
        raise ValueError("state must be float32 [B,H,d_k,d_v]")
    o = torch.empty_like(v) if out is None else out
    sp = _scale(m, seq_len)
    if d_v != d:
        rc = _load().cott_decode_step_dkdv(q.data_ptr(), k.data_ptr(), v.data_ptr(), state.data_ptr(), o.data_ptr(),
                                           B, H, d, d_v, _dt(q), ctypes.byref(sp), _stream_ptr(stream))
        if rc != 0:
            raise CottError(rc, "cott_decode_step_dkdv")
        return o
    rc = _load().cott_decode_step(q.data_ptr(), k.data_ptr(), v.data_ptr(), state.data_ptr(),
                                  o.data_ptr(), B, H, d, _dt(q), ctypes.byref(sp),
                                  _stream_ptr(stream))
    if rc != 0:
        raise CottError(rc, "cott_decode_step")
    return o


@_on_call_stream
def fwd_bwd_host(q, k, v, d_o, m, o, dq, dk, dv, dm, causal=True, seq_len=None, arena=None,
                 stream=None):
    """cott_fwd_bwd_host: every tensor argument is a HOST tensor (pinned for async copies);
    ``arena`` is a uint8 CUDA tensor (allocated here if None).  Returns the arena."""
    B, H, N, d = q.shape
    dt = _dt(q)
    lib = _load()
    need = lib.cott_host_step_arena_bytes(dt, B, H, N, d, int(bool(causal)))
    if need == _SIZE_MAX:
        raise CottError(-2, "cott_host_step_arena_bytes")
    if arena is None:
        arena = torch.empty(need, dtype=torch.uint8, device="cuda")
    rc = lib.cott_fwd_bwd_host(q.data_ptr(), k.data_ptr(), v.data_ptr(), d_o.data_ptr(),
                               o.data_ptr(), dq.data_ptr(), dk.data_ptr(), dv.data_ptr(),
                               dm.data_ptr(), m.data_ptr(),
                               seq_len.data_ptr() if seq_len is not None else None, B, H, N, d,
                               int(bool(causal)), dt, arena.data_ptr(), arena.numel(),
                               _stream_ptr(stream))
    if rc != 0:
        raise CottError(rc, "cott_fwd_bwd_host")
    return arena


def host_step_slicing(B: int, H: int) -> dict:
    """cott_host_step_slicing: how ``fwd_bwd_host`` cuts a batch into slices."""
    a, b, c = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
    rc = _load().cott_host_step_slicing(B, H, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c))
    if rc != 0:
        raise CottError(rc, "cott_host_step_slicing")
    return {"items": a.value, "heads": b.value, "n": c.value}


def launch_count() -> int:
    return int(_load().cott_launch_count())


def profile_enable(max_launches: int) -> None:
    rc = _load().cott_profile_enable(int(max_launches))
    if rc != 0:
        raise CottError(rc, "cott_profile_enable")


def profile_read(cap: int = 256):
    """Returns [(kind, milliseconds), ...] of the walk-kernel launches recorded so far."""
    ms = (ctypes.c_float * cap)()
    kinds = (ctypes.c_int * cap)()
    n = _load().cott_profile_read(ms, kinds, cap)
    if n < 0:
        raise CottError(-4, "cott_profile_read")
    return [(int(kinds[i]), float(ms[i])) for i in range(n)]


def last_async_status(workspace: torch.Tensor, stream=None) -> int:
    return int(_load().cott_last_async_status(workspace.data_ptr(), _stream_ptr(stream)))
