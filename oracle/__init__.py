"""ctypes front end of the fp64 CPU oracle (``cott_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the test-suite, the smoke check and the
benchmark's CPU-baseline / reference arm.  The GPU library never imports it,
and it imports nothing from the GPU package.

Every function takes array-likes (numpy arrays or CPU torch tensors of any
float dtype), converts them *exactly* to float64 and returns float64 numpy
arrays.  Shapes: q,k,v,o,dO ``[B,H,N,d]``; ``m`` ``[H]``; ``s`` ``[B]`` (the
scaling base of Eq. 4; ``None`` means the tensor's sequence length N).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cott_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no fast-math, so fp64 stays IEEE)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_num_threads(n: int) -> None:
    _load().oracle_set_num_threads(ctypes.c_int(int(n)))


def _f64(x) -> np.ndarray:
    if hasattr(x, "detach"):  # torch tensor (bf16 has no numpy dtype: widen first)
        x = x.detach().cpu().double().numpy()
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _prep(q, k, v, m, s):
    q, k, v, m = _f64(q), _f64(k), _f64(v), _f64(m).reshape(-1)
    B, H, N, dk = q.shape
    dv = v.shape[-1]
    assert k.shape == q.shape and v.shape == (B, H, N, dv) and m.shape == (H,)
    s = np.full((B,), float(N)) if s is None else _f64(s).reshape(-1)
    assert s.shape == (B,) and (s >= 1.0).all()
    return q, k, v, m, s, B, H, N, dk, dv


def fwd_quadratic(q, k, v, m, s=None, causal=True) -> np.ndarray:
    """Eq. 3/4 (bidirectional) or Eq. 6 (causal, diagonal kept): the definition.
    q, k ``[B,H,N,dk]``, v ``[B,H,N,dv]``; returns o ``[B,H,N,dv]``."""
    q, k, v, m, s, B, H, N, dk, dv = _prep(q, k, v, m, s)
    o = np.empty_like(v)
    _load().oracle_fwd_quadratic(_p(q), _p(k), _p(v), _p(m), _p(s), _p(o), B, H,
                                 ctypes.c_long(N), dk, dv, int(bool(causal)))
    return o


def fwd_rows(q, k, v, m, rows, s=None, causal=True) -> np.ndarray:
    """The definition on selected rows only; returns ``[B,H,len(rows),dv]``."""
    q, k, v, m, s, B, H, N, dk, dv = _prep(q, k, v, m, s)
    rows = np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
    assert rows.ndim == 1 and (rows >= 0).all() and (rows < N).all()
    out = np.empty((B, H, len(rows), dv))
    _load().oracle_fwd_rows(_p(q), _p(k), _p(v), _p(m), _p(s), _p(rows), len(rows), _p(out), B, H,
                            ctypes.c_long(N), dk, dv, int(bool(causal)))
    return out


def fwd_recurrent(q, k, v, m, s=None):
    """Eq. 8 recurrence (causal).  Returns ``(o, final_state[B,H,dk,dv])``."""
    q, k, v, m, s, B, H, N, dk, dv = _prep(q, k, v, m, s)
    o = np.empty_like(v)
    st = np.empty((B, H, dk, dv))
    _load().oracle_fwd_recurrent(_p(q), _p(k), _p(v), _p(m), _p(s), _p(o), _p(st), B, H,
                                 ctypes.c_long(N), dk, dv)
    return o, st


def fwd_bidir_assoc(q, k, v, m, s=None):
    """Eq. 5 right-hand side.  Returns ``(o, state[B,H,dk,dv])``."""
    q, k, v, m, s, B, H, N, dk, dv = _prep(q, k, v, m, s)
    o = np.empty_like(v)
    st = np.empty((B, H, dk, dv))
    _load().oracle_fwd_bidir_assoc(_p(q), _p(k), _p(v), _p(m), _p(s), _p(o), _p(st), B, H,
                                   ctypes.c_long(N), dk, dv)
    return o, st


def bwd_quadratic(q, k, v, d_o, m, s=None, causal=True):
    """Gradients of sum(dO*O) w.r.t. raw q,k,v and m.  Returns (dq,dk,dv,dm)."""
    q, k, v, m, s, B, H, N, dk, dv = _prep(q, k, v, m, s)
    d_o = _f64(d_o)
    assert d_o.shape == v.shape
    dq, dk_, dv_ = np.empty_like(q), np.empty_like(q), np.empty_like(v)
    dm = np.empty((H,))
    _load().oracle_bwd_quadratic(_p(q), _p(k), _p(v), _p(d_o), _p(m), _p(s), _p(dq), _p(dk_),
                                 _p(dv_), _p(dm), B, H, ctypes.c_long(N), dk, dv, int(bool(causal)))
    return dq, dk_, dv_, dm


def bwd_recurrent(q, k, v, d_o, m, s=None):
    """Causal backward via forward / reverse running sums.  Returns (dq,dk,dv,dm)."""
    q, k, v, m, s, B, H, N, dk, dv = _prep(q, k, v, m, s)
    d_o = _f64(d_o)
    assert d_o.shape == v.shape
    dq, dk_, dv_ = np.empty_like(q), np.empty_like(q), np.empty_like(v)
    dm = np.empty((H,))
    _load().oracle_bwd_recurrent(_p(q), _p(k), _p(v), _p(d_o), _p(m), _p(s), _p(dq), _p(dk_),
                                 _p(dv_), _p(dm), B, H, ctypes.c_long(N), dk, dv)
    return dq, dk_, dv_, dm


def fwd_segment(q, k, v, m, state_in, s=None):
    """A segment of a longer causal sequence: Eq. 8 started from ``state_in [B,H,dk,dv]``.
    Returns ``(o, state_out)``."""
    q, k, v, m, s, B, H, N, dk, dv = _prep(q, k, v, m, s)
    st_in = np.ascontiguousarray(_f64(state_in)).reshape(B, H, dk, dv)
    o = np.empty_like(v)
    st = np.empty((B, H, dk, dv))
    _load().oracle_fwd_segment(_p(q), _p(k), _p(v), _p(m), _p(s), _p(st_in), _p(o), _p(st), B, H,
                               ctypes.c_long(N), dk, dv)
    return o, st


def bwd_segment(q, k, v, d_o, m, state_in, d_state_out, s=None):
    """Gradients of ``sum(dO*O) + sum(d_state_out*state_out)`` of a segment w.r.t. raw q, k, v,
    ``state_in`` and m.  Returns ``(dq, dk, dv, d_state_in, dm)``."""
    q, k, v, m, s, B, H, N, dk, dv = _prep(q, k, v, m, s)
    d_o = _f64(d_o)
    assert d_o.shape == v.shape
    st_in = np.ascontiguousarray(_f64(state_in)).reshape(B, H, dk, dv)
    d_st_out = np.ascontiguousarray(_f64(d_state_out)).reshape(B, H, dk, dv)
    dq, dk_, dv_ = np.empty_like(q), np.empty_like(q), np.empty_like(v)
    d_st_in = np.empty((B, H, dk, dv))
    dm = np.empty((H,))
    _load().oracle_bwd_segment(_p(q), _p(k), _p(v), _p(d_o), _p(st_in), _p(d_st_out), _p(m), _p(s),
                               _p(dq), _p(dk_), _p(dv_), _p(d_st_in), _p(dm), B, H, ctypes.c_long(N), dk, dv)
    return dq, dk_, dv_, d_st_in, dm


def decode_step(q, k, v, m, s, state):
    """One Eq. 8 step.  q,k ``[B,H,dk]``, v ``[B,H,dv]``; ``state`` ``[B,H,dk,dv]`` float64 numpy,
    updated IN PLACE; ``s`` ``[B]`` or a scalar.  Returns o ``[B,H,dv]``."""
    q, k, v, m = _f64(q), _f64(k), _f64(v), _f64(m).reshape(-1)
    B, H, dk = q.shape
    dv = v.shape[-1]
    s = np.full((B,), float(s)) if np.isscalar(s) else _f64(s).reshape(-1)
    assert state.dtype == np.float64 and state.flags.c_contiguous and state.shape == (B, H, dk, dv)
    o = np.empty_like(v)
    _load().oracle_decode_step(_p(q), _p(k), _p(v), _p(m), _p(s), _p(state), _p(o), B, H, dk, dv)
    return o
