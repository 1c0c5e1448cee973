"""The C-ABI library loads, exports every symbol the header declares, and its host-only
entry points behave.  No kernel is launched here (runs without a GPU)."""
import ctypes
import os
import re

import paper_2409_18747_b200 as cott_pkg
from paper_2409_18747_b200 import cott

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "cott.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cott_[a-z_0-9]+)\s*\(", text)))


def test_exports_every_declared_symbol():
    lib = ctypes.CDLL(cott_pkg.library_path())
    names = declared_symbols()
    assert {"cott_fwd", "cott_bwd", "cott_decode_step", "cott_workspace_bytes"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_version_and_status_strings():
    lib = cott._load()
    assert lib.cott_version() >= 100
    seen = {lib.cott_status_string(s).decode() for s in (0, -1, -2, -3, -4, -5)}
    assert len(seen) == 6


def test_workspace_and_plan_are_host_only():
    for (B, H, N, d, causal) in [(1, 2, 256, 32, True), (32, 12, 512, 64, False), (4, 16, 4096, 64, True),
                                 (1, 16, 131072, 128, True)]:
        for dt in (cott.F32, cott.BF16):
            plan = cott.query_plan(cott.OP_FWD, dt, B, H, N, d, causal)
            assert plan["group"] % plan["chunk"] == 0 and plan["group"] >= 1
            wf = cott.workspace_bytes(cott.OP_FWD, dt, B, H, N, d, causal)
            wb = cott.workspace_bytes(cott.OP_BWD, dt, B, H, N, d, causal)
            assert 256 <= wf <= wb < (8 << 30)
    assert cott.workspace_bytes(cott.OP_DECODE, cott.BF16, 64, 16, 1, 128, True) == 0
    lib = cott._load()
    assert lib.cott_workspace_bytes(0, cott.BF16, 1, 1, 16, 44, 1) == ctypes.c_size_t(-1).value  # rows not of 16 bytes
    assert lib.cott_workspace_bytes(0, cott.BF16, 1, 1, 16, 136, 1) == ctypes.c_size_t(-1).value  # d beyond 128
    assert lib.cott_workspace_bytes(0, cott.F32, 1, 1, 16, 48, 1) == ctypes.c_size_t(-1).value  # fp32: 32, 64, 128 only
    # bf16 head sizes that are multiples of 8 run zero-padded in the next kernel size: the same
    # group states plus room for a caller's state in that size, in and out
    lib.cott_workspace_bytes_dkdv.restype = ctypes.c_size_t
    w64 = lib.cott_workspace_bytes(0, cott.BF16, 1, 1, 16, 64, 1)
    assert lib.cott_workspace_bytes(0, cott.BF16, 1, 1, 16, 48, 1) == w64 + 2 * 64 * 64 * 4
    assert lib.cott_workspace_bytes_dkdv(0, cott.BF16, 1, 1, 16, 64, 64, 1) == w64
    w128 = lib.cott_workspace_bytes(0, cott.BF16, 1, 1, 16, 128, 1)
    assert lib.cott_workspace_bytes_dkdv(0, cott.BF16, 1, 1, 16, 64, 128, 1) == w128 + 2 * 128 * 128 * 4
    assert lib.cott_workspace_bytes_dkdv(0, cott.F32, 1, 1, 16, 32, 64, 1) == ctypes.c_size_t(-1).value
    kd = ctypes.c_int()
    assert lib.cott_query_plan_dkdv(0, cott.BF16, 1, 1, 16, 32, 96, 1, None, None, None, ctypes.byref(kd)) == 0
    assert kd.value == 128
    assert lib.cott_query_plan_dkdv(0, cott.BF16, 1, 1, 16, 32, 40, 1, None, None, None, ctypes.byref(kd)) == 0
    assert kd.value == 64
    assert lib.cott_workspace_bytes(0, cott.BF16, 0, 1, 16, 64, 1) == ctypes.c_size_t(-1).value


def test_argument_validation_returns_before_any_launch():
    lib = cott._load()
    sp = cott._ScaleParams()
    sp.m, sp.seq_len, sp.seq_len_scalar = 256, None, 0.0  # fake non-NULL address: never dereferenced on host
    a = 4096  # fake 16-byte aligned device address; validation must fail before it is used
    null = None
    # NULL tensor
    assert lib.cott_fwd(null, a, a, a, null, 1, 1, 16, 64, 1, cott.BF16, ctypes.byref(sp), a, 1 << 20, null) == -1
    # NULL scale params / NULL m
    assert lib.cott_fwd(a, a, a, a + 65536, null, 1, 1, 16, 64, 1, cott.BF16, None, a, 1 << 20, null) == -1
    # output aliases an input
    assert lib.cott_fwd(a, a, a, a, null, 1, 1, 16, 64, 1, cott.BF16, ctypes.byref(sp), a, 1 << 20, null) == -1
    # unsupported head dimension, misaligned pointer
    assert lib.cott_fwd(a, a, a, a + 65536, null, 1, 1, 16, 44, 1, cott.BF16, ctypes.byref(sp), a, 1 << 20, null) == -2
    assert lib.cott_fwd(a + 2, a, a, a + 65536, null, 1, 1, 16, 64, 1, cott.BF16, ctypes.byref(sp), a, 1 << 20, null) == -2
    # workspace missing / too small
    assert lib.cott_fwd(a, a, a, a + 65536, null, 1, 1, 16, 64, 1, cott.BF16, ctypes.byref(sp), null, 0, null) == -3
    assert lib.cott_fwd(a, a, a, a + 65536, null, 1, 1, 16, 64, 1, cott.BF16, ctypes.byref(sp), a, 8, null) == -3
    # scaling base below one
    sp.seq_len_scalar = 0.5
    assert lib.cott_fwd(a, a, a, a + 65536, null, 1, 1, 16, 64, 1, cott.BF16, ctypes.byref(sp), a, 1 << 20, null) == -1
    assert lib.cott_decode_step(a, a, a, a, a + 65536, 1, 1, 64, cott.BF16, ctypes.byref(sp), null) == -1
    sp.seq_len_scalar = 0.0
    assert lib.cott_decode_step(a, a, a, a, a + 65536, 1, 1, 64, cott.BF16, ctypes.byref(sp), null) == -1
    # backward: NULL dm, aliasing outputs
    assert lib.cott_bwd(a, a, a, a, a + 65536, a + 131072, a + 196608, null, 1, 1, 16, 64, 1, cott.BF16,
                        ctypes.byref(sp), a, 1 << 24, null) == -1
    assert lib.cott_bwd(a, a, a, a, a + 65536, a + 65536, a + 196608, a, 1, 1, 16, 64, 1, cott.BF16,
                        ctypes.byref(sp), a, 1 << 24, null) == -1


def test_strided_and_packed_entry_points_validate_on_the_host():
    """cott_*_strided and cott_*_varlen refuse strides and shapes they cannot address before
    anything is launched (fake addresses, never dereferenced)."""
    lib = cott._load()
    sp = cott._ScaleParams()
    sp.m, sp.seq_len, sp.seq_len_scalar = 256, None, 0.0
    a, null = 4096, None
    S = cott._Strides
    ok = S(16 * 2 * 64, 64, 2 * 64)           # [B,N,H,d] with H=2, d=64, N=16
    args = (a, a, a, a + 65536, null, 1, 2, 16, 64, 1, cott.BF16)
    tail = (ctypes.byref(sp), a, 1 << 20, null)
    # token stride not a multiple of 16 bytes / smaller than a row
    assert lib.cott_fwd_strided(*args, ctypes.byref(S(4096, 64, 132)), None, *tail) == -2
    assert lib.cott_fwd_strided(*args, ctypes.byref(S(4096, 64, 32)), None, *tail) == -2
    assert lib.cott_fwd_strided(*args, None, ctypes.byref(S(4096, 8, 128)), *tail) == -2
    # good strides get as far as the workspace check
    assert lib.cott_fwd_strided(*args, ctypes.byref(ok), ctypes.byref(ok), ctypes.byref(sp), null, 0, null) == -3
    bargs = (a, a, a, a, a + 65536, a + 131072, a + 196608, a, 1, 2, 16, 64, 1, cott.BF16)
    assert lib.cott_bwd_strided(*bargs, None, None, ctypes.byref(S(4096, 64, 130)), ctypes.byref(sp), a, 1 << 24, null) == -2
    assert lib.cott_bwd_strided(*bargs, ctypes.byref(ok), None, ctypes.byref(ok), ctypes.byref(sp), null, 0, null) == -3
    # packed batches: NULL cu_seqlens, fp32 or rows that are not multiples of 16 bytes (tensor-core path only), max_seqlen > total
    v = (a, a, a, a + 65536)
    assert lib.cott_fwd_varlen(*v, null, 2, 2, 100, 60, 64, 1, cott.BF16, *tail) == -1
    assert lib.cott_fwd_varlen(*v, a, 2, 2, 100, 60, 96, 1, cott.F32, *tail) == -2          # fp32: 32, 64, 128 only
    assert lib.cott_fwd_varlen(*v, a, 2, 2, 100, 60, 36, 1, cott.BF16, *tail) == -2
    assert lib.cott_fwd_varlen(*v, a, 2, 2, 100, 200, 64, 1, cott.BF16, *tail) == -2
    assert lib.cott_fwd_varlen(*v, a, 2, 2, 100, 60, 64, 1, cott.BF16, ctypes.byref(sp), null, 0, null) == -3
    assert lib.cott_bwd_varlen(a, a, a, a, a + 65536, a + 131072, a + 196608, a, null, 2, 2, 100, 60, 64, 1,
                               cott.BF16, ctypes.byref(sp), a, 1 << 24, null) == -1


def test_outputs_that_share_bytes_with_other_tensors_are_refused():
    """Aliasing is decided by the bytes the tensors cover, not by pointer equality: dense
    tensors whose ranges meet and equally strided tensors whose rows meet are refused, while
    the interleaved slices of one fused buffer (ranges meet, rows do not) are accepted."""
    lib = cott._load()
    sp = cott._ScaleParams()
    sp.m, sp.seq_len, sp.seq_len_scalar = 256, None, 0.0
    a, null = 1 << 20, None
    B, H, N, d = 1, 2, 16, 64
    nbytes = B * H * N * d * 2
    tail = (ctypes.byref(sp), null, 0, null)          # valid calls stop at the workspace check (-3)
    f = lambda o: lib.cott_fwd(a, a + nbytes, a + 2 * nbytes, o, null, B, H, N, d, 1, cott.BF16, *tail)
    assert f(a + 3 * nbytes) == -3                     # disjoint
    assert f(a + 2 * nbytes + 128) == -1               # o starts inside v
    assert f(a - 256) == -1                            # o ends inside q
    assert f(a + nbytes - 16) == -1                    # straddles q and k
    g = lambda dq, dk, dv: lib.cott_bwd(a, a + nbytes, a + 2 * nbytes, a + 3 * nbytes, dq, dk, dv, a + 64 * nbytes,
                                        B, H, N, d, 1, cott.BF16, *tail)
    assert g(a + 4 * nbytes, a + 5 * nbytes, a + 6 * nbytes) == -3
    assert g(a + 4 * nbytes, a + 4 * nbytes + 256, a + 6 * nbytes) == -1      # dk starts inside dq
    assert g(a + 3 * nbytes + 512, a + 5 * nbytes, a + 6 * nbytes) == -1      # dq overlaps dO
    # slices of a fused [B,N,3,H,d] buffer: q, k, v interleaved per token; gradients likewise
    S = cott._Strides
    fused = S(N * 3 * H * d, d, 3 * H * d)
    row = H * d * 2
    base_in, base_out = a, a + (1 << 22)
    ok = lib.cott_bwd_strided(base_in, base_in + row, base_in + 2 * row, a + (1 << 23),
                              base_out, base_out + row, base_out + 2 * row, a + (1 << 24), B, H, N, d, 1, cott.BF16,
                              ctypes.byref(fused), None, ctypes.byref(fused), *tail)
    assert ok == -3
    bad = lib.cott_bwd_strided(base_in, base_in + row, base_in + 2 * row, a + (1 << 23),
                               base_out, base_out + row - 64, base_out + 2 * row, a + (1 << 24), B, H, N, d, 1, cott.BF16,
                               ctypes.byref(fused), None, ctypes.byref(fused), *tail)
    assert bad == -1                                    # dk's rows run into dq's
    same = lib.cott_bwd_strided(base_in, base_in + row, base_in + 2 * row, a + (1 << 23),
                                base_in + row, base_out + row, base_out + 2 * row, a + (1 << 24), B, H, N, d, 1, cott.BF16,
                                ctypes.byref(fused), None, ctypes.byref(fused), *tail)
    assert same == -1                                   # dq is the k slice


def test_slices_of_different_widths_in_one_buffer():
    """Key and value sizes of their own (48 and 80 columns): q, k, v as column slices of one
    [B,N,H,176] buffer do not meet although their ranges interleave; a dv slice that starts
    inside dk's columns does."""
    lib = cott._load()
    sp = cott._ScaleParams()
    sp.m, sp.seq_len, sp.seq_len_scalar = 256, None, 0.0
    a, g0, null = 1 << 20, 1 << 24, None
    B, H, N, dk, dv = 1, 2, 16, 48, 80
    W = 2 * dk + dv
    S = cott._Strides
    fused = S(N * H * W, W, H * W)
    tail = (ctypes.byref(sp), null, 0, null)                       # valid calls stop at the workspace check (-3)
    call = lambda dq, dk_, dv_: lib.cott_bwd_dkdv(a, a + 2 * dk, a + 4 * dk, 1 << 26, dq, dk_, dv_, 1 << 27, B, H, N,
                                                  dk, dv, 1, cott.BF16, ctypes.byref(fused), ctypes.byref(fused), None,
                                                  ctypes.byref(fused), ctypes.byref(fused), *tail)
    assert call(g0, g0 + 2 * dk, g0 + 4 * dk) == -3                # dq | dk | dv side by side in each row
    assert call(g0, g0 + 2 * dk, g0 + 4 * dk - 32) == -1           # dv starts 16 columns inside dk
    assert call(g0, g0 + 2 * dk - 16, g0 + 4 * dk) == -1           # dk starts inside dq
    assert call(a + 4 * dk + 2 * dv - 16, g0 + 2 * dk, g0 + 4 * dk) == -1   # dq starts inside v's last columns
    f = lambda o: lib.cott_fwd_dkdv(a, a + 2 * dk, a + 4 * dk, o, null, null, B, H, N, dk, dv, 1, cott.BF16,
                                    ctypes.byref(fused), ctypes.byref(fused), None, *tail)
    assert f(g0) == -3 and f(a) == -1                              # dense o elsewhere / o at q's address


def test_options_and_shutdown_are_host_only():
    assert cott.get_option("fused_bwd") in (0, 1, 2)
    old = cott.get_option("force_group")
    cott.set_option("force_group", 384)
    assert cott.get_option("force_group") == 384
    assert cott.query_plan(cott.OP_FWD, cott.BF16, 1, 2, 4096, 64, True)["group"] == 384
    cott.set_option("force_group", old)
    try:
        cott.set_option("no_such_option", 1)
    except cott.CottError as e:
        assert e.status == -1
    else:
        raise AssertionError("unknown option names must be refused")
    assert cott.get_option("no_such_option") == -1
    cott.shutdown()          # nothing created yet on a machine without a GPU: still fine
    cott.shutdown()


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(cott, "_lib", None)
    monkeypatch.setattr(cott, "_LIB_PATH", "/nonexistent/libcott.so")
    try:
        cott._load()
    except RuntimeError as e:
        assert "no CPU" in str(e)
    else:
        raise AssertionError("loading a missing library must raise")


def test_cpu_tensors_are_rejected():
    import torch
    q = torch.zeros((1, 1, 16, 64), dtype=torch.bfloat16)
    m = torch.zeros((1,))
    try:
        cott.fwd(q, q, q, m)
    except RuntimeError as e:
        assert "CUDA" in str(e)
    else:
        raise AssertionError("CPU tensors must be rejected")
