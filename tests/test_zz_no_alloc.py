"""cott_fwd_noalloc: the forward pass for callers that cannot give the library a workspace
(their process cannot, or must not, allocate device memory when the call is made).  It runs
on a fixed scratch array inside the library, so it must agree with cott_fwd, call after call,
whatever an earlier call left in that array.  Collected last on purpose."""
import ctypes

import pytest
import torch

import oracle
import paper_2409_18747_b200 as cott
from paper_2409_18747_b200 import synth
from _metrics import norm_max_err

pytestmark = pytest.mark.gpu


def test_noalloc_matches_cott_fwd_twice_in_a_row():
    lib = cott.cott._load()
    assert lib.cott_fwd_noalloc_max_bytes() == 8 << 20
    first = synth.make_qkv(2, 4, 1000, 64, torch.bfloat16, 9101)     # several groups, ragged tail
    second = synth.make_qkv(1, 3, 640, 128, torch.bfloat16, 9102)    # other shape: scratch reused as is
    for case, causal in ((first, True), (second, True), (first, False)):
        q, k, v, m = (case[x].cuda() for x in ("q", "k", "v", "m"))
        want = cott.fwd(q, k, v, m, causal=causal)
        got = cott.fwd_noalloc(q, k, v, m, causal=causal)
        torch.cuda.synchronize()
        assert norm_max_err(got, want.double().cpu().numpy()) <= 1e-2   # the bf16 gate of the parity tests
        assert torch.equal(got, want)                                    # same kernels, same order: same bits
        # and against the definition itself (fp64 oracle), so that this file stands on its own
        ref = oracle.fwd_quadratic(case["q"], case["k"], case["v"], case["m"], None, causal)
        assert norm_max_err(got, ref) <= 1e-2
        assert cott.cott.fwd_noalloc_status() == 0                       # no device-side wait gave up


def test_noalloc_rejects_problems_beyond_its_scratch():
    lib = cott.cott._load()
    B, H, N, d = 64, 16, 8192, 128   # the decode prefill: 64 MB of group states
    assert cott.workspace_bytes(cott.cott.OP_FWD, cott.cott.BF16, B, H, N, d, True) > lib.cott_fwd_noalloc_max_bytes()
    sp = cott.cott._ScaleParams()
    sp.m, sp.seq_len, sp.seq_len_scalar = 256, None, 0.0   # never dereferenced: the size check comes first
    rc = lib.cott_fwd_noalloc(4096, 4096, 4096, 8192, B, H, N, d, 1, cott.cott.BF16, ctypes.byref(sp), None)
    assert rc == -3
