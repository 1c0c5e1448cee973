"""GPU parity: libcott (through the C ABI) against the fp64 CPU oracle on the same seeded
inputs.  Tolerances: fp32 I/O max relative error (floored, see _metrics) <= 1e-4; bf16 I/O
normalised max error <= 1e-2; integer-valued index/mask cases bit-exact."""
import os

import numpy as np
import pytest
import torch

import oracle
import paper_2409_18747_b200 as cott
from paper_2409_18747_b200 import synth
from _metrics import norm_max_err, rel_err_floor

pytestmark = pytest.mark.gpu

TOL_F32 = 1e-4
TOL_BF16 = 1e-2
# Exported / decode states are fp32, but on the bf16 tensor-core path their operands (k^ and v)
# are bf16, so the state carries bf16 operand rounding: same normalised gate as bf16 outputs.
# The fp32 SIMT path accumulates exact fp32 products: 1e-5.
TOL_STATE_TC = 1e-2
TOL_STATE_F32 = 1e-5


def state_tol(dtype, d):
    return TOL_STATE_TC if dtype == torch.bfloat16 else TOL_STATE_F32     # (bf16 runs on tensor cores at every size)


def dev(x):
    return x.cuda() if isinstance(x, torch.Tensor) else x


def gate(x, ref, dtype):
    if dtype == torch.float32:
        e = rel_err_floor(x, ref)
        assert e <= TOL_F32, f"fp32 relative error {e:.3e} > {TOL_F32}"
    else:
        e = norm_max_err(x, ref)
        assert e <= TOL_BF16, f"bf16 normalised max error {e:.3e} > {TOL_BF16}"
    # shown with `pytest -s`: the measured error of every gated tensor
    print(f"[{os.environ.get('PYTEST_CURRENT_TEST', '').split('::')[-1].split(' ')[0]}] "
          f"{'fp32 rel' if dtype == torch.float32 else 'bf16 norm'} err {e:.3e}")
    return e


def dm_condition(dv_ref, v, m, s):
    """A_h = sum_{b,t} |<dV'_t, v_t>| * |dc/dm| for head h: the sum of the absolute values of the
    terms whose signed sum is dm_h.  dm is a dot product over B*N*d terms, so its rounding
    error scales with A_h, not with |dm_h| (the terms cancel heavily on random data)."""
    v = v.double().cpu().numpy()
    m = np.asarray(m.double().cpu().numpy())
    B, H, N, _ = v.shape
    s = np.full((B,), float(N)) if s is None else np.asarray(s.double().cpu().numpy() if hasattr(s, "cpu") else s)
    sg = 1.0 / (1.0 + np.exp(-m))
    per_bh = np.abs((dv_ref * v).sum(-1)).sum(-1)          # [B,H]; dv = c dV' so c is included
    return (per_bh * np.log(s)[:, None] * (sg * (1 - sg))[None, :]).sum(0)


def gate_dm(dm, ref, tol, cond, tol_cond):
    """Normalised max error of the scale-parameter gradient, max_h |dm_h - ref_h| / max_h |ref_h|,
    gated like every other bf16 (1e-2) / fp32 (1e-4) tensor.  Printed beside it, as a diagnostic
    only: the worst ratio of the error to the rounding bound tol_cond * A_h of a dot product
    whose terms cancel (see dm_condition)."""
    dm, ref = dm.double().cpu().numpy(), np.asarray(ref)
    e = np.abs(dm - ref)
    err = float(e.max() / max(np.abs(ref).max(), 1e-300))
    ratio = float((e / np.maximum(tol_cond * cond, 1e-300)).max())
    print(f"[{os.environ.get('PYTEST_CURRENT_TEST', '').split('::')[-1].split(' ')[0]}] "
          f"dm norm err {err:.3e} (gate {tol:g}); error / cancellation bound {ratio:.2f}")
    assert err <= tol, f"dm normalised max error {err:.3e} > {tol}: dm {dm} ref {ref}"
    return err


# bf16 operands carry 2^-9 relative rounding per element; fp32 about 2^-24
DM_COND_BF16 = 1e-3
DM_COND_F32 = 1e-6


@pytest.fixture
def option():
    """Sets library options (cott_set_option) for one test and restores them afterwards."""
    saved = {}

    def _set(name, value):
        saved.setdefault(name, cott.cott.get_option(name))
        cott.cott.set_option(name, value)
    yield _set
    for name, value in saved.items():
        cott.cott.set_option(name, value)


@pytest.fixture
def force_group(option):
    return lambda g: option("force_group", 0 if g is None else g)


# ------------------------------------------------------------------ the five workloads
def test_config1_tiny_causal_fp32():
    c = synth.make_config(1)
    o = cott.fwd(dev(c["q"]), dev(c["k"]), dev(c["v"]), dev(c["m"]), causal=True)
    ref = oracle.fwd_quadratic(c["q"], c["k"], c["v"], c["m"], None, True)
    ref_rec, _ = oracle.fwd_recurrent(c["q"], c["k"], c["v"], c["m"], None)
    np.testing.assert_allclose(ref_rec, ref, rtol=1e-11, atol=1e-12)
    gate(o, ref, torch.float32)
    # cosine similarity ignores row lengths: dividing out the lognormal factors changes nothing
    qn = c["q"] / c["q"].norm(dim=-1, keepdim=True)
    kn = c["k"] / c["k"].norm(dim=-1, keepdim=True)
    o2 = cott.fwd(dev(qn), dev(kn), dev(c["v"]), dev(c["m"]), causal=True)
    gate(o2, ref, torch.float32)


def test_config2_bidirectional_bf16():
    c = synth.make_config(2)
    o, st = cott.fwd(dev(c["q"]), dev(c["k"]), dev(c["v"]), dev(c["m"]), causal=False, return_state=True)
    ref, ref_state = oracle.fwd_bidir_assoc(c["q"], c["k"], c["v"], c["m"], None)
    gate(o, ref, torch.bfloat16)
    rows = [0, 1, 127, 128, 255, 256, 511]
    ref_rows = oracle.fwd_rows(c["q"], c["k"], c["v"], c["m"], rows, None, False)  # the definition itself
    gate(o[:, :, rows], ref_rows, torch.bfloat16)
    assert norm_max_err(st, ref_state) <= TOL_STATE_TC  # exported state = c K^^T V
    sub = slice(0, 2)
    ref_q = oracle.fwd_quadratic(c["q"][sub], c["k"][sub], c["v"][sub], c["m"], None, False)
    gate(o[sub], ref_q, torch.bfloat16)


def test_config3_causal_bf16_zero_keys():
    c = synth.make_config(3)
    o = cott.fwd(dev(c["q"]), dev(c["k"]), dev(c["v"]), dev(c["m"]), causal=True)
    ref, _ = oracle.fwd_recurrent(c["q"], c["k"], c["v"], c["m"], None)
    gate(o, ref, torch.bfloat16)
    sub = slice(0, 1)
    ref_q = oracle.fwd_quadratic(c["q"][sub], c["k"][sub], c["v"][sub], c["m"], None, True)
    gate(o[sub], ref_q, torch.bfloat16)
    # a zero key contributes nothing: replacing its value row by junk must not change a bit
    v2 = c["v"].clone()
    zero = (c["k"].float().abs().sum(-1) == 0)
    v2[zero] = 1000.0
    o2 = cott.fwd(dev(c["q"]), dev(c["k"]), dev(v2), dev(c["m"]), causal=True)
    assert torch.equal(o2, o)


def test_config3_backward_bf16_zero_keys():
    """Config 3 at full size with its backward (bench.py's c3-train: the GPT-2-small attention
    training step; 5 % of the key rows are exactly zero, so the clamped branch of the chain rule
    runs inside the one-walk backward): all gradients of the first batch item against the
    quadratic definition, the clamped key rows relative to their own size."""
    c = synth.make_config(3)
    B, H, N, d = c["q"].shape
    d_o = torch.randn(c["v"].shape, generator=torch.Generator().manual_seed(1003)).to(torch.bfloat16)
    dq, dk, dv, dm = cott.bwd(dev(c["q"]), dev(c["k"]), dev(c["v"]), dev(d_o), dev(c["m"]), causal=True)
    sub = slice(0, 1)
    rq, rk, rv, _ = oracle.bwd_quadratic(c["q"][sub], c["k"][sub], c["v"][sub], d_o[sub], c["m"], np.full((1,), float(N)), True)
    zero = (c["k"][sub].float().abs().sum(-1) == 0)                 # [1,H,N]
    assert zero.any()
    gate(dq[sub], rq, torch.bfloat16)
    gate(dv[sub], rv, torch.bfloat16)
    keep = ~zero
    gate(dk[sub].cpu()[keep], rk[keep.numpy()], torch.bfloat16)
    # a clamped row's gradient is dk^ / eps: compare row by row on its own scale
    got_z, ref_z = dk[sub].cpu()[zero].double().numpy(), rk[zero.numpy()]
    err = np.abs(got_z - ref_z).max(axis=-1) / np.abs(ref_z).max(axis=-1)
    assert err.max() <= TOL_BF16, f"clamped key rows: {err.max():.3e}"
    assert torch.isfinite(dm).all()


def test_config4_causal_fwd_bwd_bf16():
    c = synth.make_config(4)
    q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
    o = cott.fwd(q, k, v, m, causal=True)
    dq, dk, dv, dm = cott.bwd(q, k, v, d_o, m, causal=True)
    ref_o, _ = oracle.fwd_recurrent(c["q"], c["k"], c["v"], c["m"], None)
    gate(o, ref_o, torch.bfloat16)
    # the definition itself (masked quadratic form) at full size, and the running-sum form beside it
    rq, rk, rv, rm = oracle.bwd_quadratic(c["q"], c["k"], c["v"], c["d_o"], c["m"], None, True)
    gate(dq, rq, torch.bfloat16); gate(dk, rk, torch.bfloat16); gate(dv, rv, torch.bfloat16)
    gate_dm(dm, rm, 1e-2, dm_condition(rv, c["v"], c["m"], None), DM_COND_BF16)
    rq2, rk2, rv2, rm2 = oracle.bwd_recurrent(c["q"], c["k"], c["v"], c["d_o"], c["m"], None)
    for a_, b_ in ((rq2, rq), (rk2, rk), (rv2, rv), (rm2, rm)):
        np.testing.assert_allclose(a_, b_, rtol=1e-9, atol=1e-9 * np.abs(b_).max())
    # second route to dm:  dm_h = <dO,O>_h * (-ln s) sigma(1-sigma), from the oracle's forward
    sg = 1.0 / (1.0 + np.exp(-c["m"].double().numpy()))
    dm2 = (c["d_o"].double().numpy() * ref_o).sum(axis=(0, 2, 3)) * (-np.log(4096.0)) * sg * (1 - sg)
    np.testing.assert_allclose(rm, dm2, rtol=1e-9)


def test_config4_reduced_against_quadratic_definition():
    c = synth.make_qkv(1, 2, 1024, 64, torch.bfloat16, 2004, with_do=True)
    q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
    dq, dk, dv, dm = cott.bwd(q, k, v, d_o, m, causal=True)
    rq, rk, rv, rm = oracle.bwd_quadratic(c["q"], c["k"], c["v"], c["d_o"], c["m"], None, True)
    gate(dq, rq, torch.bfloat16); gate(dk, rk, torch.bfloat16); gate(dv, rv, torch.bfloat16)
    gate_dm(dm, rm, 1e-2, dm_condition(rv, c["v"], c["m"], None), DM_COND_BF16)


@pytest.mark.parametrize("N", synth.C5_SWEEP_N)
def test_config5_long_causal_bf16(N):
    c = synth.make_config(5, N=N)
    o = cott.fwd(dev(c["q"]), dev(c["k"]), dev(c["v"]), dev(c["m"]), causal=True)
    heads = slice(0, 16) if N <= 16384 else slice(3, 7)
    ref, _ = oracle.fwd_recurrent(c["q"][:, heads], c["k"][:, heads], c["v"][:, heads], c["m"][heads], np.array([float(N)]))
    e = gate(o[:, heads], ref, torch.bfloat16)
    print(f"config5 N={N}: normalised max error {e:.3e}")
    plan = cott.query_plan(cott.cott.OP_FWD, cott.cott.BF16, 1, 16, N, 128, True)
    G, C = plan["group"], plan["chunk"]
    rows = sorted({0, 1, C - 1, C, C + 1, G - 1, G, min(G + 1, N - 1), N // 2, N - 2, N - 1} |
                  set(np.random.default_rng(N).integers(0, N, 245).tolist()))
    rows = [r for r in rows if 0 <= r < N]
    ref_rows = oracle.fwd_rows(c["q"], c["k"], c["v"], c["m"], rows, None, True)
    den = np.abs(ref).max()
    err = np.abs(o[:, :, rows].double().cpu().numpy() - ref_rows).max() / den
    assert err <= TOL_BF16


def test_config5_decode_after_prefill():
    """B=64,H=16,d=128: prefill N=8192 through cott_fwd, then 1024 single-token steps.  The
    oracle follows a seeded subset of 16 (b,h) pairs through all 8192+1024 tokens."""
    cfg = synth.C5_DECODE
    B, H, d, N, T = cfg["B"], cfg["H"], cfg["d"], cfg["prefill"], cfg["steps"]
    g = torch.Generator(device="cuda"); g.manual_seed(1005)
    q, k, v = (torch.randn((B, H, N, d), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
               for _ in range(3))
    m = torch.randn((H,), generator=g, device="cuda", dtype=torch.float32)
    o, state = cott.fwd(q, k, v, m, causal=True, return_state=True)
    sq, sk, sv = synth.make_decode_steps(B, H, d, T, torch.bfloat16, 1006)
    rng = np.random.default_rng(1007)
    pairs = [(int(rng.integers(0, B)), int(rng.integers(0, H))) for _ in range(16)]
    state0 = state.clone()
    outs = []
    dq_, dk_, dv_ = sq.cuda(), sk.cuda(), sv.cuda()
    for t in range(T):
        outs.append(cott.decode_step(dq_[t], dk_[t], dv_[t], state, m, float(N)))
    outs = torch.stack(outs)  # [T,B,H,d]
    for (b, h) in pairs:
        qq = torch.cat([q[b, h].cpu(), sq[:, b, h]])[None, None]
        kk = torch.cat([k[b, h].cpu(), sk[:, b, h]])[None, None]
        vv = torch.cat([v[b, h].cpu(), sv[:, b, h]])[None, None]
        mm = m[h:h + 1].cpu()
        ref, ref_state = oracle.fwd_recurrent(qq, kk, vv, mm, np.array([float(N)]))
        assert norm_max_err(o[b, h], ref[0, 0, :N]) <= TOL_BF16
        assert norm_max_err(outs[:, b, h], ref[0, 0, N:]) <= TOL_BF16
        _, ref_state0 = oracle.fwd_recurrent(qq[:, :, :N], kk[:, :, :N], vv[:, :, :N], mm, np.array([float(N)]))
        assert norm_max_err(state0[b, h], ref_state0[0, 0]) <= TOL_STATE_TC
        assert norm_max_err(state[b, h], ref_state[0, 0]) <= TOL_STATE_TC


# ------------------------------------------------------------------ bit-exact index / mask logic
@pytest.mark.parametrize("dtype,d", [(torch.bfloat16, 64), (torch.bfloat16, 128), (torch.float32, 32)])
def test_exact_integer_boundaries(dtype, d, force_group):
    dt = cott.cott.BF16 if dtype == torch.bfloat16 else cott.cott.F32
    force_group(256)
    plan = cott.query_plan(cott.cott.OP_FWD, dt, 1, 2, 4096, d, True)
    G, C = plan["group"], plan["chunk"]
    one = torch.tensor([1.0], device="cuda")
    for N in sorted({1, 2, C - 1, C, C + 1, G - 1, G, G + 1, 2 * G, 3 * G + 5}):
        c = synth.make_onehot_case(1, 2, N, d, dtype, 3000 + N)
        for causal in (True, False):
            o = cott.fwd(dev(c["q"]), dev(c["k"]), dev(c["v"]), dev(c["m"]), seq_len=one, causal=causal)
            ref = oracle.fwd_quadratic(c["q"], c["k"], c["v"], c["m"], np.array([1.0]), causal)
            assert np.array_equal(ref, np.round(ref))
            assert np.array_equal(o.double().cpu().numpy(), ref), (N, causal)


def test_staircase_shows_inclusive_diagonal():
    N, d = 40, 32
    q = torch.zeros((1, 1, N, d)); q[..., 0] = 1.0
    k = q.clone()
    v = torch.zeros((1, 1, N, d))
    v[0, 0, torch.arange(N), torch.arange(N) % d] = 1.0
    m = torch.zeros((1,))
    o = cott.fwd(dev(q), dev(k), dev(v), dev(m), seq_len=1.0, causal=True).cpu()
    expect = torch.cumsum(v, dim=2)  # token t sees itself: o_0 = e_0
    assert torch.equal(o, expect)


# ------------------------------------------------------------------ small shapes, every path
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("d", [32, 64, 128])
@pytest.mark.parametrize("causal", [True, False])
def test_forward_backward_small(dtype, d, causal, force_group):
    force_group(64)  # several groups: exercises the partial-state scan
    B, H, N = 2, 3, 203  # ragged: not a multiple of any tile
    c = synth.make_qkv(B, H, N, d, dtype, 4000 + d, row_lognormal=True, with_do=True)
    s = torch.tensor([float(N), 150.0])
    args = [dev(c[x]) for x in ("q", "k", "v")]
    o, st = cott.fwd(*args, dev(c["m"]), seq_len=dev(s), causal=causal, return_state=True)
    ref = oracle.fwd_quadratic(c["q"], c["k"], c["v"], c["m"], s, causal)
    gate(o, ref, dtype)
    _, ref_state = oracle.fwd_bidir_assoc(c["q"], c["k"], c["v"], c["m"], s)
    assert norm_max_err(st, ref_state) <= state_tol(dtype, d)
    dq, dk, dv, dm = cott.bwd(*args, dev(c["d_o"]), dev(c["m"]), seq_len=dev(s), causal=causal)
    rq, rk, rv, rm = oracle.bwd_quadratic(c["q"], c["k"], c["v"], c["d_o"], c["m"], s, causal)
    gate(dq, rq, dtype); gate(dk, rk, dtype); gate(dv, rv, dtype)
    f32 = dtype == torch.float32
    gate_dm(dm, rm, 1e-4 if f32 else 1e-2, dm_condition(rv, c["v"], c["m"], s), DM_COND_F32 if f32 else DM_COND_BF16)


def test_backward_d128_several_chunks_per_group(force_group):
    """d = 128 gradient streams with groups of several chunks and a ragged tail: the two-stage
    ring, the projection tile in the A slot and the separate Bv barrier all cycle."""
    force_group(512)
    B, H, N, d = 1, 2, 1061, 128
    c = synth.make_qkv(B, H, N, d, torch.bfloat16, 4500, with_do=True)
    args = [dev(c[x]) for x in ("q", "k", "v")]
    o = cott.fwd(*args, dev(c["m"]), causal=True)
    gate(o, oracle.fwd_quadratic(c["q"], c["k"], c["v"], c["m"], None, True), torch.bfloat16)
    dq, dk, dv, dm = cott.bwd(*args, dev(c["d_o"]), dev(c["m"]), causal=True)
    rq, rk, rv, rm = oracle.bwd_quadratic(c["q"], c["k"], c["v"], c["d_o"], c["m"], None, True)
    gate(dq, rq, torch.bfloat16); gate(dk, rk, torch.bfloat16); gate(dv, rv, torch.bfloat16)
    gate_dm(dm, rm, 1e-2, dm_condition(rv, c["v"], c["m"], None), DM_COND_BF16)


def test_single_token_and_single_head():
    c = synth.make_qkv(1, 1, 1, 64, torch.float32, 4100, with_do=True)
    o = cott.fwd(dev(c["q"]), dev(c["k"]), dev(c["v"]), dev(c["m"]), causal=True)
    ref = oracle.fwd_quadratic(c["q"], c["k"], c["v"], c["m"], None, True)  # o_0 = c (q^.k^) v_0
    gate(o, ref, torch.float32)


def test_zero_query_rows_and_clamped_gradient():
    c = synth.make_qkv(1, 2, 50, 32, torch.float32, 4200, with_do=True)
    c["q"][0, 0, 7] = 0.0
    c["k"][0, 1, 9] = 0.0
    args = [dev(c[x]) for x in ("q", "k", "v")]
    o = cott.fwd(*args, dev(c["m"]), causal=True)
    assert torch.equal(o[0, 0, 7], torch.zeros(32, device="cuda"))
    dq, dk, dv, dm = cott.bwd(*args, dev(c["d_o"]), dev(c["m"]), causal=True)
    rq, rk, rv, rm = oracle.bwd_quadratic(c["q"], c["k"], c["v"], c["d_o"], c["m"], None, True)
    # clamped rows carry gradients of order 1e12: compare them relatively, the rest with the gate
    np.testing.assert_allclose(dq[0, 0, 7].cpu().numpy(), rq[0, 0, 7], rtol=1e-4)
    np.testing.assert_allclose(dk[0, 1, 9].cpu().numpy(), rk[0, 1, 9], rtol=1e-4)
    mask = torch.ones((1, 2, 50), dtype=torch.bool); mask[0, 0, 7] = False
    gate(dq.cpu()[mask], rq[mask.numpy()], torch.float32)
    mask = torch.ones((1, 2, 50), dtype=torch.bool); mask[0, 1, 9] = False
    gate(dk.cpu()[mask], rk[mask.numpy()], torch.float32)
    gate(dv, rv, torch.float32)


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("group", [256, 4096])
def test_clamped_gradient_on_tensor_core_path(d, causal, group, force_group):
    """bf16 through the tcgen05 kernels with one exactly-zero query row and one exactly-zero key
    row (in different chunks and groups): the forward gives a zero output row for the zero
    query; the gradient of a clamped row is the derivative of the clamped formula, dx = dx^ / eps
    (order 1e12), compared relatively; every other row passes the usual gate.  With several groups
    per (b, h) and with one (at d = 64 the one-launch bidirectional kernels)."""
    force_group(group)
    B, H, N = 1, 2, 700
    c = synth.make_qkv(B, H, N, d, torch.bfloat16, 4250 + d, with_do=True)
    c["q"][0, 0, 131] = 0.0
    c["k"][0, 1, 517] = 0.0
    args = [dev(c[x]) for x in ("q", "k", "v")]
    o = cott.fwd(*args, dev(c["m"]), causal=causal)
    assert torch.equal(o[0, 0, 131], torch.zeros(d, dtype=torch.bfloat16, device="cuda"))
    gate(o, oracle.fwd_quadratic(c["q"], c["k"], c["v"], c["m"], None, causal), torch.bfloat16)
    dq, dk, dv, dm = cott.bwd(*args, dev(c["d_o"]), dev(c["m"]), causal=causal)
    rq, rk, rv, rm = oracle.bwd_quadratic(c["q"], c["k"], c["v"], c["d_o"], c["m"], None, causal)
    assert np.abs(rq[0, 0, 131]).max() > 1e10 and np.abs(rk[0, 1, 517]).max() > 1e10
    for got, want in ((dq[0, 0, 131], rq[0, 0, 131]), (dk[0, 1, 517], rk[0, 1, 517])):
        e = norm_max_err(got, want)
        print(f"clamped row: normalised error {e:.3e}")
        assert e <= TOL_BF16
    mq = torch.ones((B, H, N), dtype=torch.bool); mq[0, 0, 131] = False
    mk = torch.ones((B, H, N), dtype=torch.bool); mk[0, 1, 517] = False
    gate(dq.cpu()[mq], rq[mq.numpy()], torch.bfloat16)
    gate(dk.cpu()[mk], rk[mk.numpy()], torch.bfloat16)
    gate(dv, rv, torch.bfloat16)
    gate_dm(dm, rm, 1e-2, dm_condition(rv, c["v"], c["m"], None), DM_COND_BF16)


def test_clamped_gradient_in_a_packed_batch():
    """The same in a packed variable-length batch: a zero query row and a zero key row inside
    sequences that share tiles with their neighbours."""
    H, d, lens = 2, 64, (200, 333)
    seqs = [synth.make_qkv(1, H, L, d, torch.bfloat16, 4290 + L, with_do=True) for L in lens]
    for s_ in seqs:
        s_["m"] = seqs[0]["m"]
    seqs[0]["q"][0, 1, 150] = 0.0
    seqs[1]["k"][0, 0, 40] = 0.0
    cat = lambda key: torch.cat([s_[key][0].permute(1, 0, 2) for s_ in seqs], dim=0).contiguous().cuda()
    q, k, v, d_o = (cat(x) for x in ("q", "k", "v", "d_o"))
    cu = torch.tensor([0, 200, 533], dtype=torch.int32, device="cuda")
    m = dev(seqs[0]["m"])
    dq, dk, dv, dm = cott.bwd_varlen(q, k, v, d_o, m, cu, 333, causal=True)
    off = 0
    for i, (s_, L) in enumerate(zip(seqs, lens)):
        rq, rk, rv, _ = oracle.bwd_quadratic(s_["q"], s_["k"], s_["v"], s_["d_o"], s_["m"], None, True)
        un = lambda x: x[off:off + L].permute(1, 0, 2)[None].cpu()
        mq = torch.ones((1, H, L), dtype=torch.bool); mk = mq.clone()
        if i == 0:
            mq[0, 1, 150] = False
            assert np.abs(rq[0, 1, 150]).max() > 1e10
            assert norm_max_err(un(dq)[0, 1, 150], rq[0, 1, 150]) <= TOL_BF16
        else:
            mk[0, 0, 40] = False
            assert np.abs(rk[0, 0, 40]).max() > 1e10
            assert norm_max_err(un(dk)[0, 0, 40], rk[0, 0, 40]) <= TOL_BF16
        gate(un(dq)[mq], rq[mq.numpy()], torch.bfloat16)
        gate(un(dk)[mk], rk[mk.numpy()], torch.bfloat16)
        gate(un(dv), rv, torch.bfloat16)
        off += L


def test_causality_bitwise(force_group):
    force_group(128)
    c = synth.make_qkv(1, 2, 300, 64, torch.bfloat16, 4300)
    o = cott.fwd(dev(c["q"]), dev(c["k"]), dev(c["v"]), dev(c["m"]), seq_len=300.0, causal=True)
    c2 = {x: c[x].clone() for x in ("q", "k", "v")}
    for x in c2.values():
        x[:, :, 200:] = 3.0
    o2 = cott.fwd(dev(c2["q"]), dev(c2["k"]), dev(c2["v"]), dev(c["m"]), seq_len=300.0, causal=True)
    assert torch.equal(o[:, :, :200], o2[:, :, :200])  # later tokens cannot change earlier rows


@pytest.mark.parametrize("B", [1, 4])   # B = 4: the dQ and dK streams run side by side
def test_run_to_run_determinism(B):
    c = synth.make_config(4, B=B)
    q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
    a = cott.bwd(q, k, v, d_o, m, causal=True)
    b = cott.bwd(q, k, v, d_o, m, causal=True)
    for x, y in zip(a, b):
        assert torch.equal(x, y)


# ------------------------------------------------------------------ decode step
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("d", [32, 64, 128])
def test_decode_matches_longer_forward(dtype, d):
    B, H, N, T = 2, 3, 70, 9
    c = synth.make_qkv(B, H, N + T, d, dtype, 5000 + d)
    q, k, v, m = (dev(c[x]) for x in ("q", "k", "v", "m"))
    s = torch.tensor([100.0, 64.0], device="cuda")
    full = oracle.fwd_quadratic(c["q"], c["k"], c["v"], c["m"], s.cpu(), True)
    _, state = cott.fwd(q[:, :, :N].contiguous(), k[:, :, :N].contiguous(), v[:, :, :N].contiguous(), m,
                        seq_len=s, causal=True, return_state=True)
    saved = None
    for t in range(N, N + T):
        o = cott.decode_step(q[:, :, t].contiguous(), k[:, :, t].contiguous(), v[:, :, t].contiguous(), state, m, s)
        gate(o, full[:, :, t], dtype)
        if t == N + 3:
            saved = state.clone()
    # checkpoint / resume: restoring a saved state and replaying gives identical bits
    resumed = saved.clone()
    for t in range(N + 4, N + T):
        o2 = cott.decode_step(q[:, :, t].contiguous(), k[:, :, t].contiguous(), v[:, :, t].contiguous(), resumed, m, s)
    assert torch.equal(resumed, state) and torch.equal(o2, o)
    _, ref_state = oracle.fwd_recurrent(c["q"], c["k"], c["v"], c["m"], s.cpu())
    assert norm_max_err(state, ref_state) <= state_tol(dtype, d)


def test_calls_on_a_stream_that_is_not_current():
    """Outputs and workspace the binding allocates belong to the stream the kernels run on (the
    caching allocator must not recycle them for work on the current stream meanwhile); results
    equal the call on the current stream, also after the library's own streams were destroyed
    and created again (cott_shutdown)."""
    c = synth.make_config(4, B=2, N=1024)
    q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
    want_o = cott.fwd(q, k, v, m, causal=True)
    want_g = cott.bwd(q, k, v, d_o, m, causal=True)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    for _ in range(3):
        o = cott.fwd(q, k, v, m, causal=True, stream=side)
        junk = [torch.randn(1 << 22, device="cuda") for _ in range(4)]     # allocator pressure on the current stream
        g = cott.bwd(q, k, v, d_o, m, causal=True, stream=side)
        del junk
    side.synchronize()
    assert torch.equal(o, want_o) and all(torch.equal(a, b) for a, b in zip(g, want_g))
    cott.cott.shutdown()
    g2 = cott.bwd(q, k, v, d_o, m, causal=True)
    torch.cuda.synchronize()
    assert all(torch.equal(a, b) for a, b in zip(g2, want_g))


# ------------------------------------------------------------------ host-buffer entry point
def test_fwd_bwd_host_matches_the_oracle():
    c = synth.make_config(4, B=1, N=512)
    host = {x: c[x].pin_memory() for x in ("q", "k", "v", "d_o", "m")}
    outs = {x: torch.empty_like(c["q"]).pin_memory() for x in ("o", "dq", "dk", "dv")}
    dm = torch.empty(16, dtype=torch.float32).pin_memory()
    cott.fwd_bwd_host(host["q"], host["k"], host["v"], host["d_o"], host["m"], outs["o"], outs["dq"],
                      outs["dk"], outs["dv"], dm, causal=True)
    torch.cuda.synchronize()
    ref_o = oracle.fwd_quadratic(c["q"], c["k"], c["v"], c["m"], None, True)
    rq, rk, rv, rm = oracle.bwd_quadratic(c["q"], c["k"], c["v"], c["d_o"], c["m"], None, True)
    gate(outs["o"], ref_o, torch.bfloat16)
    gate(outs["dq"], rq, torch.bfloat16); gate(outs["dk"], rk, torch.bfloat16); gate(outs["dv"], rv, torch.bfloat16)
    gate_dm(dm, rm, 1e-2, dm_condition(rv, c["v"], c["m"], None), DM_COND_BF16)


@pytest.mark.parametrize("B", [3, 20])
def test_fwd_bwd_host_slices_match_device_calls_per_slice(B):
    """The host step runs the batch in slices (B = 3: sixteen heads in four groups per batch item;
    B = 20: two batch items per slice), copies in both directions overlapping the compute; every
    slice's rows equal the device calls on that slice bit for bit, dm is the sum of the slices'
    dm in slice order; two calls in a row on one arena agree."""
    N = 640 if B == 3 else 256
    c = synth.make_config(4, B=B, N=N)
    H = 16
    sl = cott.cott.host_step_slicing(B, H)
    assert sl["n"] <= 16 and (sl["items"] == 1 or sl["heads"] == H)
    host = {x: c[x].pin_memory() for x in ("q", "k", "v", "d_o", "m")}
    outs = {x: torch.empty_like(c["q"]).pin_memory() for x in ("o", "dq", "dk", "dv")}
    dm = torch.empty(H, dtype=torch.float32).pin_memory()
    m = dev(c["m"])
    arena = None
    for _ in range(2):
        for t in outs.values():
            t.fill_(float("nan"))
        arena = cott.fwd_bwd_host(host["q"], host["k"], host["v"], host["d_o"], host["m"], outs["o"], outs["dq"],
                                  outs["dk"], outs["dv"], dm, causal=True, arena=arena)
        torch.cuda.synchronize()
        dm_rows = []
        for b0 in range(0, B, sl["items"]):
            row = torch.zeros(H, dtype=torch.float32, device="cuda")
            for h0 in range(0, H, sl["heads"]):
                cut = (slice(b0, b0 + sl["items"]), slice(h0, h0 + sl["heads"]))
                q, k, v, d_o = (dev(c[x][cut].contiguous()) for x in ("q", "k", "v", "d_o"))
                o = cott.fwd(q, k, v, m[cut[1]].contiguous(), seq_len=float(N), causal=True)
                dq, dk, dv, dm_s = cott.bwd(q, k, v, d_o, m[cut[1]].contiguous(), seq_len=float(N), causal=True)
                for name, t in (("o", o), ("dq", dq), ("dk", dk), ("dv", dv)):
                    assert torch.equal(outs[name][cut], t.cpu()), (name, b0, h0)
                row[cut[1]] = dm_s
            dm_rows.append(row)
        dm_sum = torch.zeros(H, dtype=torch.float32, device="cuda")
        for row in dm_rows:
            dm_sum = dm_sum + row
        assert torch.equal(dm, dm_sum.cpu())


# ------------------------------------------------------------------ library services
def test_profile_and_status_words():
    """Per-launch timing of the walk kernels, the launch counter and the status read-back."""
    c = synth.make_config(4, B=1)
    q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
    B, H, N, d = q.shape
    ws = torch.zeros(cott.workspace_bytes(cott.cott.OP_BWD, cott.cott.BF16, B, H, N, d, True),
                     dtype=torch.uint8, device="cuda")
    ws[:16] = 0xFF        # stale status words from "an earlier user" of the memory
    n0 = cott.cott.launch_count()
    cott.cott.profile_enable(64)
    cott.fwd(q, k, v, m, causal=True, workspace=ws)
    cott.bwd(q, k, v, d_o, m, causal=True, workspace=ws)
    rec = cott.cott.profile_read()
    cott.cott.profile_enable(0)
    kinds = [kd for kd, _ in rec]
    assert kinds.count(1) == 1 and kinds.count(3) == 1     # forward walk, fused backward walk
    assert kinds.count(0) == 2                             # a partial-state pass in front of each
    assert all(0.0 < ms < 50.0 for _, ms in rec)
    assert cott.cott.launch_count() - n0 >= len(rec)
    assert cott.cott.last_async_status(ws) == 0            # the first kernel of a call clears the words
    assert int(ws[:12].view(torch.int32).abs().sum()) == 0
    assert cott.cott.profile_read() == []                  # disabled


@pytest.mark.parametrize("B,H,N", [(2, 20, 1024), (4, 16, 1000), (1, 64, 2048)])
def test_backward_reuses_the_forward_calls_partial_states(B, H, N):
    """A training step: the causal forward leaves the per-group partial states K^^T V in its
    workspace, and cott_bwd_after_fwd reads them (transposed) instead of streaming k and v once
    more.  Gradients against the definition, and against the plain backward call."""
    c = synth.make_qkv(B, H, N, 64, torch.bfloat16, 4700 + N + H, with_do=True)
    q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
    plan = cott.cott.query_plan(cott.cott.OP_BWD, cott.cott.BF16, B, H, N, 64, True)
    assert plan["group"] < N                                  # several groups per (b, h)
    ws_f = torch.zeros(cott.workspace_bytes(cott.cott.OP_FWD, cott.cott.BF16, B, H, N, 64, True), dtype=torch.uint8, device="cuda")
    o = cott.fwd(q, k, v, m, causal=True, workspace=ws_f)
    gate(o, oracle.fwd_quadratic(c["q"], c["k"], c["v"], c["m"], None, True), torch.bfloat16)
    n0 = cott.cott.launch_count()
    got = cott.bwd(q, k, v, d_o, m, causal=True, fwd_workspace=ws_f)
    assert cott.cott.launch_count() - n0 == 2                # state pass (q, dO only) + walk
    rq, rk, rv, rm = oracle.bwd_quadratic(c["q"], c["k"], c["v"], c["d_o"], c["m"], None, True)
    gate(got[0], rq, torch.bfloat16); gate(got[1], rk, torch.bfloat16); gate(got[2], rv, torch.bfloat16)
    gate_dm(got[3], rm, 1e-2, dm_condition(rv, c["v"], c["m"], None), DM_COND_BF16)
    plain = cott.bwd(q, k, v, d_o, m, causal=True)
    for a, b in zip(got[:3], plain[:3]):
        assert norm_max_err(a, b.double().cpu().numpy()) <= TOL_BF16  # the same sums in another order, each rounded to bf16 once


def test_side_by_side_backward_matches_one_after_the_other(option):
    """B*H = 64: the dQ and dK streams run side by side, each over the whole sequence.  Same
    gradients (up to the rounding of a different grouping) as the three streams in sequence,
    also with a ragged last chunk."""
    for N in (4096, 1000):
        c = synth.make_qkv(4, 16, N, 64, torch.bfloat16, 4600 + N, with_do=True)
        q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
        option("fused_bwd", 0)
        option("pair", 1)
        a = cott.bwd(q, k, v, d_o, m, causal=True)
        option("pair", 0)
        b = cott.bwd(q, k, v, d_o, m, causal=True)
        for x, y in zip(a[:3], b[:3]):
            assert norm_max_err(x, y.double().cpu().numpy()) <= TOL_BF16
        torch.testing.assert_close(a[3], b[3], rtol=2e-2, atol=2e-2 * float(b[3].abs().max()))
    # and against the definition on a slice of the ragged case
    sub = slice(0, 1)
    rq, rk, rv, _ = oracle.bwd_quadratic(c["q"][sub], c["k"][sub], c["v"][sub], c["d_o"][sub], c["m"], None, True)
    option("pair", 1)
    dq, dk, dv, _ = cott.bwd(q, k, v, d_o, m, causal=True)
    gate(dq[sub], rq, torch.bfloat16); gate(dk[sub], rk, torch.bfloat16); gate(dv[sub], rv, torch.bfloat16)


# ------------------------------------------------------------------ stateful continuation (Eq. 8 across calls)
@pytest.mark.parametrize("dtype,d", [(torch.bfloat16, 64), (torch.bfloat16, 128), (torch.float32, 32)])
def test_segments_equal_one_long_forward(dtype, d, force_group):
    """A sequence fed in segments through cott_fwd_stateful -- cuts at chunk and group
    boundaries, next to them, and a ragged tail -- gives the rows of the definition over the
    whole sequence, and the state left by the last segment is c K^^T V of all of it."""
    force_group(256)
    B, H, N = 2, 2, 1000
    c = synth.make_qkv(B, H, N, d, dtype, 4700 + d)
    s_b = torch.tensor([float(N), 600.0])
    ref = oracle.fwd_quadratic(c["q"], c["k"], c["v"], c["m"], s_b, True)
    _, ref_state = oracle.fwd_bidir_assoc(c["q"], c["k"], c["v"], c["m"], s_b)
    q, k, v, m, s_dev = (dev(x) for x in (c["q"], c["k"], c["v"], c["m"], s_b))
    for cuts in ([0, 1000], [0, 128, 256, 257, 511, 900, 1000], [0, 1, 2, 129, 1000]):
        state, outs = None, []
        for a, b in zip(cuts[:-1], cuts[1:]):
            o, state = cott.fwd_stateful(q[:, :, a:b].contiguous(), k[:, :, a:b].contiguous(),
                                         v[:, :, a:b].contiguous(), m, s_dev, state_in=state)
            outs.append(o)
        gate(torch.cat(outs, dim=2), ref, dtype)
        assert norm_max_err(state, ref_state) <= state_tol(dtype, d)


def test_segment_continues_decode_state():
    """prefill (cott_fwd) -> a few decode steps -> a segment (cott_fwd_stateful) -> decode
    again: every row equals the row of one long causal forward."""
    B, H, d, N = 2, 3, 64, 640
    c = synth.make_qkv(B, H, N, d, torch.bfloat16, 4800)
    ref = oracle.fwd_quadratic(c["q"], c["k"], c["v"], c["m"], np.full((B,), float(N)), True)
    q, k, v, m = (dev(c[x]) for x in ("q", "k", "v", "m"))
    rows = []
    o, state = cott.fwd(q[:, :, :300].contiguous(), k[:, :, :300].contiguous(), v[:, :, :300].contiguous(),
                        m, seq_len=float(N), causal=True, return_state=True)
    rows.append(o)
    for t in range(300, 303):
        rows.append(cott.decode_step(q[:, :, t].contiguous(), k[:, :, t].contiguous(), v[:, :, t].contiguous(),
                                     state, m, float(N)).unsqueeze(2))
    o, state = cott.fwd_stateful(q[:, :, 303:639].contiguous(), k[:, :, 303:639].contiguous(),
                                 v[:, :, 303:639].contiguous(), m, float(N), state_in=state)
    rows.append(o)
    rows.append(cott.decode_step(q[:, :, 639].contiguous(), k[:, :, 639].contiguous(), v[:, :, 639].contiguous(),
                                 state, m, float(N)).unsqueeze(2))
    gate(torch.cat(rows, dim=2), ref, torch.bfloat16)


def test_stateful_argument_checks():
    c = synth.make_qkv(1, 1, 64, 64, torch.bfloat16, 4900)
    q, k, v, m = (dev(c[x]) for x in ("q", "k", "v", "m"))
    with pytest.raises(ValueError):
        cott.fwd_stateful(q, k, v, m, None)
    with pytest.raises(cott.CottError):
        cott.fwd_stateful(q, k, v, m, 0.5)           # scaling base below 1


# ------------------------------------------------------------------ many calls in a row
@pytest.mark.parametrize("shape", [(4, 16, 4096, 64), (1, 16, 4096, 128), (2, 4, 1152, 128), (3, 5, 700, 64)])
def test_repeated_calls_are_bit_identical(shape):
    """The kernels are pipelines of asynchronous roles; a timing-dependent hazard would show as
    a result that changes from call to call.  200 forward+backward calls in a row, issued
    without synchronising in between, must reproduce the first call bit for bit."""
    B, H, N, d = shape
    c = synth.make_qkv(B, H, N, d, torch.bfloat16, 5000 + N + d, with_do=True)
    q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
    ws_f = torch.zeros(cott.workspace_bytes(cott.cott.OP_FWD, cott.cott.BF16, B, H, N, d, True),
                       dtype=torch.uint8, device="cuda")
    ws_b = torch.zeros(cott.workspace_bytes(cott.cott.OP_BWD, cott.cott.BF16, B, H, N, d, True),
                       dtype=torch.uint8, device="cuda")
    first = None
    acc = torch.zeros(5, dtype=torch.int64, device="cuda")     # mismatching elements per tensor
    for it in range(200):
        o = cott.fwd(q, k, v, m, causal=True, workspace=ws_f)
        dq, dk, dv, dm = cott.bwd(q, k, v, d_o, m, causal=True, workspace=ws_b)
        outs = (o, dq, dk, dv, dm)
        if first is None:
            first = tuple(x.clone() for x in outs)
        else:
            acc += torch.stack([(x != y).sum() for x, y in zip(outs, first)])
    assert cott.cott.last_async_status(ws_f) == 0 and cott.cott.last_async_status(ws_b) == 0
    assert acc.tolist() == [0, 0, 0, 0, 0]
    assert all(torch.isfinite(x.float()).all() for x in first)


@pytest.mark.parametrize("B", [13, 32])
def test_bidirectional_backward_many_heads(B):
    """Bidirectional gradients at the BERT-base shape (B = 32: config 2 at full size, as bench.py's
    c2-train times it) and with a ragged number of (b, h) pairs: more pairs than CTA slots, one
    group of four chunks per CTA through the one-launch backward."""
    H, N, d = 12, 512, 64
    c = synth.make_qkv(B, H, N, d, torch.bfloat16, 5100, with_do=True)
    q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
    dq, dk, dv, dm = cott.bwd(q, k, v, d_o, m, causal=False)
    sub = slice(0, 2)        # the definition on the first two batch items
    rq, rk, rv, _ = oracle.bwd_quadratic(c["q"][sub], c["k"][sub], c["v"][sub], c["d_o"][sub], c["m"], None, False)
    gate(dq[sub], rq, torch.bfloat16); gate(dk[sub], rk, torch.bfloat16); gate(dv[sub], rv, torch.bfloat16)
    # dm sums over the batch: both routes on the GPU result (dm_h = sum_b <dO,O> dc/dm / c)
    o = cott.fwd(q, k, v, m, causal=False)
    sg = torch.sigmoid(m.double())
    route2 = (d_o.double() * o.double()).sum(dim=(0, 2, 3)) * (-np.log(float(N))) * sg * (1 - sg)
    torch.testing.assert_close(dm.double(), route2, rtol=5e-2, atol=5e-2 * float(route2.abs().max()))


@pytest.mark.parametrize("one_launch", [1, 0])
@pytest.mark.parametrize("shape", [(2, 3, 1, 64, 64), (2, 3, 127, 64, 64), (3, 5, 128, 64, 64), (2, 4, 129, 64, 64),
                                   (2, 7, 640, 64, 64), (1, 3, 1024, 64, 64), (2, 3, 300, 32, 64), (2, 3, 300, 64, 40),
                                   (2, 2, 200, 24, 16)])
def test_bidirectional_backward_both_forms(shape, one_launch, option, force_group):
    """The bidirectional backward at head sizes up to 64 with one group per (b, h): in one launch
    (both state totals, then the gradient rows; dm from the element-wise product of the totals)
    and as a state pass followed by the walk -- every gradient of both against the definition, dm at
    the strict gate, on chunk-count boundaries, a ragged last chunk and key / value sizes of their
    own."""
    B, H, N, dk, dv = shape
    c = synth.make_qkv(B, H, N, dk, torch.bfloat16, 6100 + N + dk + dv, with_do=True, d_v=dv)
    q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
    option("bidir_bwd", one_launch)
    force_group(4096)
    n0 = cott.cott.launch_count()
    dq, dk_, dv_, dm = cott.bwd(q, k, v, d_o, m, causal=False)
    assert cott.cott.launch_count() - n0 == (1 if one_launch else 2)
    rq, rk, rv, rm = oracle.bwd_quadratic(c["q"], c["k"], c["v"], c["d_o"], c["m"], None, False)
    gate(dq, rq, torch.bfloat16); gate(dk_, rk, torch.bfloat16); gate(dv_, rv, torch.bfloat16)
    gate_dm(dm, rm, 1e-2, dm_condition(rv, c["v"], c["m"], None), DM_COND_BF16)


def test_bidirectional_backward_one_launch_in_a_fused_buffer(force_group):
    """The one-launch bidirectional backward reads q, k, v from a fused [B, N, 3, H, d] projection
    output and writes dq, dk, dv into one: bit-identical to the dense call."""
    B, H, N, d = 2, 4, 333, 64
    c = synth.make_qkv(B, H, N, d, torch.bfloat16, 6200, with_do=True)
    q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
    force_group(4096)
    n0 = cott.cott.launch_count()
    want = cott.bwd(q, k, v, d_o, m, causal=False)
    assert cott.cott.launch_count() - n0 == 1
    fused = torch.stack([q.permute(0, 2, 1, 3), k.permute(0, 2, 1, 3), v.permute(0, 2, 1, 3)], dim=2).contiguous()   # [B,N,3,H,d]
    qs, ks, vs = (fused[:, :, i].permute(0, 2, 1, 3) for i in range(3))
    grads = torch.full_like(fused, 7.0)
    outs = tuple(grads[:, :, i].permute(0, 2, 1, 3) for i in range(3))
    d_o_bnhd = d_o.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    got = cott.bwd(qs, ks, vs, d_o_bnhd, m, causal=False, out=outs)
    for x, y in zip(got[:3], want[:3]):
        assert torch.equal(x, y)
    torch.testing.assert_close(got[3], want[3], rtol=0, atol=0)


# ------------------------------------------------------------------ seeded sweep over shapes
def _sweep_cases():
    rng = np.random.RandomState(77)
    cases = []
    for i in range(14):
        d = int(rng.choice([32, 64, 128]))
        dtype = torch.float32 if d == 32 and rng.rand() < 0.7 else torch.bfloat16
        B = int(rng.randint(1, 5)); H = int(rng.randint(1, 20))
        N = int(rng.choice([1, 2, 63, 127, 128, 129, 255, 300, 511, 640, 777]))
        cases.append((B, H, N, d, dtype, bool(rng.rand() < 0.75), i))
    return cases


@pytest.mark.parametrize("case", _sweep_cases(), ids=lambda c: f"B{c[0]}H{c[1]}N{c[2]}d{c[3]}{'bf16' if c[4] == torch.bfloat16 else 'f32'}{'c' if c[5] else 'b'}")
def test_shape_sweep_forward_backward(case):
    """Seeded sweep over batch, heads, length, head size, dtype and masking with the library's
    own plan (no forced group): forward, exported state and all gradients against the
    definition."""
    B, H, N, d, dtype, causal, i = case
    c = synth.make_qkv(B, H, N, d, dtype, 5200 + i, with_do=True)
    args = [dev(c[x]) for x in ("q", "k", "v")]
    o, st = cott.fwd(*args, dev(c["m"]), causal=causal, return_state=True)
    gate(o, oracle.fwd_quadratic(c["q"], c["k"], c["v"], c["m"], None, causal), dtype)
    _, ref_state = oracle.fwd_bidir_assoc(c["q"], c["k"], c["v"], c["m"], None)
    assert norm_max_err(st, ref_state) <= state_tol(dtype, d)
    dq, dk, dv, dm = cott.bwd(*args, dev(c["d_o"]), dev(c["m"]), causal=causal)
    rq, rk, rv, rm = oracle.bwd_quadratic(c["q"], c["k"], c["v"], c["d_o"], c["m"], None, causal)
    gate(dq, rq, dtype); gate(dk, rk, dtype); gate(dv, rv, dtype)
    f32 = dtype == torch.float32
    gate_dm(dm, rm, 1e-4 if f32 else 1e-2, dm_condition(rv, c["v"], c["m"], None), DM_COND_F32 if f32 else DM_COND_BF16)


@pytest.mark.parametrize("N", [128, 129, 256, 257, 384, 513])
@pytest.mark.parametrize("pair", ["fused", "1", "0"])
def test_chunk_count_boundaries_d64(N, pair, option):
    """One to five chunks per walk at d = 64, where the ring of three stages, the two raw-row
    buffers of the gradient epilogues and the output buffers start, wrap and drain: forward and
    all gradients against the definition, with the dK and dV streams side by side and one after
    the other."""
    option("fused_bwd", 1 if pair == "fused" else 0)
    option("pair", 0 if pair == "0" else 1)
    c = synth.make_qkv(2, 20, N, 64, torch.bfloat16, 5400 + N, with_do=True)
    q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
    o = cott.fwd(q, k, v, m, causal=True)
    gate(o, oracle.fwd_quadratic(c["q"], c["k"], c["v"], c["m"], None, True), torch.bfloat16)
    dq, dk, dv, dm = cott.bwd(q, k, v, d_o, m, causal=True)
    rq, rk, rv, rm = oracle.bwd_quadratic(c["q"], c["k"], c["v"], c["d_o"], c["m"], None, True)
    gate(dq, rq, torch.bfloat16); gate(dk, rk, torch.bfloat16); gate(dv, rv, torch.bfloat16)
    gate_dm(dm, rm, 1e-2, dm_condition(rv, c["v"], c["m"], None), DM_COND_BF16)


@pytest.mark.parametrize("N", [1, 127, 128, 129, 256, 300, 384, 513, 640, 897, 1100])
@pytest.mark.parametrize("fused", [1, 0])
def test_chunk_count_boundaries_bidirectional_d64(N, fused, option, force_group):
    """One to nine chunks through the one-launch bidirectional forward (two stages of (k, v)
    pairs, four q slots, two output tiles: every ring starts, wraps and drains, with an odd and
    an even number of chunks and a ragged last one) and through the two-launch form it replaces:
    rows and the exported state against the definition."""
    option("fused_bidir", fused)
    option("short_fwd", 0)           # (N <= 128 without a state export would take the short-sequence kernel)
    force_group(4096)
    c = synth.make_qkv(3, 7, N, 64, torch.bfloat16, 5500 + N)
    q, k, v, m = (dev(c[x]) for x in ("q", "k", "v", "m"))
    cott.cott.profile_enable(8)
    o, st = cott.fwd(q, k, v, m, causal=False, return_state=True)
    kinds = [kd for kd, _ in cott.cott.profile_read()]
    cott.cott.profile_enable(0)
    assert kinds == ([4] if fused else [0, 2])             # one launch / state pass + read-out
    gate(o, oracle.fwd_quadratic(c["q"], c["k"], c["v"], c["m"], None, False), torch.bfloat16)
    _, ref_state = oracle.fwd_bidir_assoc(c["q"], c["k"], c["v"], c["m"], None)
    assert norm_max_err(st, ref_state) <= state_tol(torch.bfloat16, 64)
    o2 = cott.fwd(q, k, v, m, causal=False)
    assert torch.equal(o2, o)


# ------------------------------------------------------------------ short sequences
@pytest.mark.parametrize("N", [1, 2, 7, 16, 33, 64, 65, 100, 128])
@pytest.mark.parametrize("dk,dv", [(64, 64), (128, 128), (32, 96)])
@pytest.mark.parametrize("causal", [True, False])
def test_short_sequences_take_the_quadratic_side(N, dk, dv, causal, option):
    """Sequences of at most 128 tokens in dense tensors: one launch of the quadratic form with
    floor(128 / N) sequences of consecutive (b, h) pairs per tile and a block-diagonal mask --
    no state.  21 pairs, so the last tile is partly empty; every row against the definition,
    and the same call through the generic walk for comparison."""
    B, H = 3, 7
    c = synth.make_qkv(B, H, N, dk, torch.bfloat16, 6600 + N + dk, d_v=dv)
    q, k, v, m = (dev(c[x]) for x in ("q", "k", "v", "m"))
    s = torch.tensor([float(N), 50.0, 300.0], device="cuda")
    ref = oracle.fwd_quadratic(c["q"], c["k"], c["v"], c["m"], s.cpu().numpy().astype(np.float64), causal)
    cott.cott.profile_enable(8)
    o = cott.fwd(q, k, v, m, seq_len=s, causal=causal)
    kinds = [kd for kd, _ in cott.cott.profile_read()]
    cott.cott.profile_enable(0)
    assert kinds == [5]
    gate(o, ref, torch.bfloat16)
    option("short_fwd", 0)
    o_walk = cott.fwd(q, k, v, m, seq_len=s, causal=causal)
    gate(o_walk, ref, torch.bfloat16)
    # neighbours in a tile do not leak into each other: changing one pair's rows changes only its output
    if N <= 64:
        option("short_fwd", 1)
        k2 = k.clone(); k2[1, 2] = -k2[1, 2]
        o2 = cott.fwd(q, k2, v, m, seq_len=s, causal=causal)
        same = torch.ones((B, H), dtype=torch.bool); same[1, 2] = False
        assert torch.equal(o2[same.cuda()], o[same.cuda()])
        assert not torch.equal(o2[1, 2], o[1, 2])


@pytest.mark.parametrize("T", [1, 5, 16, 33, 64])
@pytest.mark.parametrize("dk,dv", [(128, 128), (64, 64), (96, 40)])
def test_token_blocks_on_a_state(T, dk, dv, option):
    """Blocks of at most 64 tokens on a caller-held state take a kernel of their own (several
    CTAs per SM, the state read and written once): prefill 200 tokens, then three blocks of T
    tokens; rows and the final [d_key, d_value] state against one long causal forward by the
    definition; more (b, h) pairs than fit on the GPU at once."""
    # (d = 128: more than two pairs per SM, which takes the persistent form of the kernel)
    B, H, N0 = (10 if dk == 128 else 5), 40, 200
    N = N0 + 3 * T
    c = synth.make_qkv(B, H, N, dk, torch.bfloat16, 6700 + T + dk, d_v=dv)
    s = np.full((B,), float(N))
    q, k, v, m = (dev(c[x]) for x in ("q", "k", "v", "m"))
    seg = lambda x, a, b: x[:, :, a:b].contiguous()
    o0, state = cott.fwd(seg(q, 0, N0), seg(k, 0, N0), seg(v, 0, N0), m, seq_len=float(N), causal=True, return_state=True)
    rows = [o0]
    for i in range(3):
        a, b = N0 + i * T, N0 + (i + 1) * T
        cott.cott.profile_enable(8)
        o, state = cott.fwd_stateful(seg(q, a, b), seg(k, a, b), seg(v, a, b), m, float(N), state_in=state)
        kinds = [kd for kd, _ in cott.cott.profile_read()]
        cott.cott.profile_enable(0)
        assert kinds == [6]
        rows.append(o)
    # a sample of (b, h) pairs through the oracle (the whole batch would take a minute)
    pick = [(0, 0), (2, 17), (4, 39), (B - 1, 38)]
    sub = {x: np.stack([c[x][b_, h_].float().numpy() for b_, h_ in pick])[None] for x in ("q", "k", "v")}
    msub = np.array([float(c["m"][h_]) for _, h_ in pick])
    ref = oracle.fwd_quadratic(sub["q"], sub["k"], sub["v"], msub, np.array([float(N)]), True)[0]
    _, ref_state = oracle.fwd_recurrent(sub["q"], sub["k"], sub["v"], msub, np.array([float(N)]))
    got = torch.cat(rows, dim=2)
    got_sub = torch.stack([got[b_, h_] for b_, h_ in pick])
    gate(got_sub, ref, torch.bfloat16)
    st_sub = torch.stack([state[b_, h_] for b_, h_ in pick])
    assert norm_max_err(st_sub, ref_state[0]) <= state_tol(torch.bfloat16, max(dk, dv))
    # the same blocks through the generic walk agree
    option("block_fwd", 0)
    o_w, st_w = cott.fwd_stateful(seg(q, N - T, N), seg(k, N - T, N), seg(v, N - T, N), m, float(N),
                                  state_in=state.clone())
    option("block_fwd", 1)
    o_b, st_b = cott.fwd_stateful(seg(q, N - T, N), seg(k, N - T, N), seg(v, N - T, N), m, float(N),
                                  state_in=state.clone())
    assert norm_max_err(o_b, o_w.double().cpu().numpy()) <= TOL_BF16
    assert norm_max_err(st_b, st_w.double().cpu().numpy()) <= 1e-3
    # the block read in place from the long tensors (rows N - T .. N - 1 of every (b, h)) and
    # written into a [B,T,H,d] buffer: bit-identical to the call on contiguous copies
    out_bthd = torch.empty((B, T, H, dv), dtype=torch.bfloat16, device="cuda").permute(0, 2, 1, 3)
    o_s, st_s = cott.fwd_stateful(q[:, :, N - T:], k[:, :, N - T:], v[:, :, N - T:], m, float(N),
                                  state_in=state.clone(), out=out_bthd)
    assert not q[:, :, N - T:].is_contiguous() or T == N
    assert torch.equal(o_s, o_b) and torch.equal(st_s, st_b)


# ------------------------------------------------------------------ head sizes (d_key, d_value)
HEAD_SIZES = [(32, 32), (96, 96), (64, 128), (128, 64), (32, 64), (40, 72), (8, 16), (128, 32), (72, 8)]


@pytest.mark.parametrize("dk,dv", HEAD_SIZES)
@pytest.mark.parametrize("causal", [True, False])
def test_head_sizes_forward_backward(dk, dv, causal):
    """Key and value sizes of their own, and sizes between the kernels' 64 and 128 (bf16, any
    multiple of 8 up to 128): forward with the exported [d_key, d_value] state and all
    gradients against the definition; several groups per (b, h) and a ragged last chunk."""
    B, H, N = 2, 3, 333
    c = synth.make_qkv(B, H, N, dk, torch.bfloat16, 6100 + dk * 7 + dv, with_do=True, d_v=dv)
    q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
    plan = cott.cott.query_plan_dkdv(cott.cott.OP_FWD, cott.cott.BF16, B, H, N, dk, dv, causal)
    assert plan["path"] == 1 and plan["kernel_d"] == (64 if max(dk, dv) <= 64 else 128)
    o, st = cott.fwd(q, k, v, m, causal=causal, return_state=True)
    assert o.shape == (B, H, N, dv) and st.shape == (B, H, dk, dv)
    gate(o, oracle.fwd_quadratic(c["q"], c["k"], c["v"], c["m"], None, causal), torch.bfloat16)
    _, ref_state = (oracle.fwd_recurrent if causal else oracle.fwd_bidir_assoc)(c["q"], c["k"], c["v"], c["m"], None)
    assert norm_max_err(st, ref_state) <= state_tol(torch.bfloat16, max(dk, dv))
    dq, dk_, dv_, dm = cott.bwd(q, k, v, d_o, m, causal=causal)
    assert dq.shape == q.shape and dk_.shape == k.shape and dv_.shape == v.shape
    rq, rk, rv, rm = oracle.bwd_quadratic(c["q"], c["k"], c["v"], c["d_o"], c["m"], None, causal)
    gate(dq, rq, torch.bfloat16); gate(dk_, rk, torch.bfloat16); gate(dv_, rv, torch.bfloat16)
    gate_dm(dm, rm, 1e-2, dm_condition(rv, c["v"], c["m"], None), DM_COND_BF16)


@pytest.mark.parametrize("dk,dv", [(64, 128), (96, 96), (32, 32), (40, 72)])
def test_head_sizes_groups_segments_and_decode(dk, dv, force_group):
    """The same sizes through several groups per (b, h) with a state scan, through segments
    that hand a [d_key, d_value] state on (a padded copy inside the library), and through
    decode steps: all rows equal one long causal forward by the definition."""
    force_group(256)
    B, H, N = 2, 2, 700
    c = synth.make_qkv(B, H, N + 3, dk, torch.bfloat16, 6300 + dk + dv, d_v=dv)
    s = np.full((B,), float(N + 3))
    ref = oracle.fwd_quadratic(c["q"], c["k"], c["v"], c["m"], s, True)
    _, ref_state = oracle.fwd_recurrent(c["q"], c["k"], c["v"], c["m"], s)
    q, k, v, m = (dev(c[x]) for x in ("q", "k", "v", "m"))
    seg = lambda x, a, b: x[:, :, a:b].contiguous()
    cuts = [0, 300, 301, N]
    o, state = cott.fwd(seg(q, 0, 300), seg(k, 0, 300), seg(v, 0, 300), m, seq_len=float(N + 3), causal=True,
                        return_state=True)
    rows = [o]
    for a, b in zip(cuts[1:-1], cuts[2:]):
        o, state = cott.fwd_stateful(seg(q, a, b), seg(k, a, b), seg(v, a, b), m, float(N + 3), state_in=state)
        rows.append(o)
    for t in range(N, N + 3):
        rows.append(cott.decode_step(q[:, :, t].contiguous(), k[:, :, t].contiguous(), v[:, :, t].contiguous(),
                                     state, m, float(N + 3)).unsqueeze(2))
    gate(torch.cat(rows, dim=2), ref, torch.bfloat16)
    assert state.shape == (B, H, dk, dv)
    assert norm_max_err(state, ref_state) <= state_tol(torch.bfloat16, max(dk, dv))


def test_head_sizes_in_a_fused_projection_buffer():
    """q, k (48 columns) and v (80 columns) as slices of one [B,N,H,48+48+80] projection output,
    gradients written into the slices of a buffer of the same shape: bit-identical to the call
    on dense copies (which the test above gates against the definition)."""
    B, H, N, dk, dv = 2, 3, 200, 48, 80
    c = synth.make_qkv(B, H, N, dk, torch.bfloat16, 6500, with_do=True, d_v=dv)
    q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
    o_ref, st_ref = cott.fwd(q, k, v, m, causal=True, return_state=True)
    g_ref = cott.bwd(q, k, v, d_o, m, causal=True)
    gate(o_ref, oracle.fwd_quadratic(c["q"], c["k"], c["v"], c["m"], None, True), torch.bfloat16)
    W = 2 * dk + dv
    fused = torch.cat([x.permute(0, 2, 1, 3) for x in (q, k, v)], dim=3).contiguous()        # [B,N,H,W]
    qf, kf, vf = (fused[..., a:b].permute(0, 2, 1, 3) for a, b in ((0, dk), (dk, 2 * dk), (2 * dk, W)))
    assert qf.stride() == (N * H * W, W, H * W, 1) and not vf.is_contiguous()
    o2, st2 = cott.fwd(qf, kf, vf, m, causal=True, return_state=True)
    assert torch.equal(o2, o_ref) and torch.equal(st2, st_ref)
    gbuf = torch.full_like(fused, float("nan"))
    outs = tuple(gbuf[..., a:b].permute(0, 2, 1, 3) for a, b in ((0, dk), (dk, 2 * dk), (2 * dk, W)))
    g2 = cott.bwd(qf, kf, vf, d_o, m, causal=True, out=outs)
    for a, b in zip(g2, g_ref):
        assert torch.equal(a, b)
    assert not torch.isnan(gbuf.float()).any()             # every column of the buffer was written


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("dk,dv", [(48, 80), (256, 64), (20, 12)])
def test_decode_step_any_head_sizes(dtype, dk, dv):
    """The decode step for sizes its specialised kernel does not cover: three steps in a row
    against the oracle's step, state carried."""
    if dtype == torch.bfloat16 and (dk % 8 or dv % 8):
        dk, dv = 24, 16          # bf16 rows must be multiples of 16 bytes
    B, H = 3, 5
    g = torch.Generator().manual_seed(6400 + dk + dv)
    m = torch.randn((H,), generator=g)
    state = torch.zeros((B, H, dk, dv), dtype=torch.float32, device="cuda")
    ref_state = np.zeros((B, H, dk, dv))
    for step in range(3):
        q, k = (torch.randn((B, H, dk), generator=g).to(dtype) for _ in range(2))
        v = torch.randn((B, H, dv), generator=g).to(dtype)
        o = cott.decode_step(dev(q), dev(k), dev(v), state, dev(m), 50.0)
        ref = oracle.decode_step(q, k, v, m, 50.0, ref_state)
        gate(o, ref, dtype)
    tol = 1e-2 if dtype == torch.bfloat16 else 1e-5
    assert norm_max_err(state, ref_state) <= tol


@pytest.mark.parametrize("dtype,d", [(torch.bfloat16, 128), (torch.bfloat16, 64), (torch.float32, 32)])
def test_short_blocks_many_heads(dtype, d):
    """More (b,h) pairs than SMs and blocks of a few tokens (the shape of tokens between decode
    steps): prefill, then blocks of 1, 7, 32 and 20 tokens through cott_fwd_stateful; every row
    equals the row of one long causal forward."""
    B, H, N0 = 10, 16, 100
    cuts = [N0, N0 + 1, N0 + 8, N0 + 40, N0 + 60]
    N = cuts[-1]
    c = synth.make_qkv(B, H, N, d, dtype, 5300 + d)
    ref = oracle.fwd_quadratic(c["q"], c["k"], c["v"], c["m"], np.full((B,), float(N)), True)
    _, ref_state = oracle.fwd_bidir_assoc(c["q"], c["k"], c["v"], c["m"], np.full((B,), float(N)))
    q, k, v, m = (dev(c[x]) for x in ("q", "k", "v", "m"))
    seg = lambda x, a, b: x[:, :, a:b].contiguous()
    o, state = cott.fwd(seg(q, 0, N0), seg(k, 0, N0), seg(v, 0, N0), m, seq_len=float(N), causal=True, return_state=True)
    rows = [o]
    for a, b in zip(cuts[:-1], cuts[1:]):
        o, state = cott.fwd_stateful(seg(q, a, b), seg(k, a, b), seg(v, a, b), m, float(N), state_in=state)
        rows.append(o)
    gate(torch.cat(rows, dim=2), ref, dtype)
    assert norm_max_err(state, ref_state) <= state_tol(dtype, d)
    # a block with no state to start from is a short causal forward
    o0 = cott.fwd_stateful(seg(q, 0, 9), seg(k, 0, 9), seg(v, 0, 9), m, float(N), return_state=False)
    gate(o0, ref[:, :, :9], dtype)


# ------------------------------------------------------------------ stream capture
@pytest.mark.parametrize("causal", [True, False])
def test_a_training_step_can_be_captured_in_a_cuda_graph(causal):
    """cott_fwd and cott_bwd with caller-owned outputs and workspaces issue only kernels (and one
    memset) on the caller's stream: captured once in a CUDA graph and replayed, the step gives the
    bits of the eager calls."""
    B, H, N, d = 2, 6, 1500, 64
    c = synth.make_qkv(B, H, N, d, torch.bfloat16, 6900, with_do=True)
    q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
    o = torch.empty_like(q)
    outs = tuple(torch.empty_like(q) for _ in range(3))
    wf = torch.zeros(cott.workspace_bytes(cott.cott.OP_FWD, cott.cott.BF16, B, H, N, d, causal), dtype=torch.uint8, device="cuda")
    wb = torch.zeros(cott.workspace_bytes(cott.cott.OP_BWD, cott.cott.BF16, B, H, N, d, causal), dtype=torch.uint8, device="cuda")

    def step():
        cott.fwd(q, k, v, m, causal=causal, out=o, workspace=wf)
        return cott.bwd(q, k, v, d_o, m, causal=causal, out=outs, workspace=wb)

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for _ in range(2):
            step()                       # (first calls configure the kernels: outside the capture)
    torch.cuda.synchronize()
    ref = [t.clone() for t in step()] + [o.clone()]
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        res = step()
    torch.cuda.synchronize()
    for t in outs + (o,):
        t.zero_()
    res[3].zero_()
    graph.replay()
    torch.cuda.synchronize()
    for got, want in zip(list(res) + [o], ref):
        assert torch.equal(got, want)
    assert cott.cott.last_async_status(wf) == 0 and cott.cott.last_async_status(wb) == 0


# ------------------------------------------------------------------ backward of segments
@pytest.mark.parametrize("shape", [(2, 3, 200, 64, 64, 0), (1, 2, 1000, 64, 64, 256), (2, 2, 77, 32, 64, 0),
                                   (1, 3, 300, 48, 24, 128), (2, 2, 128, 64, 64, 0)])
def test_segment_backward_matches_the_definition(shape, force_group):
    """cott_bwd_stateful on a segment with a caller's incoming state and a gradient flowing into the
    outgoing one: dq, dk, dv, the gradient of the incoming state and dm against the definition
    (states scaled like a real history: state_in from a forward over earlier tokens), with one and
    with several groups, key / value sizes of their own, a single chunk."""
    B, H, N, dk, dv, group = shape
    if group:
        force_group(group)
    hist = synth.make_qkv(B, H, 150, dk, torch.bfloat16, 6300 + N, d_v=dv)
    c = synth.make_qkv(B, H, N, dk, torch.bfloat16, 6400 + N + dk + dv, with_do=True, d_v=dv)
    c["m"] = hist["m"]
    s = np.full((B,), float(N + 150))
    zero = np.zeros((B, H, dk, dv))
    _, st_in = oracle.fwd_segment(hist["q"], hist["k"], hist["v"], hist["m"], zero, s)
    d_st_out = np.random.default_rng(6500 + N).standard_normal((B, H, dk, dv)) * 0.5
    rq, rk, rv, rst, rm = oracle.bwd_segment(c["q"], c["k"], c["v"], c["d_o"], c["m"], st_in, d_st_out, s)
    q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
    f32 = lambda a: torch.tensor(a, dtype=torch.float32, device="cuda")
    dq, dk_, dv_, dst, dm = cott.bwd_stateful(q, k, v, d_o, m, float(N + 150), state_in=f32(st_in), d_state_out=f32(d_st_out))
    gate(dq, rq, torch.bfloat16); gate(dk_, rk, torch.bfloat16); gate(dv_, rv, torch.bfloat16)
    assert norm_max_err(dst, rst) <= TOL_STATE_TC    # (q^ enters the sum rounded to bf16, like every tensor-core state)
    gate_dm(dm, rm, 1e-2, dm_condition(rv, c["v"], c["m"], s), DM_COND_BF16)
    # without states it is the plain causal backward
    a = cott.bwd_stateful(q, k, v, d_o, m, float(N + 150), return_d_state=False)
    b = cott.bwd(q, k, v, d_o, m, seq_len=float(N + 150), causal=True)
    for x, y in zip(a[:3], b[:3]):
        assert float((x.float() - y.float()).abs().max()) <= TOL_BF16 * float(y.float().abs().max())


@pytest.mark.parametrize("d", [64, 128])
def test_segment_backwards_chain_to_the_whole_sequence(d):
    """Three segments forward (cott_fwd_stateful), then backward last to first with the state
    gradients handed on: the gradients of one backward over the whole sequence (the definition),
    dm the sum of the segments' parts."""
    B, H, N = 2, 4, 900
    cuts = [(0, 256), (256, 600), (600, 900)]
    c = synth.make_qkv(B, H, N, d, torch.bfloat16, 6600, with_do=True)
    q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
    seg = lambda x, a, b: x[:, :, a:b].contiguous()
    states = [None]
    for a, b in cuts:
        _, st = cott.fwd_stateful(seg(q, a, b), seg(k, a, b), seg(v, a, b), m, float(N), state_in=states[-1])
        states.append(st)
    d_state = None
    grads = []
    dm = torch.zeros(H, device="cuda")
    for (a, b), st_in in reversed(list(zip(cuts, states[:-1]))):
        g = cott.bwd_stateful(seg(q, a, b), seg(k, a, b), seg(v, a, b), seg(d_o, a, b), m, float(N),
                              state_in=st_in, d_state_out=d_state)
        grads.append(g[:3])
        d_state = g[3]
        dm += g[4]
    grads.reverse()
    rq, rk, rv, rm = oracle.bwd_quadratic(c["q"], c["k"], c["v"], c["d_o"], c["m"], None, True)
    for i, ref in enumerate((rq, rk, rv)):
        gate(torch.cat([g[i] for g in grads], dim=2), ref, torch.bfloat16)
    gate_dm(dm, rm, 1e-2, dm_condition(rv, c["v"], c["m"], None), DM_COND_BF16)


@pytest.mark.parametrize("case", [(torch.float32, 32, 150, 0, 1), (torch.float32, 64, 300, 64, 1), (torch.float32, 128, 90, 0, 1),
                                  (torch.bfloat16, 128, 400, 128, 0),
                                  (torch.bfloat16, 128, 400, 128, 1), (torch.bfloat16, 128, 1000, 4096, 1), (torch.bfloat16, 128, 130, 0, 1)])
def test_segment_backward_through_three_walks(case, force_group, option):
    """cott_bwd_stateful where the one-walk tensor-core backward does not reach -- three running-sum
    walks whose sums start from the caller's state (transposed), the transposed gradient of the
    outgoing state and that gradient itself: the fp32-accumulating kernels for fp32 I/O (and, with
    force_path = 0, bf16), the tensor-core walks for bf16 at head size 128 (several groups, one
    group, a ragged second chunk), where the totals of two streams give the gradient of the
    incoming state and correct the dm sum."""
    dtype, d, N, group, tensor_cores = case
    if group:
        force_group(group)
    if not tensor_cores:
        option("force_path", 0)
    B, H = 2, 3
    hist = synth.make_qkv(B, H, 100, d, dtype, 6800 + d)
    c = synth.make_qkv(B, H, N, d, dtype, 6810 + d + N, with_do=True)
    c["m"] = hist["m"]
    s = np.full((B,), float(N + 100))
    _, st_in = oracle.fwd_segment(hist["q"], hist["k"], hist["v"], hist["m"], np.zeros((B, H, d, d)), s)
    d_st_out = np.random.default_rng(6820 + d).standard_normal((B, H, d, d)) * 0.5
    rq, rk, rv, rst, rm = oracle.bwd_segment(c["q"], c["k"], c["v"], c["d_o"], c["m"], st_in, d_st_out, s)
    q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
    f32 = lambda a: torch.tensor(a, dtype=torch.float32, device="cuda")
    dq, dk_, dv_, dst, dm = cott.bwd_stateful(q, k, v, d_o, m, float(N + 100), state_in=f32(st_in), d_state_out=f32(d_st_out))
    gate(dq, rq, dtype); gate(dk_, rk, dtype); gate(dv_, rv, dtype)
    assert norm_max_err(dst, rst) <= (TOL_STATE_F32 if dtype == torch.float32 else TOL_STATE_TC)
    if dtype == torch.float32:
        gate_dm(dm, rm, 1e-4, dm_condition(rv, c["v"], c["m"], s), DM_COND_F32)
    else:
        gate_dm(dm, rm, 1e-2, dm_condition(rv, c["v"], c["m"], s), DM_COND_BF16)


@pytest.mark.parametrize("sizes", [(96, 96, 300, 128), (64, 128, 500, 4096), (128, 40, 260, 0), (72, 88, 130, 0)])
def test_segment_backward_head_sizes_above_64(sizes, force_group):
    """cott_bwd_stateful at bf16 head sizes that run in the kernels of size 128 (zero-filled
    tiles): the caller's [d_k, d_v] states enter and leave through padded copies."""
    dk, dv, N, group = sizes
    if group:
        force_group(group)
    B, H = 2, 3
    hist = synth.make_qkv(B, H, 90, dk, torch.bfloat16, 6850 + dk, d_v=dv)
    c = synth.make_qkv(B, H, N, dk, torch.bfloat16, 6860 + dk + dv, with_do=True, d_v=dv)
    c["m"] = hist["m"]
    s = np.full((B,), float(N + 90))
    _, st_in = oracle.fwd_segment(hist["q"], hist["k"], hist["v"], hist["m"], np.zeros((B, H, dk, dv)), s)
    d_st_out = np.random.default_rng(6870 + dk).standard_normal((B, H, dk, dv)) * 0.5
    rq, rk, rv, rst, rm = oracle.bwd_segment(c["q"], c["k"], c["v"], c["d_o"], c["m"], st_in, d_st_out, s)
    q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
    f32 = lambda a: torch.tensor(a, dtype=torch.float32, device="cuda")
    dq, dk_, dv_, dst, dm = cott.bwd_stateful(q, k, v, d_o, m, float(N + 90), state_in=f32(st_in), d_state_out=f32(d_st_out))
    gate(dq, rq, torch.bfloat16); gate(dk_, rk, torch.bfloat16); gate(dv_, rv, torch.bfloat16)
    assert norm_max_err(dst, rst) <= TOL_STATE_TC
    gate_dm(dm, rm, 1e-2, dm_condition(rv, c["v"], c["m"], s), DM_COND_BF16)


@pytest.mark.parametrize("dtype,d", [(torch.bfloat16, 64), (torch.bfloat16, 128), (torch.float32, 32)])
def test_segment_backward_strided_matches_dense(dtype, d):
    """cott_bwd_stateful_strided: q, k, v, dO stored [B,N,H,d] and gradients written into a fused
    [B,N,3,H,d] buffer give the bits of the dense call."""
    B, H, N = 2, 5, 333
    c = synth.make_qkv(B, H, N, d, dtype, 6950 + d, with_do=True)
    q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
    g = torch.Generator(device="cuda"); g.manual_seed(9)
    st_in = torch.randn((B, H, d, d), generator=g, device="cuda")
    d_st_out = torch.randn((B, H, d, d), generator=g, device="cuda")
    want = cott.bwd_stateful(q, k, v, d_o, m, 1000.0, state_in=st_in, d_state_out=d_st_out)
    qs, ks, vs, dos = (_as_bnhd(x) for x in (q, k, v, d_o))
    grads = torch.full((B, N, 3, H, d), 7.0, dtype=dtype, device="cuda")
    outs = tuple(grads[:, :, i].permute(0, 2, 1, 3) for i in range(3))
    got = cott.bwd_stateful(qs, ks, vs, dos, m, 1000.0, state_in=st_in, d_state_out=d_st_out, out=outs)
    for x, y in zip(got[:3], want[:3]):
        assert torch.equal(x, y)
    assert torch.equal(got[3], want[3])
    torch.testing.assert_close(got[4], want[4], rtol=0, atol=0)


def test_segment_backward_refuses_what_it_does_not_cover():
    c = synth.make_qkv(1, 2, 64, 32, torch.float32, 6700, with_do=True)
    q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
    wide = torch.zeros((1, 2, 64, 48), dtype=torch.float32, device="cuda")
    with pytest.raises(cott.CottError):
        cott.bwd_stateful(wide, wide.clone(), wide.clone(), wide.clone(), m, 64.0)   # fp32 covers 32 / 64 / 128 only
    c = synth.make_qkv(1, 2, 64, 64, torch.bfloat16, 6701, with_do=True)
    q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
    with pytest.raises(cott.CottError):
        cott.bwd_stateful(q, k, v, d_o, m, None)                     # no scaling base


# ------------------------------------------------------------------ a wait that runs out
@pytest.mark.parametrize("op", ["fwd", "bwd", "bidir", "bidir_bwd", "bidir_bwd_walk", "short", "block"])
def test_bounded_wait_runs_out_and_reports(op, option, force_group):
    """Every device-side wait has a bound.  With the bound set to zero a wait gives up unless
    its hand-off is there within a few polls -- and the first tiles of a kernel cannot come
    from memory that fast, so a wait is certain to run out.  The kernel then reports where,
    lets its copies in flight land, frees its tensor memory and returns; the context stays
    usable and the next call is correct.  (No GPU fault is involved: the kernels end normally.)
    One case per warp-specialised kernel: the generic walk, the fused backward (causal and
    bidirectional instance), the one-launch bidirectional backward, the bidirectional, the
    short-sequence and the block forward."""
    causal = op not in ("bidir", "bidir_bwd", "bidir_bwd_walk")
    force_group(512 if causal else 4096)
    if op == "bidir_bwd_walk":
        option("bidir_bwd", 0)
    N = {"short": 64, "block": 16}.get(op, 1024)
    c = synth.make_qkv(1, 2, N, 64, torch.bfloat16, 5400, with_do=True)
    q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
    is_bwd = op in ("bwd", "bidir_bwd", "bidir_bwd_walk")
    code = cott.cott.OP_BWD if is_bwd else cott.cott.OP_FWD
    ws = torch.zeros(cott.workspace_bytes(code, cott.cott.BF16, 1, 2, N, 64, causal),
                     dtype=torch.uint8, device="cuda")
    state0 = torch.zeros((1, 2, 64, 64), dtype=torch.float32, device="cuda")
    if is_bwd:
        call = lambda: cott.bwd(q, k, v, d_o, m, causal=causal, workspace=ws)
    elif op == "block":
        call = lambda: cott.fwd_stateful(q, k, v, m, float(N), state_in=state0, workspace=ws)[0]
    else:
        call = lambda: cott.fwd(q, k, v, m, causal=causal, workspace=ws)
    option("wait_limit_kcycles", 0)
    call()
    assert cott.cott.last_async_status(ws) == -5                 # COTT_ERR_TIMEOUT
    words = ws[:12].view(torch.int32).cpu().numpy().view(np.uint32)
    assert words[0] == 1 and (words[1] >> 31) == 1               # where the first wait gave up
    assert ((words[1] >> 4) & 0x3FF) < 512                       # a barrier of the kernel's block
    option("wait_limit_kcycles", -1)
    out = call()
    assert cott.cott.last_async_status(ws) == 0
    if not is_bwd:
        gate(out, oracle.fwd_quadratic(c["q"], c["k"], c["v"], c["m"], None, causal), torch.bfloat16)
    else:
        rq, rk, rv, _ = oracle.bwd_quadratic(c["q"], c["k"], c["v"], c["d_o"], c["m"], None, causal)
        gate(out[0], rq, torch.bfloat16); gate(out[1], rk, torch.bfloat16); gate(out[2], rv, torch.bfloat16)


# ------------------------------------------------------------------ tensors that are not dense [B,H,N,d]
def _as_bnhd(x):
    """The same values stored as [B,N,H,d], seen as [B,H,N,d] (what a projection GEMM leaves)."""
    return x.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)


@pytest.mark.parametrize("dtype,d", [(torch.bfloat16, 64), (torch.bfloat16, 128), (torch.float32, 32)])
@pytest.mark.parametrize("causal", [True, False])
def test_strided_layouts_match_dense(dtype, d, causal):
    """[B,N,H,d] storage and the slices of a fused [B,N,3,H,d] projection output, read and
    written in place: bit-identical to the same call on dense [B,H,N,d] copies (the arithmetic
    does not depend on where the rows sit), forward, exported state and all gradients; and the
    dense result itself against the definition."""
    B, H, N = 2, 5, 333
    c = synth.make_qkv(B, H, N, d, dtype, 5600 + d, with_do=True)
    q, k, v, d_o, m = (dev(c[x]) for x in ("q", "k", "v", "d_o", "m"))
    o_ref, st_ref = cott.fwd(q, k, v, m, causal=causal, return_state=True)
    g_ref = cott.bwd(q, k, v, d_o, m, causal=causal)
    gate(o_ref, oracle.fwd_quadratic(c["q"], c["k"], c["v"], c["m"], None, causal), dtype)

    # (1) [B,N,H,d] storage for everything, outputs included (empty_like keeps the strides)
    qb, kb, vb, dob = (_as_bnhd(x) for x in (q, k, v, d_o))
    assert not qb.is_contiguous()
    o1, st1 = cott.fwd(qb, kb, vb, m, causal=causal, return_state=True)
    assert o1.stride() == qb.stride()
    assert torch.equal(o1, o_ref) and torch.equal(st1, st_ref)
    g1 = cott.bwd(qb, kb, vb, dob, m, causal=causal)
    for a, b in zip(g1, g_ref):
        assert torch.equal(a, b)

    # (2) fused projection output [B,N,3,H,d]; gradients into a fused buffer of the same shape;
    #     o and dO dense [B,H,N,d]
    fused = torch.stack([x.permute(0, 2, 1, 3) for x in (q, k, v)], dim=2).contiguous()   # [B,N,3,H,d]
    qf, kf, vf = (fused[:, :, i].permute(0, 2, 1, 3) for i in range(3))
    assert qf.stride() == (N * 3 * H * d, d, 3 * H * d, 1)
    o2 = cott.fwd(qf, kf, vf, m, causal=causal, out=torch.empty_like(q))
    assert torch.equal(o2, o_ref)
    gfused = torch.full_like(fused, float("nan"))
    outs = tuple(gfused[:, :, i].permute(0, 2, 1, 3) for i in range(3))
    g2 = cott.bwd(qf, kf, vf, d_o, m, causal=causal, out=outs)
    for a, b in zip(g2[:3], g_ref[:3]):
        assert torch.equal(a, b)
    assert torch.equal(g2[3], g_ref[3])
    assert torch.isfinite(gfused.float()).all()          # every element of the fused buffer was written


def test_strided_argument_checks():
    """Strides the kernels cannot address are refused, not mis-read: rows that are not
    contiguous, token strides that are not a multiple of 16 bytes."""
    c = synth.make_qkv(1, 2, 64, 64, torch.bfloat16, 5700)
    q, k, v, m = (dev(c[x]) for x in ("q", "k", "v", "m"))
    with pytest.raises(ValueError):
        cott.fwd(q.transpose(2, 3), k.transpose(2, 3), v.transpose(2, 3), m)      # rows not contiguous
    wide = torch.zeros((1, 2, 64, 68), dtype=torch.bfloat16, device="cuda")       # token stride 136 bytes
    with pytest.raises(cott.CottError):
        cott.fwd(wide[..., :64], wide[..., :64], wide[..., :64], m, out=torch.empty_like(q))
    with pytest.raises(ValueError):
        cott.fwd(q, _as_bnhd(k), v, m)                                            # q, k, v must share strides


# ------------------------------------------------------------------ packed variable-length batches
def _pack(c, lens):
    """Rows of the sequences back to back: [total, H, d] from per-sequence [1, H, L, d] arrays."""
    return {k2: torch.cat([torch.from_numpy(np.ascontiguousarray(s[k2][0])).permute(1, 0, 2) for s in c], dim=0)
            for k2 in ("q", "k", "v", "d_o")}


@pytest.mark.parametrize("d", [64, 128, 32, 96])
@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("lens", [(300, 1, 128, 129, 77), (1000, 513), (64,)])
def test_packed_varlen_matches_per_sequence_definition(d, causal, lens):
    """Sequences of different lengths back to back in [total, H, d]: every sequence's rows equal
    the definition evaluated on that sequence alone (scaling base = its own length), forward and
    all gradients; dm is the sum over the sequences.  Rows of a neighbour that share a tile with
    the end of a sequence must neither be attended to nor overwritten."""
    _check_packed_batch(d, causal, lens)


@pytest.mark.parametrize("d", [64, 128, 96])
@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("group", [128, 256])
def test_packed_varlen_with_several_groups_per_sequence(d, causal, group, force_group):
    """A packed batch whose sequences are cut into groups (few long sequences would otherwise leave
    most of the GPU idle): group g of a sequence is its rows g * group .. + group - 1 as far as
    they exist, so sequences have different numbers of groups, some groups end ragged and the
    shortest sequences leave whole groups empty.  Same checks as with one group per sequence."""
    force_group(group)
    _check_packed_batch(d, causal, (650, 1, 256, 257, 129, 900))


@pytest.mark.parametrize("d", [64, 128])
def test_packed_varlen_skewed_batch_uses_finer_groups(d):
    """One long sequence among short ones: with the workspace of cott_workspace_bytes_varlen the
    group size follows the total token count (more, shorter groups than the dense plan for
    max_seqlen), with the dense query's workspace the dense groups -- both against the definition,
    and the finer partition launches more CTAs for the long sequence (a different launch count is
    not required, equal results within the bf16 tolerance are)."""
    H, lens = 8, (3000, 200, 129, 64)
    seqs = [synth.make_qkv(1, H, L, d, torch.bfloat16, 7000 + L, with_do=True) for L in lens]
    for s_ in seqs:
        s_["m"] = seqs[0]["m"]
    cat = lambda key: torch.cat([s_[key][0].permute(1, 0, 2) for s_ in seqs], dim=0).contiguous().cuda()
    q, k, v, d_o = (cat(x) for x in ("q", "k", "v", "d_o"))
    cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32, device="cuda")
    m = dev(seqs[0]["m"])
    B, T, Lmax = len(lens), sum(lens), max(lens)
    results = []
    for fine in (True, False):
        size = (lambda op: cott.workspace_bytes_varlen(op, cott.cott.BF16, B, H, T, Lmax, d, True)) if fine else \
               (lambda op: cott.workspace_bytes(op, cott.cott.BF16, B, H, Lmax, d, True))
        wf = torch.zeros(size(cott.cott.OP_FWD), dtype=torch.uint8, device="cuda")
        wb = torch.zeros(size(cott.cott.OP_BWD), dtype=torch.uint8, device="cuda")
        o = cott.fwd_varlen(q, k, v, m, cu, Lmax, causal=True, workspace=wf)
        g = cott.bwd_varlen(q, k, v, d_o, m, cu, Lmax, causal=True, workspace=wb)
        assert cott.cott.last_async_status(wf) == 0 and cott.cott.last_async_status(wb) == 0
        results.append((o,) + tuple(g))
    off = 0
    for s_, L in zip(seqs, lens):
        ref = oracle.fwd_quadratic(s_["q"], s_["k"], s_["v"], s_["m"], None, True)
        rq, rk, rv, _ = oracle.bwd_quadratic(s_["q"], s_["k"], s_["v"], s_["d_o"], s_["m"], None, True)
        un = lambda x: x[off:off + L].permute(1, 0, 2)[None]
        for r in results:
            gate(un(r[0]), ref, torch.bfloat16)
            gate(un(r[1]), rq, torch.bfloat16); gate(un(r[2]), rk, torch.bfloat16); gate(un(r[3]), rv, torch.bfloat16)
        off += L


def _check_packed_batch(d, causal, lens):
    H = 3
    seqs = [synth.make_qkv(1, H, L, d, torch.bfloat16, 5800 + 7 * i + L, with_do=True) for i, L in enumerate(lens)]
    m_np = seqs[0]["m"]
    for s in seqs:
        s["m"] = m_np
    packed = {k2: v2.to(torch.bfloat16).cuda() for k2, v2 in _pack(
        [{k3: (x.float().numpy() if isinstance(x, torch.Tensor) else x) for k3, x in s.items()} for s in seqs], lens).items()}
    cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32, device="cuda")
    m = dev(m_np)
    o = cott.fwd_varlen(packed["q"], packed["k"], packed["v"], m, cu, max(lens), causal=causal)
    dq, dk, dv, dm = cott.bwd_varlen(packed["q"], packed["k"], packed["v"], packed["d_o"], m, cu, max(lens), causal=causal)
    dm_ref = np.zeros(H)
    conds = np.zeros(H)
    off = 0
    for s, L in zip(seqs, lens):
        ref = oracle.fwd_quadratic(s["q"], s["k"], s["v"], s["m"], None, causal)          # [1,H,L,d]
        rq, rk, rv, rm = oracle.bwd_quadratic(s["q"], s["k"], s["v"], s["d_o"], s["m"], None, causal)
        sl = slice(off, off + L)
        unpack = lambda x: x[sl].permute(1, 0, 2)[None]                                     # [1,H,L,d]
        gate(unpack(o), ref, torch.bfloat16)
        gate(unpack(dq), rq, torch.bfloat16); gate(unpack(dk), rk, torch.bfloat16); gate(unpack(dv), rv, torch.bfloat16)
        dm_ref += rm
        conds += dm_condition(rv, s["v"], s["m"], None)
        off += L
    gate_dm(dm, dm_ref, 1e-2, conds, DM_COND_BF16)


@pytest.mark.parametrize("causal", [True, False])
def test_packed_varlen_fp32(causal):
    """fp32 I/O of a packed batch (the fp32-accumulating SIMT kernels, d = 32): every sequence
    against the definition evaluated on it alone at the fp32 gate; neighbours' rows untouched."""
    H, d, lens = 3, 32, (70, 1, 16, 33)
    seqs = [synth.make_qkv(1, H, L, d, torch.float32, 5900 + 7 * i + L, with_do=True) for i, L in enumerate(lens)]
    m_np = seqs[0]["m"]
    cat = lambda key: torch.cat([s[key][0].permute(1, 0, 2) for s in seqs], dim=0).contiguous().cuda()
    q, k, v, d_o = (cat(x) for x in ("q", "k", "v", "d_o"))
    cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32, device="cuda")
    m = dev(m_np)
    o = cott.fwd_varlen(q, k, v, m, cu, max(lens), causal=causal)
    dq, dk, dv, dm = cott.bwd_varlen(q, k, v, d_o, m, cu, max(lens), causal=causal)
    dm_ref, conds, off = np.zeros(H), np.zeros(H), 0
    for s, L in zip(seqs, lens):
        ref = oracle.fwd_quadratic(s["q"], s["k"], s["v"], m_np, None, causal)
        rq, rk, rv, rm = oracle.bwd_quadratic(s["q"], s["k"], s["v"], s["d_o"], m_np, None, causal)
        unpack = lambda x: x[off:off + L].permute(1, 0, 2)[None]
        gate(unpack(o), ref, torch.float32)
        gate(unpack(dq), rq, torch.float32); gate(unpack(dk), rk, torch.float32); gate(unpack(dv), rv, torch.float32)
        dm_ref += rm
        conds += dm_condition(rv, s["v"], m_np, None)
        off += L
    gate_dm(dm, dm_ref, 1e-4, conds, DM_COND_F32)


def test_packed_varlen_leaves_neighbours_alone():
    """The ragged end of a sequence shares a 128-row tile with the start of the next one: after a
    forward into a buffer filled with a marker, exactly the rows of the batch are written."""
    H, d, lens = 2, 64, (5, 200, 3)
    T = sum(lens)
    g = torch.Generator(device="cuda"); g.manual_seed(3)
    q, k, v = (torch.randn((T + 40, H, d), generator=g, device="cuda").to(torch.bfloat16) for _ in range(3))
    cu = torch.tensor([0, 5, 205, 208], dtype=torch.int32, device="cuda")
    m = torch.zeros(H, device="cuda")
    out = torch.full((T + 40, H, d), 7.0, dtype=torch.bfloat16, device="cuda")
    cott.fwd_varlen(q[:T], k[:T], v[:T], m, cu, 200, out=out[:T])
    assert (out[T:] == 7.0).all()                       # nothing past the batch
    assert not (out[:T] == 7.0).all(dim=-1).any()       # every row of the batch written
    # sequence 1 alone gives the same rows as inside the batch
    cu1 = torch.tensor([0, 200], dtype=torch.int32, device="cuda")
    alone = cott.fwd_varlen(q[5:205].contiguous(), k[5:205].contiguous(), v[5:205].contiguous(), m, cu1, 200)
    assert torch.equal(alone, out[5:205])


@pytest.mark.parametrize("d", [64, 40])
def test_packed_varlen_bidirectional_forward_in_one_launch(d, force_group):
    """A packed bidirectional batch with one group per sequence goes through the one-launch forward
    kernel (d <= 64): every sequence against the definition, exactly the rows of the batch written
    (ragged ends share tiles with the next sequence), an empty sequence in the middle."""
    H, lens = 3, (5, 200, 0, 129, 128, 511)
    force_group(4096)
    seqs = [synth.make_qkv(1, H, L, d, torch.bfloat16, 7100 + L) if L else None for L in lens]
    m_np = seqs[0]["m"]
    cat = lambda key: torch.cat([s_[key][0].permute(1, 0, 2) for s_ in seqs if s_ is not None], dim=0).contiguous().cuda()
    q, k, v = (cat(x) for x in ("q", "k", "v"))
    T = sum(lens)
    cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32, device="cuda")
    out = torch.full((T + 40, H, d), 7.0, dtype=torch.bfloat16, device="cuda")
    n0 = cott.cott.launch_count()
    cott.fwd_varlen(q, k, v, dev(m_np), cu, max(lens), causal=False, out=out[:T])
    assert cott.cott.launch_count() - n0 == 1
    assert (out[T:] == 7.0).all()
    assert not (out[:T] == 7.0).all(dim=-1).any()
    off = 0
    for s_, L in zip(seqs, lens):
        if s_ is None:
            continue
        ref = oracle.fwd_quadratic(s_["q"], s_["k"], s_["v"], m_np, None, False)
        gate(out[off:off + L].permute(1, 0, 2)[None], ref, torch.bfloat16)
        off += L


@pytest.mark.parametrize("causal", [True, False])
def test_packed_varlen_gradients_leave_neighbours_alone(causal, option, force_group):
    """The one-launch backward of a packed batch (d = 64): the rows of a ragged last chunk leave as
    plain stores, so every sequence's gradient rows are, bit for bit, those of the same sequence
    passed alone -- nothing of a neighbour is overwritten or attended to -- and the two backward
    paths (one launch / role-swapped walks) agree within the bf16 tolerance."""
    H, d, lens = 2, 64, (5, 200, 3, 128, 131)
    T = sum(lens)
    force_group(4096)        # (one group per sequence in both calls: the same kernel, the same bits)
    g = torch.Generator(device="cuda"); g.manual_seed(11)
    q, k, v, d_o = (torch.randn((T, H, d), generator=g, device="cuda").to(torch.bfloat16) for _ in range(4))
    m = torch.randn((H,), generator=g, device="cuda")
    cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32, device="cuda")
    grads = cott.bwd_varlen(q, k, v, d_o, m, cu, max(lens), causal=causal)
    dm_sum = torch.zeros_like(grads[3])
    off = 0
    for L in lens:
        sl = slice(off, off + L)
        cu1 = torch.tensor([0, L], dtype=torch.int32, device="cuda")
        # (the scaling base of a sequence is its own length in both calls)
        alone = cott.bwd_varlen(q[sl].contiguous(), k[sl].contiguous(), v[sl].contiguous(), d_o[sl].contiguous(),
                                m, cu1, L, causal=causal)
        for x, y in zip(grads[:3], alone[:3]):
            assert torch.equal(x[sl], y)
        dm_sum += alone[3]
        off += L
    torch.testing.assert_close(grads[3], dm_sum, rtol=1e-4, atol=1e-4 * float(dm_sum.abs().max()))
    option("fused_bwd", 0)
    walks = cott.bwd_varlen(q, k, v, d_o, m, cu, max(lens), causal=causal)
    for x, y in zip(grads[:3], walks[:3]):
        scale = float(y.float().abs().max())
        assert float((x.float() - y.float()).abs().max()) <= TOL_BF16 * scale


@pytest.mark.parametrize("group", [0, 128])
def test_packed_varlen_with_empty_sequences(group, force_group):
    """Sequences of length zero anywhere in the batch: nothing is read or written for them, the
    others are unaffected, and the call reports no error -- with one group per sequence and with
    several (every group of an empty sequence is empty)."""
    if group:
        force_group(group)
    H, d = 2, 64
    g = torch.Generator(device="cuda"); g.manual_seed(5)
    lens = (0, 130, 0, 64, 0)
    T = sum(lens)
    q, k, v, d_o = (torch.randn((T, H, d), generator=g, device="cuda").to(torch.bfloat16) for _ in range(4))
    m = torch.zeros(H, device="cuda")
    cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32, device="cuda")
    cu2 = torch.tensor([0, 130, 194], dtype=torch.int32, device="cuda")
    for causal in (True, False):
        ws = torch.zeros(cott.workspace_bytes(cott.cott.OP_BWD, cott.cott.BF16, len(lens), H, 130, d, causal),
                         dtype=torch.uint8, device="cuda")
        a = cott.fwd_varlen(q, k, v, m, cu, 130, causal=causal, workspace=ws)
        assert cott.cott.last_async_status(ws) == 0
        b = cott.fwd_varlen(q, k, v, m, cu2, 130, causal=causal)
        assert torch.equal(a, b)
        ga = cott.bwd_varlen(q, k, v, d_o, m, cu, 130, causal=causal, workspace=ws)
        assert cott.cott.last_async_status(ws) == 0
        gb = cott.bwd_varlen(q, k, v, d_o, m, cu2, 130, causal=causal)
        for x, y in zip(ga[:3], gb[:3]):
            assert torch.equal(x, y)
        torch.testing.assert_close(ga[3], gb[3], rtol=1e-3, atol=1e-3 * float(gb[3].abs().max()))


def test_packed_varlen_with_given_scaling_bases():
    """Per-sequence scaling bases passed by the caller (sp->seq_len) instead of the lengths."""
    H, d, lens = 2, 64, (150, 260)
    bases = np.array([512.0, 1024.0])
    seqs = [synth.make_qkv(1, H, L, d, torch.bfloat16, 5900 + L, with_do=True) for L in lens]
    for s_ in seqs:
        s_["m"] = seqs[0]["m"]
    cat = lambda key: torch.cat([s_[key][0].permute(1, 0, 2) for s_ in seqs], dim=0).contiguous().cuda()
    q, k, v, d_o = (cat(x) for x in ("q", "k", "v", "d_o"))
    cu = torch.tensor([0, 150, 410], dtype=torch.int32, device="cuda")
    m = dev(seqs[0]["m"])
    sl = torch.tensor(bases, dtype=torch.float32, device="cuda")
    o = cott.fwd_varlen(q, k, v, m, cu, 260, seq_len=sl)
    dq, dk, dv, dm = cott.bwd_varlen(q, k, v, d_o, m, cu, 260, seq_len=sl)
    off, dm_ref, conds = 0, np.zeros(H), np.zeros(H)
    for s_, L, base in zip(seqs, lens, bases):
        sb = np.array([base])
        ref = oracle.fwd_quadratic(s_["q"], s_["k"], s_["v"], s_["m"], sb, True)
        rq, rk, rv, rm = oracle.bwd_quadratic(s_["q"], s_["k"], s_["v"], s_["d_o"], s_["m"], sb, True)
        un = lambda x: x[off:off + L].permute(1, 0, 2)[None]
        gate(un(o), ref, torch.bfloat16)
        gate(un(dq), rq, torch.bfloat16); gate(un(dk), rk, torch.bfloat16); gate(un(dv), rv, torch.bfloat16)
        dm_ref += rm; conds += dm_condition(rv, s_["v"], s_["m"], sb)
        off += L
    gate_dm(dm, dm_ref, 1e-2, conds, DM_COND_BF16)


_FIRST_CALL_SCRIPT = r"""
import sys, torch
sys.path.insert(0, sys.argv[1])
import paper_2409_18747_b200 as cott
from paper_2409_18747_b200 import synth
bad = 0
for (B, H, N, d, causal) in ((2, 5, 333, 128, False), (2, 5, 333, 128, True), (2, 5, 333, 64, False)):
    c = synth.make_qkv(B, H, N, d, torch.bfloat16, 6000 + d, with_do=True)
    q, k, v, d_o, m = (c[x].cuda() for x in ("q", "k", "v", "d_o", "m"))
    runs = []
    for _ in range(4):
        o = cott.fwd(q, k, v, m, causal=causal)
        runs.append((o,) + tuple(cott.bwd(q, k, v, d_o, m, causal=causal)))
    torch.cuda.synchronize()
    bad += sum(not torch.equal(x, y) for r in runs[:-1] for x, y in zip(r, runs[-1]))
print("MISMATCH" if bad else "SAME")
"""


def test_first_calls_of_a_fresh_process_equal_later_ones():
    """The first launches of a process run with cold instruction caches and skewed warps: a
    hand-off that is only ordered by luck shows there first (this caught row scales read before
    they were written).  Six fresh processes; in each, every call must equal the last one bit for bit."""
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    for _ in range(6):
        out = subprocess.run([sys.executable, "-c", _FIRST_CALL_SCRIPT, root], capture_output=True, text=True,
                             timeout=300)
        assert out.returncode == 0, out.stderr[-2000:]
        assert out.stdout.strip().endswith("SAME"), out.stdout[-500:]


@pytest.mark.parametrize("dtype,d", [(torch.bfloat16, 64), (torch.float32, 32)])
def test_stateful_segments_on_strided_tensors(dtype, d):
    """cott_fwd_stateful_strided: segments cut out of [B,N,H,d] storage (views, no copies) give
    the same rows and the same final state, bit for bit, as contiguous copies of the segments."""
    B, H, N = 2, 3, 700
    c = synth.make_qkv(B, H, N, d, dtype, 6100 + d)
    q, k, v, m = (dev(c[x]) for x in ("q", "k", "v", "m"))
    qb, kb, vb = (_as_bnhd(x) for x in (q, k, v))
    cuts = [0, 130, 131, 512, 700]
    st_a = st_b = None
    for a, b in zip(cuts[:-1], cuts[1:]):
        seg = lambda x: x[:, :, a:b]
        oa, st_a = cott.fwd_stateful(seg(q).contiguous(), seg(k).contiguous(), seg(v).contiguous(), m, float(N),
                                     state_in=st_a)
        ob, st_b = cott.fwd_stateful(seg(qb), seg(kb), seg(vb), m, float(N), state_in=st_b,
                                     out=torch.empty_like(oa))
        assert not seg(qb).is_contiguous()
        assert torch.equal(oa, ob) and torch.equal(st_a, st_b)
