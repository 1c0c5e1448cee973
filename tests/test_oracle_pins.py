"""Pins of the fp64 oracle against things other than itself: a hand-worked example, closed
forms, invariants, numpy GEMM/tril, brute-force Python loops and finite differences.
All CPU; the GPU library is not involved."""
import json
import math
import os

import numpy as np
import pytest

import oracle

HERE = os.path.dirname(os.path.abspath(__file__))


def rnd(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


@pytest.fixture(scope="module")
def hand():
    with open(os.path.join(HERE, "golden", "hand_example.json")) as f:
        g = json.load(f)
    t = lambda key: np.array(g[key], dtype=np.float64).reshape(1, 1, 4, 2)
    g["_t"] = {k: t(k) for k in ("Q", "K", "V", "dO")}
    return g


# ---------------------------------------------------------------- hand-worked example
def test_hand_example_forward(hand):
    Q, K, V = hand["_t"]["Q"], hand["_t"]["K"], hand["_t"]["V"]
    m, s = np.array(hand["m"]), np.array(hand["s"])
    np.testing.assert_allclose(oracle.fwd_quadratic(Q, K, V, m, s, True)[0, 0], hand["O_causal"], rtol=0, atol=1e-14)
    np.testing.assert_allclose(oracle.fwd_quadratic(Q, K, V, m, s, False)[0, 0], hand["O_bidirectional"], rtol=0, atol=1e-14)
    o_rec, st = oracle.fwd_recurrent(Q, K, V, m, s)
    np.testing.assert_allclose(o_rec[0, 0], hand["O_causal"], rtol=0, atol=1e-14)
    np.testing.assert_allclose(st[0, 0], hand["state_final"], rtol=0, atol=1e-14)
    o_bi, st_bi = oracle.fwd_bidir_assoc(Q, K, V, m, s)
    np.testing.assert_allclose(o_bi[0, 0], hand["O_bidirectional"], rtol=0, atol=1e-14)
    np.testing.assert_allclose(st_bi[0, 0], hand["state_final"], rtol=0, atol=1e-14)
    rows = oracle.fwd_rows(Q, K, V, m, [3, 0], s, True)
    np.testing.assert_allclose(rows[0, 0], [hand["O_causal"][3], hand["O_causal"][0]], rtol=0, atol=1e-14)


@pytest.mark.parametrize("bwd", [oracle.bwd_quadratic, oracle.bwd_recurrent])
def test_hand_example_backward(hand, bwd):
    Q, K, V, dO = (hand["_t"][k] for k in ("Q", "K", "V", "dO"))
    m, s = np.array(hand["m"]), np.array(hand["s"])
    dq, dk, dv, dm = bwd(Q, K, V, dO, m, s)
    np.testing.assert_allclose(dq[0, 0], hand["dQ_causal"], rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(dk[0, 0], hand["dK_causal"], rtol=1e-12, atol=1e-15)  # row 2: clamped branch
    np.testing.assert_allclose(dv[0, 0], hand["dV_causal"], rtol=1e-12, atol=1e-15)
    assert dm[0] == pytest.approx(hand["dm_causal"], rel=1e-12)
    assert dm[0] == pytest.approx(-1.26 * math.log(4.0), rel=1e-12)


def test_hand_example_variant(hand):
    Q, K, V, dO = (hand["_t"][k].copy() for k in ("Q", "K", "V", "dO"))
    K[0, 0, 2] = hand["variant_K_row2"]
    m, s = np.array(hand["m"]), np.array(hand["s"])
    o = oracle.fwd_quadratic(Q, K, V, m, s, True)
    np.testing.assert_allclose(o[0, 0, 2:], hand["variant_O_causal_rows_2_3"], rtol=0, atol=1e-14)
    dq, dk, dv, dm = oracle.bwd_quadratic(Q, K, V, dO, m, s)
    np.testing.assert_allclose(dk[0, 0, 2], hand["variant_dK_row2"], rtol=0, atol=1e-14)
    np.testing.assert_allclose(dv[0, 0, 2], hand["variant_dV_row2"], rtol=0, atol=1e-14)
    assert dm[0] == pytest.approx(hand["variant_dm"], rel=1e-11)


# ---------------------------------------------------------------- brute force in pure Python
def brute_force(q, k, v, m, s, causal):
    B, H, N, d = q.shape
    o = np.zeros_like(q)
    for b in range(B):
        for h in range(H):
            c = s[b] ** (-(1.0 / (1.0 + math.exp(-m[h]))))
            for t in range(N):
                nq = max(math.sqrt(sum(x * x for x in q[b, h, t])), 1e-12)
                for j in range(N):
                    if causal and j > t:
                        continue
                    nk = max(math.sqrt(sum(x * x for x in k[b, h, j])), 1e-12)
                    cos = sum(q[b, h, t, a] * k[b, h, j, a] for a in range(d)) / (nq * nk)
                    for e in range(d):
                        o[b, h, t, e] += cos * v[b, h, j, e] * c
    return o


@pytest.mark.parametrize("causal", [True, False])
def test_brute_force_tiny(causal):
    B, H, N, d = 2, 2, 7, 3
    q, k, v = rnd((B, H, N, d), 1), rnd((B, H, N, d), 2), rnd((B, H, N, d), 3)
    k[0, 1, 4] = 0.0
    m, s = rnd((H,), 4), np.array([7.0, 3.5])
    ref = brute_force(q, k, v, m, s, causal)
    np.testing.assert_allclose(oracle.fwd_quadratic(q, k, v, m, s, causal), ref, rtol=1e-12, atol=1e-13)


# ---------------------------------------------------------------- library-routine cross-check
def numpy_forward(q, k, v, m, s, causal):
    nq = np.maximum(np.linalg.norm(q, axis=-1, keepdims=True), 1e-12)
    nk = np.maximum(np.linalg.norm(k, axis=-1, keepdims=True), 1e-12)
    scores = (q / nq) @ np.swapaxes(k / nk, -1, -2)
    if causal:
        scores = np.tril(scores)
    c = s[:, None] ** (-(1.0 / (1.0 + np.exp(-m[None, :]))))
    return (scores @ v) * c[:, :, None, None]


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("shape", [(2, 3, 37, 8), (1, 2, 130, 32)])
def test_numpy_gemm_tril(causal, shape):
    B, H, N, d = shape
    q, k, v = rnd(shape, 11), rnd(shape, 12), rnd(shape, 13)
    q *= np.exp(rnd((B, H, N, 1), 14))
    m, s = rnd((H,), 15), np.linspace(N, N / 2, B)
    ref = numpy_forward(q, k, v, m, s, causal)
    np.testing.assert_allclose(oracle.fwd_quadratic(q, k, v, m, s, causal), ref, rtol=1e-11, atol=1e-12)


# ---------------------------------------------------------------- identities between the forms
def test_three_way_consistency():
    shape = (2, 3, 150, 16)
    B, H, N, d = shape
    q, k, v = rnd(shape, 21), rnd(shape, 22), rnd(shape, 23)
    m, s = rnd((H,), 24), np.array([150.0, 97.0])
    oq = oracle.fwd_quadratic(q, k, v, m, s, True)
    orr, st = oracle.fwd_recurrent(q, k, v, m, s)
    np.testing.assert_allclose(orr, oq, rtol=1e-11, atol=1e-12)
    ob = oracle.fwd_quadratic(q, k, v, m, s, False)
    oa, sa = oracle.fwd_bidir_assoc(q, k, v, m, s)
    np.testing.assert_allclose(oa, ob, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(st, sa, rtol=1e-12, atol=1e-13)          # final state = c K^^T V
    np.testing.assert_allclose(oq[:, :, -1], ob[:, :, -1], rtol=1e-11, atol=1e-12)  # last causal row sees all
    rows = [0, 1, 63, 64, 65, 149]
    np.testing.assert_allclose(oracle.fwd_rows(q, k, v, m, rows, s, True), oq[:, :, rows], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(oracle.fwd_rows(q, k, v, m, rows, s, False), ob[:, :, rows], rtol=1e-12, atol=1e-13)


def test_backward_forms_agree():
    shape = (2, 2, 40, 8)
    q, k, v, do = (rnd(shape, i) for i in (31, 32, 33, 34))
    m, s = rnd((2,), 35), np.array([40.0, 11.0])
    a = oracle.bwd_quadratic(q, k, v, do, m, s, True)
    b = oracle.bwd_recurrent(q, k, v, do, m, s)
    for x, y in zip(a, b):
        np.testing.assert_allclose(x, y, rtol=1e-10, atol=1e-12)


# ---------------------------------------------------------------- closed forms and invariants
def test_closed_form_constant_rows():
    B, H, N, d = 1, 2, 9, 4
    u, w = np.array([1.0, -2.0, 0.5, 3.0]), np.array([0.25, -1.0, 2.0, 0.0])
    q = np.broadcast_to(u * 3.0, (B, H, N, d)).copy()
    k = np.broadcast_to(u * 0.1, (B, H, N, d)).copy()
    v = np.broadcast_to(w, (B, H, N, d)).copy()
    m, s = np.array([0.3, -1.2]), np.array([float(N)])
    o = oracle.fwd_quadratic(q, k, v, m, s, True)
    ob = oracle.fwd_quadratic(q, k, v, m, s, False)
    for h in range(H):
        c = N ** (-(1 / (1 + math.exp(-m[h]))))
        for t in range(N):
            np.testing.assert_allclose(o[0, h, t], c * (t + 1) * w, rtol=1e-12, atol=1e-14)
            np.testing.assert_allclose(ob[0, h, t], c * N * w, rtol=1e-12, atol=1e-14)
    # m -> +inf with s = N: the bidirectional output is exactly w; s = 1: c = 1 for any m
    o_inf = oracle.fwd_quadratic(q, k, v, np.array([50.0, 60.0]), s, False)
    np.testing.assert_allclose(o_inf[0, 0, 0], w, rtol=1e-12, atol=1e-14)
    o_s1 = oracle.fwd_quadratic(q, k, v, m, np.array([1.0]), True)
    np.testing.assert_allclose(o_s1[0, 1, 4], 5 * w, rtol=1e-12, atol=1e-14)


def test_invariants():
    shape = (1, 2, 64, 8)
    q, k, v = rnd(shape, 41), rnd(shape, 42), rnd(shape, 43)
    m, s = np.array([0.5, -0.7]), np.array([64.0])
    o = oracle.fwd_quadratic(q, k, v, m, s, True)
    # scale invariance in Q and K rows (cosine similarity, Eq. 2)
    fq, fk = np.exp(rnd((1, 2, 64, 1), 44)), np.exp(rnd((1, 2, 64, 1), 45))
    np.testing.assert_allclose(oracle.fwd_quadratic(q * fq, k * fk, v, m, s, True), o, rtol=1e-11, atol=1e-12)
    # linearity in V
    np.testing.assert_allclose(oracle.fwd_quadratic(q, k, 2.5 * v, m, s, True), 2.5 * o, rtol=1e-12, atol=1e-13)
    # causality: future tokens do not change earlier outputs, bit for bit
    q2, k2, v2 = q.copy(), k.copy(), v.copy()
    q2[:, :, 40:] += 1.0; k2[:, :, 40:] *= -3.0; v2[:, :, 40:] = 7.0
    assert np.array_equal(oracle.fwd_quadratic(q2, k2, v2, m, s, True)[:, :, :40], o[:, :, :40])
    # bound: |o_t| <= c * sum_{j<=t} |v_j|_inf since every score lies in [-1,1]
    for h in range(2):
        c = 64.0 ** (-(1 / (1 + math.exp(-m[h]))))
        assert 1 / 64.0 <= c <= 1.0
        bound = c * np.cumsum(np.abs(v[0, h]).max(axis=-1))
        assert (np.abs(o[0, h]).max(axis=-1) <= bound + 1e-12).all()
    # recovered scores: with V = identity columns the output row is c * score row
    N, d = 8, 8
    qq, kk = rnd((1, 1, N, d), 46), rnd((1, 1, N, d), 47)
    sc = oracle.fwd_quadratic(qq, kk, np.eye(N).reshape(1, 1, N, N)[..., :d], np.array([0.0]), np.array([1.0]), False)
    assert (np.abs(sc) <= 1.0 + 1e-12).all()


def test_gradient_invariants():
    shape = (1, 2, 24, 8)
    q, k, v, do = (rnd(shape, i) for i in (51, 52, 53, 54))
    m, s = np.array([0.2, 1.1]), np.array([24.0])
    dq, dk, dv, dm = oracle.bwd_quadratic(q, k, v, do, m, s, True)
    # degree-0 homogeneity in each Q / K row: the gradient is orthogonal to the row
    assert np.abs((dq * q).sum(-1)).max() < 1e-12
    assert np.abs((dk * k).sum(-1)).max() < 1e-12
    # two routes to dm: <dO,O> = c <dV',V>  =>  dm_h = <dO,O>_h * (-ln s) sigma(1-sigma)
    o = oracle.fwd_quadratic(q, k, v, m, s, True)
    for h in range(2):
        sg = 1 / (1 + math.exp(-m[h]))
        assert dm[h] == pytest.approx((do[0, h] * o[0, h]).sum() * (-math.log(24.0)) * sg * (1 - sg), rel=1e-11)


def test_dm_sum_by_query_rows_equals_sum_by_value_rows():
    """The identity the causal tensor-core backward relies on for dm, written out with numpy:
    with dV'_j = sum_{i>=j} (q^_i.k^_j) dO_i and dQ^_i = sum_{j<=i} (dO_i.v_j) k^_j (both without
    the factor c), sum_j <dV'_j, v_j> = sum_i <q^_i, dQ^_i>, and dm_h of the oracle is that sum
    times dc/dm.  Bidirectional: the same with full sums."""
    N, d = 19, 6
    q, k, v, do = (rnd((N, d), i) for i in (61, 62, 63, 64))
    k[5] = 0.0                                   # a zero key row takes the clamped branch
    qh = q / np.maximum(np.linalg.norm(q, axis=-1, keepdims=True), 1e-12)
    kh = k / np.maximum(np.linalg.norm(k, axis=-1, keepdims=True), 1e-12)
    for causal in (True, False):
        mask = np.tril(np.ones((N, N))) if causal else np.ones((N, N))
        p = (qh @ kh.T) * mask                   # [i, j]
        dvp = p.T @ do                           # dV'
        dqh = ((do @ v.T) * mask) @ kh           # dQ^
        by_value_rows = (dvp * v).sum()
        by_query_rows = (qh * dqh).sum()
        assert by_query_rows == pytest.approx(by_value_rows, rel=1e-12)
        m, s = np.array([0.4]), np.array([float(N)])
        dm = oracle.bwd_quadratic(q[None, None], k[None, None], v[None, None], do[None, None], m, s, causal)[3]
        sg = 1 / (1 + math.exp(-m[0]))
        dcdm = -math.log(float(N)) * sg * (1 - sg) * float(N) ** (-sg)
        assert dm[0] == pytest.approx(by_query_rows * dcdm, rel=1e-10)


# ---------------------------------------------------------------- finite differences
@pytest.mark.parametrize("causal", [True, False])
def test_finite_differences(causal):
    shape = (2, 2, 6, 4)
    q, k, v, do = (rnd(shape, i) for i in (61, 62, 63, 64))
    m, s = np.array([0.4, -0.9]), np.array([6.0, 4.0])
    dq, dk, dv, dm = oracle.bwd_quadratic(q, k, v, do, m, s, causal)
    loss = lambda q_, k_, v_, m_: float((oracle.fwd_quadratic(q_, k_, v_, m_, s, causal) * do).sum())
    h = 1e-6
    rng = np.random.default_rng(65)
    for name, x, g in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        for _ in range(12):
            idx = tuple(rng.integers(0, n) for n in shape)
            xp, xm = x.copy(), x.copy()
            xp[idx] += h; xm[idx] -= h
            args_p = {"q": q, "k": k, "v": v}; args_p[name] = xp
            args_m = {"q": q, "k": k, "v": v}; args_m[name] = xm
            fd = (loss(args_p["q"], args_p["k"], args_p["v"], m) - loss(args_m["q"], args_m["k"], args_m["v"], m)) / (2 * h)
            assert g[idx] == pytest.approx(fd, rel=2e-6, abs=2e-8), (name, idx)
    for hh in range(2):
        mp, mm = m.copy(), m.copy()
        mp[hh] += h; mm[hh] -= h
        fd = (loss(q, k, v, mp) - loss(q, k, v, mm)) / (2 * h)
        assert dm[hh] == pytest.approx(fd, rel=2e-6, abs=2e-8)


def test_clamped_branch_gradient():
    """Gradient of the clamped formula on a zero K row: dk = dk^ / eps."""
    shape = (1, 1, 5, 3)
    q, k, v, do = (rnd(shape, i) for i in (71, 72, 73, 74))
    k[0, 0, 2] = 0.0
    m, s = np.array([0.0]), np.array([5.0])
    dq, dk, dv, dm = oracle.bwd_quadratic(q, k, v, do, m, s, True)
    # d k^_2 = sum_{t>=2} (dO_t . v'_2) q^_t   (printed dK formula, row 2)
    qh = q / np.linalg.norm(q, axis=-1, keepdims=True)
    c = 5.0 ** -0.5
    dkh2 = sum((do[0, 0, t] @ (c * v[0, 0, 2])) * qh[0, 0, t] for t in range(2, 5))
    np.testing.assert_allclose(dk[0, 0, 2], dkh2 / 1e-12, rtol=1e-10)
    assert np.array_equal(dv[0, 0, 2], np.zeros(3))  # zero key: its value gets no gradient


# ---------------------------------------------------------------- decode
def test_prefill_then_decode_equals_longer_forward():
    B, H, N, T, d = 2, 2, 20, 6, 4
    q, k, v = rnd((B, H, N + T, d), 81), rnd((B, H, N + T, d), 82), rnd((B, H, N + T, d), 83)
    m, s = np.array([0.5, -0.3]), np.array([30.0, 26.0])
    full = oracle.fwd_quadratic(q, k, v, m, s, True)
    _, st = oracle.fwd_recurrent(q[:, :, :N], k[:, :, :N], v[:, :, :N], m, s)
    st = np.ascontiguousarray(st)
    for t in range(N, N + T):
        o = oracle.decode_step(q[:, :, t], k[:, :, t], v[:, :, t], m, s, st)
        np.testing.assert_allclose(o, full[:, :, t], rtol=1e-11, atol=1e-12)
    _, st_full = oracle.fwd_recurrent(q, k, v, m, s)
    np.testing.assert_allclose(st, st_full, rtol=1e-12, atol=1e-13)


# ------------------------------------------------------------------ different key and value sizes
def _frac(x):
    from fractions import Fraction
    return np.array([[float(Fraction(e)) for e in row] for row in x])


@pytest.fixture(scope="module")
def hand_rect():
    with open(os.path.join(HERE, "golden", "hand_example_dk2_dv3.json")) as f:
        return json.load(f)


def test_hand_example_with_different_key_and_value_sizes(hand_rect):
    """d_key = 2, d_value = 3 (section 2.1 of the paper lets them differ): every tensor of the
    forward, the final state and all gradients against fractions worked out by hand."""
    g = hand_rect
    t4 = lambda x: np.array(x, dtype=np.float64)[None, None]
    q, k, v, d_o = t4(g["Q"]), t4(g["K"]), t4(g["V"]), t4(g["dO"])
    m, s = np.array(g["m"]), np.array(g["s"])
    tol = dict(rtol=0, atol=1e-14)
    np.testing.assert_allclose(oracle.fwd_quadratic(q, k, v, m, s, True)[0, 0], _frac(g["O_causal"]), **tol)
    np.testing.assert_allclose(oracle.fwd_quadratic(q, k, v, m, s, False)[0, 0], _frac(g["O_bidirectional"]), **tol)
    o, st = oracle.fwd_recurrent(q, k, v, m, s)
    assert st.shape == (1, 1, 2, 3)
    np.testing.assert_allclose(o[0, 0], _frac(g["O_causal"]), **tol)
    np.testing.assert_allclose(st[0, 0], _frac(g["state_final"]), **tol)
    o, st = oracle.fwd_bidir_assoc(q, k, v, m, s)
    np.testing.assert_allclose(o[0, 0], _frac(g["O_bidirectional"]), **tol)
    np.testing.assert_allclose(st[0, 0], _frac(g["state_final"]), **tol)
    np.testing.assert_allclose(oracle.fwd_rows(q, k, v, m, [1], s, True)[0, 0, 0], _frac(g["O_causal"])[1], **tol)
    from fractions import Fraction
    dm_ref = float(Fraction(g["dm_causal_over_ln4"])) * np.log(4.0)
    for bwd in (oracle.bwd_quadratic, oracle.bwd_recurrent):
        dq, dk, dv, dm = bwd(q, k, v, d_o, m, s)
        np.testing.assert_allclose(dq[0, 0], _frac(g["dQ_causal"]), **tol)
        np.testing.assert_allclose(dk[0, 0], _frac(g["dK_causal"]), **tol)
        np.testing.assert_allclose(dv[0, 0], _frac(g["dV_causal"]), **tol)
        np.testing.assert_allclose(dm[0], dm_ref, rtol=1e-13)
    # one decode step per token reproduces the rows and the state
    state = np.zeros((1, 1, 2, 3))
    for t in range(2):
        o_t = oracle.decode_step(q[:, :, t], k[:, :, t], v[:, :, t], m, s, state)
        np.testing.assert_allclose(o_t[0, 0], _frac(g["O_causal"])[t], **tol)
    np.testing.assert_allclose(state[0, 0], _frac(g["state_final"]), **tol)


@pytest.mark.parametrize("dk,dv", [(3, 7), (8, 5), (16, 4)])
@pytest.mark.parametrize("causal", [True, False])
def test_unequal_sizes_are_the_square_problem_with_zero_columns(dk, dv, causal):
    """Zero columns change no norm, no score and no product: the dk x dv problem embedded in a
    square one of size max(dk, dv) by zero-padding q, k (or v, dO) must give the same outputs
    and gradients, zeros in the padded columns -- which ties the rectangular code to the
    square case every other pin covers.  The padded dq, dk columns are exactly zero only for
    unclamped rows (all rows here)."""
    B, H, N, D = 2, 2, 19, max(dk, dv)
    q, k = rnd((B, H, N, dk), 71), rnd((B, H, N, dk), 72)
    v, d_o = rnd((B, H, N, dv), 73), rnd((B, H, N, dv), 74)
    m, s = rnd((H,), 75), np.array([7.0, 30.0])
    pad = lambda x: np.concatenate([x, np.zeros(x.shape[:-1] + (D - x.shape[-1],))], axis=-1)
    o = oracle.fwd_quadratic(q, k, v, m, s, causal)
    o_sq = oracle.fwd_quadratic(pad(q), pad(k), pad(v), m, s, causal)
    np.testing.assert_allclose(o_sq[..., :dv], o, rtol=1e-13, atol=1e-13)
    assert np.all(o_sq[..., dv:] == 0.0)
    got = oracle.bwd_quadratic(q, k, v, d_o, m, s, causal)
    ref = oracle.bwd_quadratic(pad(q), pad(k), pad(v), pad(d_o), m, s, causal)
    for g_, r_, w in zip(got[:3], ref[:3], (dk, dk, dv)):
        np.testing.assert_allclose(r_[..., :w], g_, rtol=1e-12, atol=1e-12)
        assert w == D or np.abs(r_[..., w:]).max() == 0.0
    np.testing.assert_allclose(got[3], ref[3], rtol=1e-12)
    if causal:
        o_r, st = oracle.fwd_recurrent(q, k, v, m, s)
        _, st_sq = oracle.fwd_recurrent(pad(q), pad(k), pad(v), m, s)
        np.testing.assert_allclose(o_r, o, rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(st_sq[:, :, :dk, :dv], st, rtol=1e-13, atol=1e-13)
        rec = oracle.bwd_recurrent(q, k, v, d_o, m, s)
        for a, b in zip(rec, got):
            np.testing.assert_allclose(a, b, rtol=1e-10, atol=1e-10)
    else:
        o_a, st = oracle.fwd_bidir_assoc(q, k, v, m, s)
        np.testing.assert_allclose(o_a, o, rtol=1e-12, atol=1e-12)
        assert st.shape == (B, H, dk, dv)


@pytest.mark.parametrize("causal", [True, False])
def test_unequal_sizes_numpy_and_finite_differences(causal):
    """dk = 5, dv = 3 against the masked-GEMM form in numpy, and the gradients against central
    differences of the forward definition."""
    B, H, N, dk, dv = 1, 2, 9, 5, 3
    q, k = rnd((B, H, N, dk), 81), rnd((B, H, N, dk), 82)
    v, d_o = rnd((B, H, N, dv), 83), rnd((B, H, N, dv), 84)
    m, s = rnd((H,), 85), np.array([11.0])
    np.testing.assert_allclose(oracle.fwd_quadratic(q, k, v, m, s, causal), numpy_forward(q, k, v, m, s, causal),
                               rtol=1e-12, atol=1e-12)
    dq, dk_, dv_, dm = oracle.bwd_quadratic(q, k, v, d_o, m, s, causal)
    loss = lambda q_, k_, v_, m_: float((oracle.fwd_quadratic(q_, k_, v_, m_, s, causal) * d_o).sum())
    eps = 1e-6
    r = np.random.default_rng(86)
    for name, x, g in (("q", q, dq), ("k", k, dk_), ("v", v, dv_)):
        for _ in range(6):
            idx = tuple(r.integers(0, n) for n in x.shape)
            xp, xm = x.copy(), x.copy()
            xp[idx] += eps; xm[idx] -= eps
            args_p = {"q": (xp, k, v), "k": (q, xp, v), "v": (q, k, xp)}[name]
            args_m = {"q": (xm, k, v), "k": (q, xm, v), "v": (q, k, xm)}[name]
            fd = (loss(*args_p, m) - loss(*args_m, m)) / (2 * eps)
            assert abs(fd - g[idx]) <= 1e-6 * max(1.0, abs(fd)), (name, idx, fd, g[idx])
    for h in range(H):
        mp, mm = m.copy(), m.copy()
        mp[h] += eps; mm[h] -= eps
        fd = (loss(q, k, v, mp) - loss(q, k, v, mm)) / (2 * eps)
        assert abs(fd - dm[h]) <= 1e-6 * max(1.0, abs(fd))


# ---------------------------------------------------------------- segments of a longer sequence
def _segment_case(seed, B=2, H=3, N=37, dk=6, dv=5):
    q, k = rnd((B, H, N, dk), seed), rnd((B, H, N, dk), seed + 1)
    v, do = rnd((B, H, N, dv), seed + 2), rnd((B, H, N, dv), seed + 3)
    m, s = rnd((H,), seed + 4), np.full((B,), float(N))
    return q, k, v, do, m, s


def test_segment_forward_composes_to_the_whole_sequence():
    """Eq. 8 started from a caller's state: with a zero state it is the recurrence from zero; cut
    anywhere, two segments give the outputs and the final state of the quadratic definition of the
    whole sequence (the scaling base belongs to the whole sequence)."""
    q, k, v, _, m, s = _segment_case(700)
    B, H, N, dk = q.shape
    dv = v.shape[-1]
    zero = np.zeros((B, H, dk, dv))
    o0, st0 = oracle.fwd_segment(q, k, v, m, zero, s)
    o_rec, st_rec = oracle.fwd_recurrent(q, k, v, m, s)
    assert np.array_equal(o0, o_rec) and np.array_equal(st0, st_rec)
    whole = oracle.fwd_quadratic(q, k, v, m, s, True)
    for cut in (1, 16, N - 1):
        o1, st1 = oracle.fwd_segment(q[:, :, :cut], k[:, :, :cut], v[:, :, :cut], m, zero, s)
        o2, st2 = oracle.fwd_segment(q[:, :, cut:], k[:, :, cut:], v[:, :, cut:], m, st1, s)
        np.testing.assert_allclose(np.concatenate([o1, o2], axis=2), whole, rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(st2, st_rec, rtol=1e-12, atol=1e-13)


def test_segment_backward_reduces_and_composes():
    """Backward of a segment.  (1) With a zero incoming state and no gradient into the outgoing one
    it is the quadratic definition's backward, and the gradient of the incoming state is
    sum_t q^_t dO_t^T (numpy).  (2) Chained over two segments -- the second one's d_state_in is the
    first one's d_state_out -- the gradients are those of the whole sequence, dm the sum."""
    q, k, v, do, m, s = _segment_case(710)
    B, H, N, dk = q.shape
    dv = v.shape[-1]
    zero = np.zeros((B, H, dk, dv))
    rq, rk, rv, rm = oracle.bwd_quadratic(q, k, v, do, m, s, True)
    dq, dk_, dv_, dst, dm = oracle.bwd_segment(q, k, v, do, m, zero, zero, s)
    for got, want in ((dq, rq), (dk_, rk), (dv_, rv), (dm, rm)):
        np.testing.assert_allclose(got, want, rtol=1e-11, atol=1e-12)
    qh = q / np.maximum(np.linalg.norm(q, axis=-1, keepdims=True), 1e-12)
    np.testing.assert_allclose(dst, np.einsum("bhta,bhte->bhae", qh, do), rtol=1e-12, atol=1e-13)
    for cut in (1, 20, N - 1):
        a, b = slice(0, cut), slice(cut, N)
        _, st1 = oracle.fwd_segment(q[:, :, a], k[:, :, a], v[:, :, a], m, zero, s)
        g2 = oracle.bwd_segment(q[:, :, b], k[:, :, b], v[:, :, b], do[:, :, b], m, st1, zero, s)
        g1 = oracle.bwd_segment(q[:, :, a], k[:, :, a], v[:, :, a], do[:, :, a], m, zero, g2[3], s)
        for i, want in enumerate((rq, rk, rv)):
            np.testing.assert_allclose(np.concatenate([g1[i], g2[i]], axis=2), want, rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(g1[4] + g2[4], rm, rtol=1e-11, atol=1e-12)


def test_segment_backward_finite_differences():
    """Central differences of L = <dO, O> + <d_state_out, state_out> through the segment forward
    (itself pinned above) in entries of state_in, q, k, v and in m."""
    q, k, v, do, m, s = _segment_case(720, B=1, H=2, N=9, dk=4, dv=3)
    B, H, N, dk = q.shape
    dv = v.shape[-1]
    st_in, d_st_out = rnd((B, H, dk, dv), 730), rnd((B, H, dk, dv), 731)
    s = np.array([64.0])

    def loss(q_, k_, v_, m_, st_):
        o, st = oracle.fwd_segment(q_, k_, v_, m_, st_, s)
        return float((do * o).sum() + (d_st_out * st).sum())

    dq, dk_, dv_, dst, dm = oracle.bwd_segment(q, k, v, do, m, st_in, d_st_out, s)
    eps = 1e-6
    rng = np.random.default_rng(740)
    for name, arr, grad in (("q", q, dq), ("k", k, dk_), ("v", v, dv_), ("state_in", st_in, dst)):
        for _ in range(6):
            idx = tuple(int(rng.integers(0, n)) for n in arr.shape)
            args = {"q": q, "k": k, "v": v, "state_in": st_in}
            hi, lo = arr.copy(), arr.copy()
            hi[idx] += eps; lo[idx] -= eps
            up = dict(args); up[name] = hi
            dn = dict(args); dn[name] = lo
            fd = (loss(up["q"], up["k"], up["v"], m, up["state_in"]) - loss(dn["q"], dn["k"], dn["v"], m, dn["state_in"])) / (2 * eps)
            assert grad[idx] == pytest.approx(fd, rel=1e-6, abs=1e-8), (name, idx)
    for h in range(H):
        mh, ml = m.copy(), m.copy()
        mh[h] += eps; ml[h] -= eps
        fd = (loss(q, k, v, mh, st_in) - loss(q, k, v, ml, st_in)) / (2 * eps)
        assert dm[h] == pytest.approx(fd, rel=1e-6, abs=1e-8)
