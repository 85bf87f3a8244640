"""Pins for the float64 oracle: closed forms, brute force, finite differences and the
paper's printed facts.  None of these re-use the oracle's own formulae, so a dropped
term, a wrong sign or index, or a transposed operand in oracle/ fails at least one."""
import math
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rnd(shape, seed, std=1.0):
    return std * np.random.default_rng(seed).standard_normal(shape)


def scalar_sigmoid(x):
    """Textbook definition with math.exp, independent of oracle.sigmoid."""
    if x >= 0:
        return 1.0 / (1.0 + math.exp(-x))
    e = math.exp(x)
    return e / (1.0 + e)


def brute_forward(q, k, v, scale, bias, causal, slopes):
    """Pure-Python loops over every (b, h, i, j, d): the definition, element by element."""
    B, H, N, D = q.shape
    o = np.zeros((B, H, N, D))
    for b in range(B):
        for h in range(H):
            m = 0.0 if slopes is None else float(slopes[h])
            for i in range(N):
                for j in range(N):
                    if causal and j > i:
                        continue
                    s = 0.0
                    for d in range(D):
                        s += q[b, h, i, d] * k[b, h, j, d]
                    x = scale * s + bias - m * abs(i - j)
                    p = scalar_sigmoid(x)
                    for d in range(D):
                        o[b, h, i, d] += p * v[b, h, j, d]
    return o


# ----------------------------------------------------------------------------- sigmoid


def test_sigmoid_identities():
    x = np.linspace(-40, 40, 2001)
    s = oracle.sigmoid(x)
    assert np.all(np.isfinite(s))
    np.testing.assert_allclose(s + oracle.sigmoid(-x), 1.0, rtol=0, atol=2.3e-16)  # 1 ulp
    assert oracle.sigmoid(np.array([0.0]))[0] == 0.5
    assert np.all(np.diff(s) >= 0)
    # Section 4: sigmoid(x) = 0.5 * (1 + tanh(0.5 x))
    np.testing.assert_allclose(s, 0.5 * (1.0 + np.tanh(0.5 * x)), rtol=0, atol=2.3e-16)
    ref = np.array([scalar_sigmoid(t) for t in x])
    np.testing.assert_allclose(s, ref, rtol=1e-15, atol=0)


def test_sigmoid_extremes():
    s = oracle.sigmoid(np.array([-1e4, -745.0, 745.0, 1e4]))
    assert s[0] == 0.0 and s[-1] == 1.0
    assert np.all(np.isfinite(s))


def test_sigmoid_derivative_is_p_times_one_minus_p():
    # Appendix E: d p / d z = p (1 - p)
    z = np.linspace(-6, 6, 25)
    h = 1e-6
    fd = (oracle.sigmoid(z + h) - oracle.sigmoid(z - h)) / (2 * h)
    p = oracle.sigmoid(z)
    np.testing.assert_allclose(fd, p * (1 - p), rtol=1e-7, atol=1e-10)  # fd truncation + rounding at h = 1e-6


# ------------------------------------------------------------------------------ masks


def test_causal_mask_matches_printed_n3_example():
    golden = np.loadtxt(os.path.join(GOLDEN, "causal_mask_n3.txt"))
    np.testing.assert_array_equal(oracle.causal_mask(3), golden)
    np.testing.assert_array_equal(oracle.causal_mask(3, 1, 3), golden[1:3])


def test_position_bias_is_minus_slope_times_distance():
    pb = oracle.position_bias(5, 0.25)
    for i in range(5):
        for j in range(5):
            assert pb[i, j] == -0.25 * abs(i - j)
    np.testing.assert_array_equal(oracle.position_bias(5, 0.25, 2, 4), pb[2:4])


# ---------------------------------------------------------------------------- forward


@pytest.mark.parametrize("causal", [False, True])
def test_forward_q_zero_closed_form(causal):
    B, H, N, D = 2, 3, 17, 8
    k, v = rnd((B, H, N, D), 1), rnd((B, H, N, D), 2)
    q = np.zeros((B, H, N, D))
    b = -math.log(N)
    o = oracle.sigattn_fwd(q, k, v, 1 / math.sqrt(D), b, causal)
    sb = scalar_sigmoid(b)
    if causal:
        expect = sb * np.cumsum(v, axis=2)
    else:
        expect = np.broadcast_to(sb * v.sum(axis=2, keepdims=True), v.shape)
    np.testing.assert_allclose(o, expect, rtol=1e-13, atol=1e-14)


@pytest.mark.parametrize("causal", [False, True])
def test_forward_bias_limits(causal):
    B, H, N, D = 1, 2, 9, 4
    q, k, v = rnd((B, H, N, D), 3), rnd((B, H, N, D), 4), rnd((B, H, N, D), 5)
    o_lo = oracle.sigattn_fwd(q, k, v, 0.5, -1e4, causal)
    assert np.all(o_lo == 0.0)
    o_hi = oracle.sigattn_fwd(q, k, v, 0.5, 1e4, causal)
    expect = np.cumsum(v, axis=2) if causal else np.broadcast_to(v.sum(axis=2, keepdims=True), v.shape)
    np.testing.assert_allclose(o_hi, expect, rtol=1e-14, atol=1e-14)


def test_forward_single_token():
    D = 6
    q, k, v = rnd((1, 1, 1, D), 6), rnd((1, 1, 1, D), 7), rnd((1, 1, 1, D), 8)
    scale, b = 0.37, -0.8
    for causal in (False, True):
        o = oracle.sigattn_fwd(q, k, v, scale, b, causal, alibi_slopes=[0.5])
        p = scalar_sigmoid(scale * float(q[0, 0, 0] @ k[0, 0, 0]) + b)
        np.testing.assert_allclose(o[0, 0, 0], p * v[0, 0, 0], rtol=1e-15)


def test_forward_complement_identity():
    # sigmoid(x) + sigmoid(-x) = 1  =>  O(Q, b) + O(-Q, -b) = column sum of V
    B, H, N, D = 2, 2, 11, 5
    q, k, v = rnd((B, H, N, D), 9), rnd((B, H, N, D), 10), rnd((B, H, N, D), 11)
    o1 = oracle.sigattn_fwd(q, k, v, 0.4, -1.3)
    o2 = oracle.sigattn_fwd(-q, k, v, 0.4, 1.3)
    np.testing.assert_allclose(o1 + o2, np.broadcast_to(v.sum(2, keepdims=True), v.shape), rtol=1e-13, atol=1e-13)


def test_forward_matches_sequence_form_and_direct_formula():
    # Eq. 4: at b = -log n the weights are exp(s) / (exp(s) + n)
    B, H, N, D = 1, 2, 13, 8
    q, k, v = rnd((B, H, N, D), 12), rnd((B, H, N, D), 13), rnd((B, H, N, D), 14)
    scale = 1 / math.sqrt(D)
    o = oracle.sigattn_fwd(q, k, v, scale, -math.log(N))
    np.testing.assert_allclose(o, oracle.sigattn_fwd_sequence_form(q, k, v, scale, N), rtol=1e-13, atol=1e-15)
    # the same second form retyped here with einsum, so the pin does not lean on oracle/
    e = np.exp(scale * np.einsum("bhid,bhjd->bhij", q, k))
    np.testing.assert_allclose(o, np.einsum("bhij,bhjd->bhid", e / (e + N), v), rtol=1e-13, atol=1e-15)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("with_slopes", [False, True])
def test_forward_brute_force(causal, with_slopes):
    B, H, N, D = 2, 2, 7, 3
    q, k, v = rnd((B, H, N, D), 15), rnd((B, H, N, D), 16), rnd((B, H, N, D), 17)
    slopes = np.array([0.5, 0.0625]) if with_slopes else None
    scale, b = 0.61, -1.1
    o = oracle.sigattn_fwd(q, k, v, scale, b, causal, slopes)
    np.testing.assert_allclose(o, brute_forward(q, k, v, scale, b, causal, slopes), rtol=1e-13, atol=1e-14)


def test_forward_causal_first_and_last_rows():
    B, H, N, D = 1, 1, 10, 4
    q, k, v = rnd((B, H, N, D), 18), rnd((B, H, N, D), 19), rnd((B, H, N, D), 20)
    scale, b = 0.5, -0.3
    oc = oracle.sigattn_fwd(q, k, v, scale, b, True)
    of = oracle.sigattn_fwd(q, k, v, scale, b, False)
    p00 = scalar_sigmoid(scale * float(q[0, 0, 0] @ k[0, 0, 0]) + b)
    np.testing.assert_allclose(oc[0, 0, 0], p00 * v[0, 0, 0], rtol=1e-14)
    np.testing.assert_allclose(oc[0, 0, -1], of[0, 0, -1], rtol=1e-14)
    assert not np.allclose(oc[0, 0, 3], of[0, 0, 3])


def test_forward_huge_slope_keeps_only_the_diagonal():
    B, H, N, D = 1, 2, 6, 4
    q, k, v = rnd((B, H, N, D), 21), rnd((B, H, N, D), 22), rnd((B, H, N, D), 23)
    scale, b = 0.5, 0.2
    o = oracle.sigattn_fwd(q, k, v, scale, b, True, alibi_slopes=[1e4, 1e4])
    for h in range(H):
        for i in range(N):
            p = scalar_sigmoid(scale * float(q[0, h, i] @ k[0, h, i]) + b)
            np.testing.assert_allclose(o[0, h, i], p * v[0, h, i], rtol=1e-13)


def test_forward_structure_properties():
    B, H, N, D = 2, 3, 9, 4
    q, k, v = rnd((B, H, N, D), 24), rnd((B, H, N, D), 25), rnd((B, H, N, D), 26)
    scale, b = 0.45, -1.0
    o = oracle.sigattn_fwd(q, k, v, scale, b)
    # zero slopes == no slopes
    np.testing.assert_array_equal(o, oracle.sigattn_fwd(q, k, v, scale, b, alibi_slopes=np.zeros(H)))
    # joint permutation of keys and values leaves O unchanged; permuting queries permutes O
    perm = np.random.default_rng(0).permutation(N)
    np.testing.assert_allclose(o, oracle.sigattn_fwd(q, k[:, :, perm], v[:, :, perm], scale, b), rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(o[:, :, perm], oracle.sigattn_fwd(q[:, :, perm], k, v, scale, b), rtol=1e-13, atol=1e-14)
    # linear in V
    v2 = rnd((B, H, N, D), 27)
    np.testing.assert_allclose(
        oracle.sigattn_fwd(q, k, 2 * v - 3 * v2, scale, b),
        2 * o - 3 * oracle.sigattn_fwd(q, k, v2, scale, b), rtol=1e-12, atol=1e-13)
    # heads and batches are independent; each head uses its own slope
    slopes = np.array([0.5, 0.25, 0.125])
    os_ = oracle.sigattn_fwd(q, k, v, scale, b, True, slopes)
    for bb in range(B):
        for h in range(H):
            one = oracle.sigattn_fwd(q[bb:bb + 1, h:h + 1], k[bb:bb + 1, h:h + 1], v[bb:bb + 1, h:h + 1],
                                     scale, b, True, slopes[h:h + 1])
            np.testing.assert_array_equal(os_[bb, h], one[0, 0])
    # row slabs give the same result as all rows at once
    np.testing.assert_allclose(os_, oracle.sigattn_fwd(q, k, v, scale, b, True, slopes, row_block=4), rtol=1e-14, atol=1e-15)


# --------------------------------------------------------------------------- backward


def loss(q, k, v, d_o, scale, b, causal, slopes):
    return float(np.sum(oracle.sigattn_fwd(q, k, v, scale, b, causal, slopes) * d_o))


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("with_slopes", [False, True])
def test_backward_finite_differences(causal, with_slopes):
    """Central differences of L = sum(O * dO).  This is what settles the 1/sqrt(d)
    factor in dQ, dK against the sqrt(d) printed in Appendix F.1."""
    B, H, N, D = 1, 2, 6, 4
    q, k, v, d_o = (rnd((B, H, N, D), s) for s in (30, 31, 32, 33))
    slopes = np.array([0.5, 0.125]) if with_slopes else None
    scale, b = 1 / math.sqrt(D), -math.log(N)
    dq, dk, dv = oracle.sigattn_bwd(q, k, v, d_o, scale, b, causal, slopes)
    h = 1e-6
    for name, x, g in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        fd = np.zeros_like(x)
        it = np.nditer(x, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            old = x[idx]
            x[idx] = old + h
            lp = loss(q, k, v, d_o, scale, b, causal, slopes)
            x[idx] = old - h
            lm = loss(q, k, v, d_o, scale, b, causal, slopes)
            x[idx] = old
            fd[idx] = (lp - lm) / (2 * h)
        err = np.linalg.norm(fd - g) / np.linalg.norm(fd)
        assert err < 1e-7, (name, err)
        if name in ("q", "k"):
            # the printed sqrt(d) factor would be off by exactly d
            assert np.linalg.norm(fd - D * g) / np.linalg.norm(fd) > 1.0


def test_backward_single_token_closed_form():
    D = 5
    q, k, v, d_o = (rnd((1, 1, 1, D), s) for s in (40, 41, 42, 43))
    scale, b = 0.3, -0.4
    dq, dk, dv = oracle.sigattn_bwd(q, k, v, d_o, scale, b, True)
    p = scalar_sigmoid(scale * float(q[0, 0, 0] @ k[0, 0, 0]) + b)
    ds = float(d_o[0, 0, 0] @ v[0, 0, 0]) * p * (1 - p)
    np.testing.assert_allclose(dv[0, 0, 0], p * d_o[0, 0, 0], rtol=1e-14)
    np.testing.assert_allclose(dq[0, 0, 0], scale * ds * k[0, 0, 0], rtol=1e-14)
    np.testing.assert_allclose(dk[0, 0, 0], scale * ds * q[0, 0, 0], rtol=1e-14)


@pytest.mark.parametrize("causal", [False, True])
def test_backward_brute_force_loops(causal):
    B, H, N, D = 1, 2, 5, 3
    q, k, v, d_o = (rnd((B, H, N, D), s) for s in (50, 51, 52, 53))
    slopes = np.array([0.25, 0.5])
    scale, b = 0.7, -0.9
    dq, dk, dv = oracle.sigattn_bwd(q, k, v, d_o, scale, b, causal, slopes)
    rq, rk, rv = np.zeros_like(q), np.zeros_like(q), np.zeros_like(q)
    for h in range(H):
        for i in range(N):
            for j in range(N):
                if causal and j > i:
                    continue
                x = scale * float(q[0, h, i] @ k[0, h, j]) + b - slopes[h] * abs(i - j)
                p = scalar_sigmoid(x)
                dp = float(d_o[0, h, i] @ v[0, h, j])
                ds = p * (1 - p) * dp
                rv[0, h, j] += p * d_o[0, h, i]
                rq[0, h, i] += scale * ds * k[0, h, j]
                rk[0, h, j] += scale * ds * q[0, h, i]
    np.testing.assert_allclose(dq, rq, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(dk, rk, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(dv, rv, rtol=1e-13, atol=1e-15)


def test_backward_structure_properties():
    B, H, N, D = 2, 2, 8, 4
    q, k, v, d_o = (rnd((B, H, N, D), s) for s in (60, 61, 62, 63))
    scale, b = 0.5, -1.2
    # Q = 0 => dK = 0 ; dV linear in dO ; row slabs agree
    _, dk0, _ = oracle.sigattn_bwd(np.zeros_like(q), k, v, d_o, scale, b, True)
    assert np.all(dk0 == 0.0)
    g1 = oracle.sigattn_bwd(q, k, v, d_o, scale, b, True)
    g2 = oracle.sigattn_bwd(q, k, v, 3.0 * d_o, scale, b, True)
    for a, c in zip(g1, g2):
        np.testing.assert_allclose(3.0 * a, c, rtol=1e-13, atol=1e-15)
    g3 = oracle.sigattn_bwd(q, k, v, d_o, scale, b, True, row_block=3)
    for a, c in zip(g1, g3):
        np.testing.assert_allclose(a, c, rtol=1e-13, atol=1e-15)
    # causal: the last key receives gradient only from the last query
    dq, dk, dv = g1
    p = scalar_sigmoid(scale * float(q[0, 0, -1] @ k[0, 0, -1]) + b)
    np.testing.assert_allclose(dv[0, 0, -1], p * d_o[0, 0, -1], rtol=1e-13)


# ------------------------------------------------------- bias per (batch, head) and its gradient


def test_bias_per_batch_and_head_equals_separate_scalar_calls():
    """A [B, H] bias must act as if every (batch, head) were computed alone with its own
    scalar bias; a [B] vector is one bias per sequence (b = -log n of each sample)."""
    B, H, N, D = 3, 2, 5, 4
    q, k, v, d_o = (rnd((B, H, N, D), s) for s in (60, 61, 62, 63))
    bias = rnd((B, H), 64)
    slopes = np.array([0.5, 0.25])
    o = oracle.sigattn_fwd(q, k, v, 0.4, bias, True, slopes)
    grads = oracle.sigattn_bwd(q, k, v, d_o, 0.4, bias, True, slopes)
    for b in range(B):
        for h in range(H):
            sel = (slice(b, b + 1), slice(h, h + 1))
            np.testing.assert_array_equal(
                o[sel], oracle.sigattn_fwd(q[sel], k[sel], v[sel], 0.4, float(bias[b, h]), True, slopes[h:h + 1]))
            one = oracle.sigattn_bwd(q[sel], k[sel], v[sel], d_o[sel], 0.4, float(bias[b, h]), True, slopes[h:h + 1])
            for g, r in zip(grads, one):
                np.testing.assert_array_equal(g[sel], r)
    per_sample = -np.log(np.array([3.0, 4.0, 5.0]))
    np.testing.assert_array_equal(oracle.sigattn_fwd(q, k, v, 0.4, per_sample, False),
                                  oracle.sigattn_fwd(q, k, v, 0.4, np.repeat(per_sample[:, None], H, axis=1), False))
    o_brute = np.concatenate([brute_forward(q[b:b + 1], k[b:b + 1], v[b:b + 1], 0.4, float(per_sample[b]), False, None)
                              for b in range(B)])
    np.testing.assert_allclose(oracle.sigattn_fwd(q, k, v, 0.4, per_sample, False), o_brute, rtol=1e-13, atol=1e-15)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("with_slopes", [False, True])
def test_bias_gradient_finite_differences(causal, with_slopes):
    """Central differences of L = sum(O * dO) with respect to each entry of a [B, H] bias."""
    B, H, N, D = 2, 2, 6, 4
    q, k, v, d_o = (rnd((B, H, N, D), s) for s in (70, 71, 72, 73))
    slopes = np.array([0.5, 0.125]) if with_slopes else None
    bias = -math.log(N) + 0.3 * rnd((B, H), 74)
    scale = 1 / math.sqrt(D)
    db = oracle.sigattn_bwd_dbias(q, k, v, d_o, scale, bias, causal, slopes)
    assert db.shape == (B, H)
    h = 1e-6
    fd = np.zeros_like(bias)
    for idx in np.ndindex(*bias.shape):
        bp, bm = bias.copy(), bias.copy()
        bp[idx] += h
        bm[idx] -= h
        fd[idx] = (loss(q, k, v, d_o, scale, bp, causal, slopes) - loss(q, k, v, d_o, scale, bm, causal, slopes)) / (2 * h)
    assert np.linalg.norm(fd - db) / np.linalg.norm(fd) < 1e-7
    # a scalar bias shared by everything gets the sum of the entries
    shared = -math.log(N)
    total = float(oracle.sigattn_bwd_dbias(q, k, v, d_o, scale, shared, causal, slopes).sum())
    fd_shared = (loss(q, k, v, d_o, scale, shared + h, causal, slopes) - loss(q, k, v, d_o, scale, shared - h, causal, slopes)) / (2 * h)
    assert abs(total - fd_shared) < 1e-7 * max(1.0, abs(fd_shared))


def test_bias_gradient_single_token_closed_form_and_brute_force():
    D = 5
    q, k, v, d_o = (rnd((1, 1, 1, D), s) for s in (80, 81, 82, 83))
    scale, b = 0.3, -0.4
    p = scalar_sigmoid(scale * float(q[0, 0, 0] @ k[0, 0, 0]) + b)
    expect = float(d_o[0, 0, 0] @ v[0, 0, 0]) * p * (1 - p)
    np.testing.assert_allclose(oracle.sigattn_bwd_dbias(q, k, v, d_o, scale, b, True), [[expect]], rtol=1e-14)
    # brute force over every (i, j) of a small causal problem with slopes
    B, H, N, D = 1, 2, 5, 3
    q, k, v, d_o = (rnd((B, H, N, D), s) for s in (84, 85, 86, 87))
    slopes = np.array([0.25, 0.5])
    bias = np.array([[-0.9, 0.2]])
    ref = np.zeros((B, H))
    for h in range(H):
        for i in range(N):
            for j in range(i + 1):
                x = 0.7 * float(q[0, h, i] @ k[0, h, j]) + bias[0, h] - slopes[h] * (i - j)
                pp = scalar_sigmoid(x)
                ref[0, h] += pp * (1 - pp) * float(d_o[0, h, i] @ v[0, h, j])
    np.testing.assert_allclose(oracle.sigattn_bwd_dbias(q, k, v, d_o, 0.7, bias, True, slopes), ref, rtol=1e-13)


# ------------------------------------------------------------- fewer key/value heads than query heads


@pytest.mark.parametrize("h_kv", [1, 2])
def test_grouped_kv_heads_forward_and_backward(h_kv):
    """k, v with H_kv heads: the forward must equal the element-by-element definition on
    keys/values repeated per query head, the gradients must match central differences of
    L = sum(O * dO) taken on the SHARED k, v (so sums over the group are checked too)."""
    B, H, N, D = 1, 4, 5, 3
    G = H // h_kv
    q, d_o = rnd((B, H, N, D), 90), rnd((B, H, N, D), 91)
    k, v = rnd((B, h_kv, N, D), 92), rnd((B, h_kv, N, D), 93)
    slopes = np.array([0.5, 0.25, 0.125, 0.0625])
    scale, b = 0.6, -1.1
    o = oracle.sigattn_fwd(q, k, v, scale, b, True, slopes)
    np.testing.assert_allclose(o, brute_forward(q, np.repeat(k, G, axis=1), np.repeat(v, G, axis=1), scale, b, True, slopes),
                               rtol=1e-13, atol=1e-15)
    dq, dk, dv = oracle.sigattn_bwd(q, k, v, d_o, scale, b, True, slopes)
    assert dk.shape == k.shape and dv.shape == v.shape
    h = 1e-6
    for name, x, g in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        fd = np.zeros_like(x)
        for idx in np.ndindex(*x.shape):
            old = x[idx]
            x[idx] = old + h
            lp = loss(q, k, v, d_o, scale, b, True, slopes)
            x[idx] = old - h
            lm = loss(q, k, v, d_o, scale, b, True, slopes)
            x[idx] = old
            fd[idx] = (lp - lm) / (2 * h)
        assert np.linalg.norm(fd - g) / np.linalg.norm(fd) < 1e-7, name
    with pytest.raises(ValueError):
        oracle.sigattn_fwd(q, rnd((B, 3, N, D), 94), rnd((B, 3, N, D), 95), scale, b)


def test_temperature_gradient_is_a_reduction_of_q_and_dq():
    """sigma(e^t [Q K^T / sqrt(d)] + b) V (Appendix G.2.2): with scale' = scale e^t passed as
    the scale, dL/dt = sum_i <Q_i, dQ_i>, because dQ_i = scale' sum_j dS_ij K_j."""
    B, H, N, D = 1, 2, 6, 4
    q, k, v, d_o = (rnd((B, H, N, D), s) for s in (100, 101, 102, 103))
    scale, b, t = 0.5, -1.3, 0.4
    dq, _, _ = oracle.sigattn_bwd(q, k, v, d_o, scale * math.exp(t), b, True)
    h = 1e-6
    fd = (loss(q, k, v, d_o, scale * math.exp(t + h), b, True, None) - loss(q, k, v, d_o, scale * math.exp(t - h), b, True, None)) / (2 * h)
    assert abs(float(np.sum(q * dq)) - fd) < 1e-7 * max(1.0, abs(fd))


@pytest.mark.parametrize("causal,with_slopes", [(False, False), (True, False), (True, True)])
def test_temperature_gradient_finite_differences_and_closed_forms(causal, with_slopes):
    """oracle.sigattn_bwd_dtemp, written from the logits, against (a) central differences in t of
    L(scale * e^t), one head at a time so that every [b, h] entry is pinned on its own, (b) the
    reduction sum_i <Q_i, dQ_i> of the independently pinned dQ, (c) the N = 1 closed form."""
    B, H, N, D = 2, 3, 6, 4
    q, k, v, d_o = (rnd((B, H, N, D), s) for s in (110, 111, 112, 113))
    slopes = np.array([0.5, 0.25, 0.125]) if with_slopes else None
    bias = rnd((B, H), 114)
    scale, t, hstep = 0.5, 0.3, 1e-6
    s_t = scale * math.exp(t)
    dt = oracle.sigattn_bwd_dtemp(q, k, v, d_o, s_t, bias, causal, slopes)
    assert dt.shape == (B, H)
    for b in range(B):
        for h in range(H):
            sel = (slice(b, b + 1), slice(h, h + 1))
            sl = None if slopes is None else slopes[h:h + 1]

            def L(tt):
                o = oracle.sigattn_fwd(q[sel], k[sel], v[sel], scale * math.exp(tt), bias[b, h], causal, sl)
                return float(np.sum(o * d_o[sel]))
            fd = (L(t + hstep) - L(t - hstep)) / (2 * hstep)
            assert abs(dt[b, h] - fd) < 1e-7 * max(1.0, abs(fd)), (b, h)
    dq, _, _ = oracle.sigattn_bwd(q, k, v, d_o, s_t, bias, causal, slopes)
    np.testing.assert_allclose(dt, np.sum(q * dq, axis=(2, 3)), rtol=1e-11, atol=1e-14)
    # N = 1: x = s_t q.k + b, dL/dt = P (1 - P) (dO.v) s_t q.k
    q1, k1, v1, g1 = (rnd((1, 1, 1, D), s) for s in (115, 116, 117, 118))
    x = s_t * float(q1[0, 0, 0] @ k1[0, 0, 0]) - 0.7
    pw = scalar_sigmoid(x)
    want = pw * (1 - pw) * float(g1[0, 0, 0] @ v1[0, 0, 0]) * s_t * float(q1[0, 0, 0] @ k1[0, 0, 0])
    got = oracle.sigattn_bwd_dtemp(q1, k1, v1, g1, s_t, -0.7, causal)
    assert abs(got[0, 0] - want) < 1e-14 * max(1.0, abs(want))


# ------------------------------------------------------------------ N_q queries against N_k keys


def test_queries_at_the_end_of_a_longer_key_sequence():
    """Decoding with a cache: the last N_q rows of square causal attention over N_k
    positions must equal rectangular attention of those N_q queries against all N_k keys,
    forward and backward (dK, dV of the rectangular call see only those queries)."""
    B, H, NK, NQ, D = 1, 2, 7, 3, 4
    q_full, k, v, do_full = (rnd((B, H, NK, D), s) for s in (110, 111, 112, 113))
    slopes = np.array([0.5, 0.125])
    scale, b = 0.5, -0.7
    q, d_o = q_full[:, :, NK - NQ:], do_full[:, :, NK - NQ:]
    o_sq = oracle.sigattn_fwd(q_full, k, v, scale, b, True, slopes)
    o = oracle.sigattn_fwd(q, k, v, scale, b, True, slopes)
    assert o.shape == (B, H, NQ, D)
    np.testing.assert_allclose(o, o_sq[:, :, NK - NQ:], rtol=1e-14, atol=1e-16)
    do_masked = np.zeros_like(do_full)
    do_masked[:, :, NK - NQ:] = d_o
    dq_sq, dk_sq, dv_sq = oracle.sigattn_bwd(q_full, k, v, do_masked, scale, b, True, slopes)
    dq, dk, dv = oracle.sigattn_bwd(q, k, v, d_o, scale, b, True, slopes)
    np.testing.assert_allclose(dq, dq_sq[:, :, NK - NQ:], rtol=1e-13, atol=1e-16)
    np.testing.assert_allclose(dk, dk_sq, rtol=1e-13, atol=1e-16)
    np.testing.assert_allclose(dv, dv_sq, rtol=1e-13, atol=1e-16)
    # one query against the whole cache, element by element
    o1 = oracle.sigattn_fwd(q[:, :, -1:], k, v, scale, b, True, slopes)
    for h in range(H):
        ref = np.zeros(D)
        for j in range(NK):
            x = scale * float(q[0, h, -1] @ k[0, h, j]) + b - slopes[h] * (NK - 1 - j)
            ref += scalar_sigmoid(x) * v[0, h, j]
        np.testing.assert_allclose(o1[0, h, 0], ref, rtol=1e-13)


def test_cross_attention_without_mask_brute_force():
    B, H, NQ, NK, D = 1, 1, 5, 3, 2
    q, d_o = rnd((B, H, NQ, D), 120), rnd((B, H, NQ, D), 121)
    k, v = rnd((B, H, NK, D), 122), rnd((B, H, NK, D), 123)
    scale, b = 0.8, -0.2
    o = oracle.sigattn_fwd(q, k, v, scale, b, False)
    ref = np.zeros_like(o)
    for i in range(NQ):
        for j in range(NK):
            ref[0, 0, i] += scalar_sigmoid(scale * float(q[0, 0, i] @ k[0, 0, j]) + b) * v[0, 0, j]
    np.testing.assert_allclose(o, ref, rtol=1e-13)
    dq, dk, dv = oracle.sigattn_bwd(q, k, v, d_o, scale, b, False)
    h = 1e-6
    for name, x, g in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        fd = np.zeros_like(x)
        for idx in np.ndindex(*x.shape):
            old = x[idx]
            x[idx] = old + h
            lp = loss(q, k, v, d_o, scale, b, False, None)
            x[idx] = old - h
            lm = loss(q, k, v, d_o, scale, b, False, None)
            x[idx] = old
            fd[idx] = (lp - lm) / (2 * h)
        assert np.linalg.norm(fd - g) / np.linalg.norm(fd) < 1e-7, name


# ------------------------------------------------------------------------- key/value shards


@pytest.mark.parametrize("causal", [False, True])
def test_key_value_shards_sum_to_the_whole(causal):
    """O and dQ are plain sums over contiguous key/value shards, dK and dV of a shard need
    only that shard; each shard call places the queries relative to its own first key.  One
    shard (entirely after some queries) is also checked element by element."""
    B, H, N, D = 1, 2, 9, 3
    q, k, v, d_o = (rnd((B, H, N, D), s) for s in (130, 131, 132, 133))
    slopes = np.array([0.5, 0.125])
    scale, b = 0.6, -0.8
    o = oracle.sigattn_fwd(q, k, v, scale, b, causal, slopes)
    dq, dk, dv = oracle.sigattn_bwd(q, k, v, d_o, scale, b, causal, slopes)
    bounds = [0, 2, 5, 9]
    o_sum, dq_sum = np.zeros_like(o), np.zeros_like(dq)
    for lo, hi in zip(bounds[:-1], bounds[1:]):
        ks, vs = k[:, :, lo:hi], v[:, :, lo:hi]
        o_sum += oracle.sigattn_fwd(q, ks, vs, scale, b, causal, slopes, pos0=-lo)
        g = oracle.sigattn_bwd(q, ks, vs, d_o, scale, b, causal, slopes, pos0=-lo)
        dq_sum += g[0]
        np.testing.assert_allclose(g[1], dk[:, :, lo:hi], rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(g[2], dv[:, :, lo:hi], rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(o_sum, o, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(dq_sum, dq, rtol=1e-12, atol=1e-15)
    lo, hi = 5, 9   # the last shard: queries 0..4 lie before all of its keys when causal
    part = oracle.sigattn_fwd(q, k[:, :, lo:hi], v[:, :, lo:hi], scale, b, causal, slopes, pos0=-lo)
    ref = np.zeros_like(part)
    for h in range(H):
        for i in range(N):
            for j in range(lo, hi):
                if causal and j > i:
                    continue
                x = scale * float(q[0, h, i] @ k[0, h, j]) + b - slopes[h] * abs(i - j)
                ref[0, h, i] += scalar_sigmoid(x) * v[0, h, j]
    np.testing.assert_allclose(part, ref, rtol=1e-13, atol=1e-16)
    if causal:
        assert np.all(part[:, :, :lo] == 0.0)


# ----------------------------------------------------------------------- padded batches


@pytest.mark.parametrize("causal", [False, True])
def test_padded_batch_equals_separate_unpadded_calls(causal):
    """seqlens: the valid part of every output equals the call on the unpadded sequence
    alone, whatever the padding holds; the padded part is exactly zero."""
    B, H, N, D = 3, 2, 7, 3
    q, k, v, d_o = (rnd((B, H, N, D), s) for s in (140, 141, 142, 143))
    lens = [7, 4, 1]
    slopes = np.array([0.5, 0.25])
    scale = 0.7
    bias = -np.log(np.array(lens, dtype=np.float64))     # b = -log n of each sample
    o = oracle.sigattn_fwd(q, k, v, scale, bias, causal, slopes, seqlens=lens)
    dq, dk, dv = oracle.sigattn_bwd(q, k, v, d_o, scale, bias, causal, slopes, seqlens=lens)
    db = oracle.sigattn_bwd_dbias(q, k, v, d_o, scale, bias, causal, slopes, seqlens=lens)
    for b, n in enumerate(lens):
        sel = (slice(b, b + 1), slice(None), slice(0, n))
        args = (q[sel], k[sel], v[sel])
        np.testing.assert_allclose(o[sel], oracle.sigattn_fwd(*args, scale, float(bias[b]), causal, slopes), rtol=1e-14, atol=1e-16)
        one = oracle.sigattn_bwd(*args, d_o[sel], scale, float(bias[b]), causal, slopes)
        for g, r in zip((dq, dk, dv), one):
            np.testing.assert_allclose(g[sel], r, rtol=1e-13, atol=1e-16)
        np.testing.assert_allclose(db[b], oracle.sigattn_bwd_dbias(*args, d_o[sel], scale, float(bias[b]), causal, slopes)[0], rtol=1e-13)
        for g in (o, dq, dk, dv):
            assert np.all(g[b, :, n:] == 0.0)
    # the padding must not matter
    q2, k2, v2, do2 = q.copy(), k.copy(), v.copy(), d_o.copy()
    for b, n in enumerate(lens):
        for t in (q2, k2, v2, do2):
            t[b, :, n:] = 1e3
    np.testing.assert_array_equal(oracle.sigattn_fwd(q2, k2, v2, scale, bias, causal, slopes, seqlens=lens), o)
    for g, r in zip(oracle.sigattn_bwd(q2, k2, v2, do2, scale, bias, causal, slopes, seqlens=lens), (dq, dk, dv)):
        np.testing.assert_array_equal(g, r)
    with pytest.raises(ValueError):
        oracle.sigattn_fwd(q, k, v, scale, -1.0, causal, seqlens=[7, 8, 1])


# ------------------------------------------------------- sequence-length normalisation


@pytest.mark.parametrize("alpha", [1.0, 0.5])
def test_seqlen_norm_matches_printed_n3_bases(alpha):
    """The causal row factors are the printed bases 1, 0.5, 0.33 raised to alpha (0.33 is
    1/3 to two places); without a mask every row gets n^-alpha."""
    bases = np.loadtxt(os.path.join(GOLDEN, "seqlen_norm_n3.txt"))
    r = oracle.seqlen_norm(3, alpha, True)
    np.testing.assert_allclose(r, bases ** alpha, rtol=1.1e-2)
    assert r[0] == 1.0 and r[1] == 0.5 ** alpha
    assert np.all(np.diff(r) < 0)          # more keys, smaller factor
    np.testing.assert_allclose(oracle.seqlen_norm(3, alpha, False), np.full(3, 3.0 ** -alpha), rtol=1e-15)
    # queries at the end of a longer key sequence count the keys they see
    np.testing.assert_allclose(oracle.seqlen_norm(2, alpha, True, n_k=5), np.array([4.0, 5.0]) ** -alpha, rtol=1e-15)
    assert oracle.seqlen_norm(3, alpha, True, n_k=4, pos0=-2)[:2].tolist() == [0.0, 0.0]


@pytest.mark.parametrize("causal", [False, True])
def test_seqlen_norm_q_zero_closed_form(causal):
    """Q = 0, b = 0: every kept weight is 1/2.  With alpha = 1 row i of O is half the mean
    of the values it sees (a running mean when causal); with alpha = 1/2 half the sum over
    sqrt(count)."""
    B, H, N, D = 2, 2, 9, 3
    q = np.zeros((B, H, N, D))
    k, v = rnd((B, H, N, D), 150), rnd((B, H, N, D), 151)
    count = np.arange(1, N + 1, dtype=np.float64) if causal else np.full(N, float(N))
    sums = np.cumsum(v, axis=2) if causal else np.repeat(v.sum(axis=2, keepdims=True), N, axis=2)
    for alpha in (1.0, 0.5):
        o = oracle.sigattn_fwd(q, k, v, 0.3, 0.0, causal, row_scale=oracle.seqlen_norm(N, alpha, causal))
        np.testing.assert_allclose(o, 0.5 * sums / (count ** alpha)[None, None, :, None], rtol=1e-13, atol=1e-15)


@pytest.mark.parametrize("causal", [False, True])
def test_row_scale_brute_force_and_finite_differences(causal):
    """Any vector of row factors: forward by explicit loops; gradients of L = sum(O * dO)
    with respect to Q, K, V and a per-(batch, head) bias by central differences."""
    B, H, N, D = 1, 2, 5, 3
    q, k, v, d_o = (rnd((B, H, N, D), s) for s in (160, 161, 162, 163))
    slopes = np.array([0.5, 0.125])
    scale = 0.6
    bias = np.array([[-0.7, 0.2]])
    r = np.array([1.0, 0.7, 0.1, 2.0, 0.0]) if not causal else oracle.seqlen_norm(N, 0.5, True)
    o = oracle.sigattn_fwd(q, k, v, scale, bias, causal, slopes, row_scale=r)
    ref = np.zeros_like(o)
    for h in range(H):
        for i in range(N):
            for j in range(N):
                if causal and j > i:
                    continue
                x = scale * float(q[0, h, i] @ k[0, h, j]) + bias[0, h] - slopes[h] * abs(i - j)
                ref[0, h, i] += r[i] * scalar_sigmoid(x) * v[0, h, j]
    np.testing.assert_allclose(o, ref, rtol=1e-13, atol=1e-16)

    def f():
        return float(np.sum(oracle.sigattn_fwd(q, k, v, scale, bias, causal, slopes, row_scale=r) * d_o))

    dq, dk, dv = oracle.sigattn_bwd(q, k, v, d_o, scale, bias, causal, slopes, row_scale=r)
    db = oracle.sigattn_bwd_dbias(q, k, v, d_o, scale, bias, causal, slopes, row_scale=r)
    step = 1e-6
    for name, x, g in (("q", q, dq), ("k", k, dk), ("v", v, dv), ("bias", bias, db)):
        fd = np.zeros_like(x)
        it = np.nditer(x, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            old = x[idx]
            x[idx] = old + step
            lp = f()
            x[idx] = old - step
            lm = f()
            x[idx] = old
            fd[idx] = (lp - lm) / (2 * step)
        err = np.linalg.norm(fd - g) / np.linalg.norm(fd)
        assert err < 1e-7, (name, err)
    # the factor must reach dV as well as dQ, dK: dropping it from any of them is far off
    plain = oracle.sigattn_bwd(q, k, v, d_o, scale, bias, causal, slopes)
    for g, pl in zip((dq, dk, dv), plain):
        assert np.linalg.norm(g - pl) / np.linalg.norm(g) > 0.05


# ------------------------------------------------------------------------ packed batches


@pytest.mark.parametrize("causal", [False, True])
def test_packed_batch_equals_separate_calls(causal):
    """cu_seqlens: sequences stored one after the other; every output equals the call on
    that sequence alone (with its own bias), including an empty sequence in the middle."""
    H, D = 2, 3
    lens = [4, 0, 7, 1]
    cu = np.concatenate([[0], np.cumsum(lens)])
    T = int(cu[-1])
    q, k, v, d_o = (rnd((1, H, T, D), s) for s in (170, 171, 172, 173))
    slopes = np.array([0.5, 0.25])
    scale = 0.7
    bias = np.array([[-1.0, -0.5], [9.0, 9.0], [-2.0, 0.3], [0.0, -3.0]])   # per (sequence, head)
    o = oracle.sigattn_fwd(q, k, v, scale, bias, causal, slopes, cu_seqlens=cu)
    dq, dk, dv = oracle.sigattn_bwd(q, k, v, d_o, scale, bias, causal, slopes, cu_seqlens=cu)
    db = oracle.sigattn_bwd_dbias(q, k, v, d_o, scale, bias, causal, slopes, cu_seqlens=cu)
    assert db.shape == (4, H) and np.all(db[1] == 0.0)
    for s, n in enumerate(lens):
        if n == 0:
            continue
        sel = (slice(None), slice(None), slice(int(cu[s]), int(cu[s + 1])))
        b = bias[s][None, :]
        np.testing.assert_allclose(o[sel], oracle.sigattn_fwd(q[sel], k[sel], v[sel], scale, b, causal, slopes),
                                   rtol=1e-13, atol=1e-16)
        one = oracle.sigattn_bwd(q[sel], k[sel], v[sel], d_o[sel], scale, b, causal, slopes)
        for g, r in zip((dq, dk, dv), one):
            np.testing.assert_allclose(g[sel], r, rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(db[s], oracle.sigattn_bwd_dbias(q[sel], k[sel], v[sel], d_o[sel], scale, b, causal, slopes)[0],
                                   rtol=1e-12)
    # one sequence is the plain call
    np.testing.assert_allclose(oracle.sigattn_fwd(q, k, v, scale, -1.0, causal, slopes, cu_seqlens=[0, T]),
                               oracle.sigattn_fwd(q, k, v, scale, -1.0, causal, slopes), rtol=1e-14)
    with pytest.raises(ValueError):
        oracle.sigattn_fwd(q, k, v, scale, -1.0, causal, cu_seqlens=[0, 5, 3, T])


@pytest.mark.parametrize("causal", [True, False])
def test_packed_batch_brute_force_with_shared_kv_heads(causal):
    """Explicit loops over the packed layout with one key/value head for two query heads:
    forward, and every gradient of L = sum(O * dO) written out entry by entry (dK and dV of
    the shared head are sums over both query heads, db is per (sequence, head))."""
    H, D = 2, 2
    cu = [0, 3, 5]
    q, d_o = rnd((1, H, 5, D), 180), rnd((1, H, 5, D), 183)
    k, v = rnd((1, 1, 5, D), 181), rnd((1, 1, 5, D), 182)
    scale, bias = 0.9, np.array([[-0.4, 0.1], [0.6, -1.1]])
    slopes = np.array([0.3, 0.0])
    o = oracle.sigattn_fwd(q, k, v, scale, bias, causal, slopes, cu_seqlens=cu)
    dq, dk, dv = oracle.sigattn_bwd(q, k, v, d_o, scale, bias, causal, slopes, cu_seqlens=cu)
    db = oracle.sigattn_bwd_dbias(q, k, v, d_o, scale, bias, causal, slopes, cu_seqlens=cu)
    ref = np.zeros_like(o)
    rdq, rdk, rdv, rdb = np.zeros_like(q), np.zeros_like(k), np.zeros_like(v), np.zeros((2, H))
    for h in range(H):
        for s in range(2):
            for i in range(cu[s], cu[s + 1]):
                for j in range(cu[s], (i + 1) if causal else cu[s + 1]):
                    x = scale * float(q[0, h, i] @ k[0, 0, j]) + bias[s, h] - slopes[h] * abs(i - j)
                    pw = scalar_sigmoid(x)
                    ref[0, h, i] += pw * v[0, 0, j]
                    g = pw * (1.0 - pw) * float(d_o[0, h, i] @ v[0, 0, j])   # dL/dx_ij
                    rdv[0, 0, j] += pw * d_o[0, h, i]
                    rdq[0, h, i] += scale * g * k[0, 0, j]
                    rdk[0, 0, j] += scale * g * q[0, h, i]
                    rdb[s, h] += g
    np.testing.assert_allclose(o, ref, rtol=1e-13, atol=1e-16)
    for got, want in ((dq, rdq), (dk, rdk), (dv, rdv), (db, rdb)):
        np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-15)


@pytest.mark.parametrize("causal", [True, False])
def test_packed_batch_shared_kv_heads_finite_differences(causal):
    """Central differences of L = sum(O * dO) with respect to every entry of q, of the shared k
    and v, and of the per-(sequence, head) bias, for a packed batch with H_kv < H (two groups of
    two query heads, an empty sequence in the middle)."""
    H, H_kv, D = 4, 2, 3
    cu = [0, 2, 2, 6]
    T = cu[-1]
    q, d_o = rnd((1, H, T, D), 190), rnd((1, H, T, D), 193)
    k, v = rnd((1, H_kv, T, D), 191), rnd((1, H_kv, T, D), 192)
    bias = rnd((3, H), 194)
    slopes = np.array([0.5, 0.25, 0.0, 0.125])
    scale = 0.6

    def L(bq, bk, bv, bb):
        return float(np.sum(oracle.sigattn_fwd(bq, bk, bv, scale, bb, causal, slopes, cu_seqlens=cu) * d_o))

    dq, dk, dv = oracle.sigattn_bwd(q, k, v, d_o, scale, bias, causal, slopes, cu_seqlens=cu)
    db = oracle.sigattn_bwd_dbias(q, k, v, d_o, scale, bias, causal, slopes, cu_seqlens=cu)
    assert np.all(db[1] == 0.0)
    h = 1e-6
    args = [q.copy(), k.copy(), v.copy(), bias.copy()]
    for which, g in enumerate((dq, dk, dv, db)):
        fd = np.zeros_like(g)
        x = args[which]
        for idx in np.ndindex(*x.shape):
            old = x[idx]
            x[idx] = old + h
            lp = L(*args)
            x[idx] = old - h
            lm = L(*args)
            x[idx] = old
            fd[idx] = (lp - lm) / (2 * h)
        assert np.linalg.norm(fd - g) / np.linalg.norm(fd) < 1e-7, which
