"""Oracle vs what the mathematics fixes: linearity, special cases, closed forms, invariances."""
import itertools

import numpy as np
import pytest


def _rand(rng, Lq, Lk, D):
    f = lambda L: rng.standard_normal((L, D))
    return [f(Lq), f(Lk), f(Lk), f(Lq), f(Lk), f(Lk)]


ROUTES = ["def", "fold"]


def _call(oracle, route, Q, K, V, tQ, tK, tV, s, Bc=7):
    if route == "def":
        return oracle.attn_jvp_def(Q, K, V, tQ, tK, tV, s)
    return oracle.attn_jvp_fold(Q, K, V, tQ, tK, tV, s, Bc=Bc)


@pytest.mark.parametrize("route", ROUTES)
def test_linearity_and_zero_tangent(oracle, route):
    rng = np.random.default_rng(0)
    Q, K, V, tQ1, tK1, tV1 = _rand(rng, 13, 29, 8)
    _, _, _, tQ2, tK2, tV2 = _rand(rng, 13, 29, 8)
    a, b = 1.7, -0.6
    O, t1, L, m1 = _call(oracle, route, Q, K, V, tQ1, tK1, tV1, 0.35)
    _, t2, _, m2 = _call(oracle, route, Q, K, V, tQ2, tK2, tV2, 0.35)
    _, t12, _, m12 = _call(oracle, route, Q, K, V, a * tQ1 + b * tQ2, a * tK1 + b * tK2, a * tV1 + b * tV2, 0.35)
    np.testing.assert_allclose(t12, a * t1 + b * t2, atol=1e-12, rtol=0)
    np.testing.assert_allclose(m12, a * m1 + b * m2, atol=1e-12, rtol=0)
    z = np.zeros_like
    O0, t0, L0, m0 = _call(oracle, route, Q, K, V, z(Q), z(K), z(V), 0.35)
    assert np.all(t0 == 0.0) and np.all(m0 == 0.0)
    np.testing.assert_array_equal(O0, O)
    np.testing.assert_array_equal(L0, L)


@pytest.mark.parametrize("route", ROUTES)
def test_single_key(oracle, route):
    """Lk = 1: P = 1, so O = V_0, tO = tV_0, LSE = s q.k_0, mu = s (tq.k_0 + q.tk_0)."""
    rng = np.random.default_rng(1)
    Q, K, V, tQ, tK, tV = _rand(rng, 6, 1, 5)
    O, tO, LSE, MU = _call(oracle, route, Q, K, V, tQ, tK, tV, 0.7)
    np.testing.assert_allclose(O, np.repeat(V, 6, 0), atol=1e-15)
    np.testing.assert_allclose(tO, np.repeat(tV, 6, 0), atol=1e-15)
    np.testing.assert_allclose(LSE, 0.7 * (Q @ K[0]), atol=1e-14)
    np.testing.assert_allclose(MU, 0.7 * (tQ @ K[0] + Q @ tK[0]), atol=1e-14)


@pytest.mark.parametrize("route", ROUTES)
def test_primal_is_plain_softmax_attention(oracle, route):
    """O and LSE against the textbook formula computed with numpy/scipy primitives."""
    from scipy.special import logsumexp, softmax
    rng = np.random.default_rng(2)
    Q, K, V, tQ, tK, tV = _rand(rng, 11, 23, 6)
    O, _, LSE, _ = _call(oracle, route, Q, K, V, tQ, tK, tV, 0.4)
    S = 0.4 * Q @ K.T
    np.testing.assert_allclose(O, softmax(S, axis=1) @ V, atol=1e-13)
    np.testing.assert_allclose(LSE, logsumexp(S, axis=1), atol=1e-13)


@pytest.mark.parametrize("route", ROUTES)
def test_tq_tk_zero_is_attention_on_tv(oracle, route):
    """tQ = tK = 0 => tS = 0 => tO = P tV: plain attention with V := tV."""
    from scipy.special import softmax
    rng = np.random.default_rng(3)
    Q, K, V, tQ, tK, tV = _rand(rng, 9, 17, 4)
    _, tO, _, MU = _call(oracle, route, Q, K, V, 0 * tQ, 0 * tK, tV, 0.5)
    np.testing.assert_allclose(tO, softmax(0.5 * Q @ K.T, axis=1) @ tV, atol=1e-13)
    assert np.all(MU == 0)


@pytest.mark.parametrize("route", ROUTES)
def test_zero_query_closed_form(oracle, route):
    """Q = 0 => P uniform: O = mean V, LSE = ln Lk,
    tO_i = (s/Lk) sum_j (c_ij - mean_j c_ij) V_j + mean tV with c_ij = tQ_i.K_j."""
    rng = np.random.default_rng(4)
    Q, K, V, tQ, tK, tV = _rand(rng, 7, 19, 5)
    Q = np.zeros_like(Q)
    s = 0.9
    O, tO, LSE, MU = _call(oracle, route, Q, K, V, tQ, tK, tV, s)
    np.testing.assert_allclose(O, np.repeat(V.mean(0, keepdims=True), 7, 0), atol=1e-14)
    np.testing.assert_allclose(LSE, np.log(19.0), atol=1e-14)
    c = tQ @ K.T
    want = (s / 19.0) * (c - c.mean(1, keepdims=True)) @ V + tV.mean(0, keepdims=True)
    np.testing.assert_allclose(tO, want, atol=1e-13)
    np.testing.assert_allclose(MU, s * c.mean(1), atol=1e-13)


@pytest.mark.parametrize("route", ROUTES)
def test_constant_values_give_zero_tangent(oracle, route):
    """All V rows equal and tV = 0: O is constant in Q,K so tO = 0 for any tQ, tK."""
    rng = np.random.default_rng(5)
    Q, K, V, tQ, tK, tV = _rand(rng, 8, 21, 6)
    V = np.repeat(V[:1], 21, 0)
    O, tO, _, _ = _call(oracle, route, Q, K, V, tQ, tK, 0 * tV, 0.6)
    np.testing.assert_allclose(O, np.repeat(V[:1], 8, 0), atol=1e-14)
    assert np.abs(tO).max() < 1e-13


@pytest.mark.parametrize("route", ROUTES)
def test_row_shift_invariance(oracle, route):
    """K[:, -1] = 1 and tK = 0: tQ[:, -1] only adds a per-row constant to tS, which cancels in tO
    (softmax is shift invariant) but shows up in mu."""
    rng = np.random.default_rng(6)
    Q, K, V, tQ, tK, tV = _rand(rng, 8, 21, 6)
    K[:, -1] = 1.0
    tK = np.zeros_like(tK)
    _, a, _, ma = _call(oracle, route, Q, K, V, tQ, tK, tV, 0.6)
    tQ2 = tQ.copy()
    tQ2[:, -1] += rng.standard_normal(8) * 3
    _, b, _, mb = _call(oracle, route, Q, K, V, tQ2, tK, tV, 0.6)
    np.testing.assert_allclose(a, b, atol=1e-12)
    np.testing.assert_allclose(mb - ma, 0.6 * (tQ2[:, -1] - tQ[:, -1]), atol=1e-12)


@pytest.mark.parametrize("route", ROUTES)
def test_key_permutation_invariance(oracle, route):
    rng = np.random.default_rng(8)
    Q, K, V, tQ, tK, tV = _rand(rng, 5, 33, 4)
    perm = rng.permutation(33)
    a = _call(oracle, route, Q, K, V, tQ, tK, tV, 0.5)
    b = _call(oracle, route, Q, K[perm], V[perm], tQ, tK[perm], tV[perm], 0.5)
    for u, v in zip(a, b):
        np.testing.assert_allclose(u, v, atol=1e-13)


def test_scale_is_not_differentiated_and_enters_both_s_and_ts(oracle):
    """Scaling Q and tQ by c with scale s equals scale c*s with the original Q, tQ (tK = 0)."""
    rng = np.random.default_rng(9)
    Q, K, V, tQ, tK, tV = _rand(rng, 6, 14, 4)
    a = oracle.attn_jvp_def(2.5 * Q, K, V, 2.5 * tQ, 0 * tK, tV, 0.2)
    b = oracle.attn_jvp_def(Q, K, V, tQ, 0 * tK, tV, 0.5)
    for u, v in zip(a, b):
        np.testing.assert_allclose(u, v, atol=1e-13)


def test_block_fold_equals_definition_on_tiny_shapes_brute_force(oracle):
    """Every Lq, Lk in {1,2,3,5}, D in {1,2,4}, Bc in {1,2,3,64}: the streaming route reorders sums only."""
    rng = np.random.default_rng(10)
    for Lq, Lk, D in itertools.product((1, 2, 3, 5), (1, 2, 3, 5), (1, 2, 4)):
        Q, K, V, tQ, tK, tV = _rand(rng, Lq, Lk, D)
        ref = oracle.attn_jvp_def(Q, K, V, tQ, tK, tV, 0.8)
        for Bc in (1, 2, 3, 64):
            got = oracle.attn_jvp_fold(Q, K, V, tQ, tK, tV, 0.8, Bc=Bc)
            for u, v in zip(ref, got):
                assert np.abs(u - v).max() <= 1e-12 * (1 + np.abs(u).max())


def test_block_fold_block_size_independence_long_rows(oracle):
    rng = np.random.default_rng(12)
    Q, K, V, tQ, tK, tV = _rand(rng, 4, 1000, 32)
    Q *= 3  # peaked softmax: running max changes late, exercises the rescale terms
    ref = oracle.attn_jvp_def(Q, K, V, tQ, tK, tV, 0.3)
    for Bc in (1, 64, 128, 333, 1000, 4096):
        got = oracle.attn_jvp_fold(Q, K, V, tQ, tK, tV, 0.3, Bc=Bc)
        for u, v in zip(ref, got):
            assert np.abs(u - v).max() <= 1e-11 * (1 + np.abs(u).max())


def test_increasing_maxima_rescale_path(oracle):
    """Keys ordered so that every block raises the running max (alpha < 1 at every step)."""
    rng = np.random.default_rng(13)
    Q, K, V, tQ, tK, tV = _rand(rng, 3, 64, 8)
    K = K * np.linspace(0.1, 6.0, 64)[:, None]
    ref = oracle.attn_jvp_def(Q, K, V, tQ, tK, tV, 1.0)
    got = oracle.attn_jvp_fold(Q, K, V, tQ, tK, tV, 1.0, Bc=4)
    for u, v in zip(ref, got):
        assert np.abs(u - v).max() <= 1e-11 * (1 + np.abs(u).max())
