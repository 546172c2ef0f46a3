"""Oracle tangents vs central finite differences of the oracle's own primal outputs.

tO must equal d/d(eps) O(x + eps t) and mu must equal d/d(eps) LSE(x + eps t):
(f(x + eps t) - f(x - eps t)) / (2 eps) at eps = 1e-4 has O(eps^2) error.
This pins every term of the tangent formula (a dropped term, a wrong sign or a
swapped operand changes the derivative) without reference to another implementation.
"""
import numpy as np
import pytest

EPS = 1e-4


def _rand(rng, Lq, Lk, D, st=1.0):
    f = lambda L, s: rng.standard_normal((L, D)) * s
    return dict(Q=f(Lq, 1), K=f(Lk, 1), V=f(Lk, 1), tQ=f(Lq, st), tK=f(Lk, st), tV=f(Lk, st))


def _fd(oracle, x, scale, which=("tQ", "tK", "tV")):
    plus = {k: x[k] + EPS * x["t" + k] if ("t" + k) in which else x[k] for k in ("Q", "K", "V")}
    minus = {k: x[k] - EPS * x["t" + k] if ("t" + k) in which else x[k] for k in ("Q", "K", "V")}
    z = np.zeros_like
    Op, _, Lp, _ = oracle.attn_jvp_def(plus["Q"], plus["K"], plus["V"], z(x["Q"]), z(x["K"]), z(x["V"]), scale)
    Om, _, Lm, _ = oracle.attn_jvp_def(minus["Q"], minus["K"], minus["V"], z(x["Q"]), z(x["K"]), z(x["V"]), scale)
    return (Op - Om) / (2 * EPS), (Lp - Lm) / (2 * EPS)


@pytest.mark.parametrize("Lq,Lk,D,scale", [(37, 53, 16, 0.25), (8, 300, 64, 0.125), (5, 1, 8, 1.0),
                                          (16, 2048, 128, 128 ** -0.5)])
@pytest.mark.parametrize("route", ["def", "fold"])
def test_fd_all_tangents(oracle, Lq, Lk, D, scale, route):
    rng = np.random.default_rng(Lq * 1000 + Lk)
    x = _rand(rng, Lq, Lk, D)
    if route == "def":
        _, tO, _, MU = oracle.attn_jvp_def(x["Q"], x["K"], x["V"], x["tQ"], x["tK"], x["tV"], scale)
    else:
        _, tO, _, MU = oracle.attn_jvp_fold(x["Q"], x["K"], x["V"], x["tQ"], x["tK"], x["tV"], scale, Bc=48)
    fd_tO, fd_mu = _fd(oracle, x, scale)
    assert np.abs(tO - fd_tO).max() <= 1e-6 * max(1.0, np.abs(tO).max())
    assert np.abs(MU - fd_mu).max() <= 1e-6 * max(1.0, np.abs(MU).max())


@pytest.mark.parametrize("only", ["tQ", "tK", "tV"])
def test_fd_one_tangent_at_a_time(oracle, only):
    """Each of the three partial derivatives separately (catches cancelling mistakes)."""
    rng = np.random.default_rng(7)
    x = _rand(rng, 19, 41, 12)
    t = {k: (x[k] if k == only else np.zeros_like(x[k])) for k in ("tQ", "tK", "tV")}
    _, tO, _, MU = oracle.attn_jvp_def(x["Q"], x["K"], x["V"], t["tQ"], t["tK"], t["tV"], 0.3)
    fd_tO, fd_mu = _fd(oracle, x, 0.3, which=(only,))
    assert np.abs(tO - fd_tO).max() <= 1e-6 * max(1.0, np.abs(tO).max())
    assert np.abs(MU - fd_mu).max() <= 1e-6
    if only == "tV":
        assert np.abs(MU).max() == 0.0  # LSE does not depend on V


def test_fd_none_tangents_mean_zero(oracle):
    """tK = tV = None (constant cross-attention context) equals explicit zeros and FD in Q only."""
    rng = np.random.default_rng(11)
    x = _rand(rng, 9, 77, 32)
    z = np.zeros_like(x["K"])
    a = oracle.attn_jvp_def(x["Q"], x["K"], x["V"], x["tQ"], None, None, 0.2)
    b = oracle.attn_jvp_def(x["Q"], x["K"], x["V"], x["tQ"], z, z, 0.2)
    c = oracle.attn_jvp_fold(x["Q"], x["K"], x["V"], x["tQ"], None, None, 0.2, Bc=16)
    for u, v, w in zip(a, b, c):
        np.testing.assert_array_equal(u, v)
        np.testing.assert_allclose(u, w, atol=1e-13, rtol=0)
    fd_tO, _ = _fd(oracle, x, 0.2, which=("tQ",))
    assert np.abs(a[1] - fd_tO).max() <= 1e-6
