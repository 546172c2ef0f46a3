"""Pins of the RMS-norm JVP oracle: finite differences, PyTorch forward-mode on a textbook RMSNorm,
scale invariance (a tangent along x vanishes), linearity, a hand-computed row."""
import math

import numpy as np
import pytest
import torch


def _rand(rows, D, seed):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((rows, D)), rng.standard_normal((rows, D)), rng.standard_normal(D)


def test_finite_differences(oracle):
    x, tx, w = _rand(7, 16, 0)
    e = 1e-5
    y, ty = oracle.rmsnorm_jvp(x, tx, w, 1e-6)
    yp, _ = oracle.rmsnorm_jvp(x + e * tx, None, w, 1e-6)
    ym, _ = oracle.rmsnorm_jvp(x - e * tx, None, w, 1e-6)
    assert np.abs((yp - ym) / (2 * e) - ty).max() < 1e-8


@pytest.mark.parametrize("D", [1, 8, 128])
def test_against_torch_forward_mode(oracle, D):
    x, tx, w = _rand(5, D, D)
    eps = 1e-5
    f = lambda a: a * torch.rsqrt(a.pow(2).mean(-1, keepdim=True) + eps) * torch.from_numpy(w)
    wy, wty = torch.func.jvp(f, (torch.from_numpy(x),), (torch.from_numpy(tx),))
    y, ty = oracle.rmsnorm_jvp(x, tx, w, eps)
    np.testing.assert_allclose(y, wy.numpy(), atol=1e-13)
    np.testing.assert_allclose(ty, wty.numpy(), atol=1e-13)


def test_tangent_along_x_vanishes_without_eps(oracle):
    """RMSNorm(c x) = RMSNorm(x) for c > 0 when eps = 0, so the derivative in the direction x is 0."""
    x, _, w = _rand(6, 32, 3)
    _, ty = oracle.rmsnorm_jvp(x, 2.5 * x, w, 0.0)
    assert np.abs(ty).max() < 1e-14


def test_linearity_and_hand_row(oracle):
    x, t1, w = _rand(4, 8, 4)
    _, t2, _ = _rand(4, 8, 5)
    _, a = oracle.rmsnorm_jvp(x, t1, w, 1e-6)
    _, b = oracle.rmsnorm_jvp(x, t2, w, 1e-6)
    _, c = oracle.rmsnorm_jvp(x, 2 * t1 - 3 * t2, w, 1e-6)
    np.testing.assert_allclose(c, 2 * a - 3 * b, atol=1e-13)
    # x = (3, 4), w = (1, 2), eps = 0: n = sqrt(12.5); tx = (1, 0): x.tx = 3
    y, ty = oracle.rmsnorm_jvp([[3.0, 4.0]], [[1.0, 0.0]], [1.0, 2.0], 0.0)
    n = math.sqrt(12.5)
    np.testing.assert_allclose(y, [[3 / n, 8 / n]], atol=1e-15)
    np.testing.assert_allclose(ty, [[1 / n - 3 * 3 / (2 * n ** 3), 2 * (0 - 4 * 3 / (2 * n ** 3))]], atol=1e-15)
