"""Oracle vs hand-derived worked examples (tests/golden/attn_jvp_hand_examples.txt)."""
import math
import os

import numpy as np
import pytest

GOLD = os.path.join(os.path.dirname(__file__), "golden", "attn_jvp_hand_examples.txt")


def _load():
    vals = {}
    with open(GOLD) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if "=" in line:
                k, v = line.split("=")
                vals[k.strip()] = float(v)
    return vals


def _example_a():
    ln3 = math.log(3.0)
    return dict(Q=[[1.0]], K=[[0.0], [ln3]], V=[[1.0], [5.0]],
                tQ=[[1.0]], tK=[[1.0], [0.0]], tV=[[2.0], [-1.0]], scale=1.0)


def _example_b():
    return dict(Q=[[1, 0], [0, 2]], K=[[1, 0], [0, 1], [1, 1]], V=[[1, 2], [3, 4], [5, 6]],
                tQ=[[0, 1], [1, 0]], tK=[[1, 0], [0, -1], [.5, .5]], tV=[[0, 1], [1, 0], [-1, 2]],
                scale=0.5)


@pytest.mark.parametrize("route", ["def", "fold_1", "fold_2", "fold_64"])
def test_example_a(oracle, route):
    g = _load()
    ex = _example_a()
    if route == "def":
        O, tO, LSE, MU = oracle.attn_jvp_def(**ex)
    else:
        O, tO, LSE, MU = oracle.attn_jvp_fold(**ex, Bc=int(route.split("_")[1]))
    assert O[0, 0] == pytest.approx(g["A.O"], abs=1e-13)
    assert LSE[0] == pytest.approx(g["A.LSE"], abs=1e-13)
    assert MU[0] == pytest.approx(g["A.mu"], abs=1e-13)
    assert tO[0, 0] == pytest.approx(g["A.tO"], abs=1e-13)
    # the closed forms themselves
    assert g["A.tO"] == pytest.approx(0.75 * math.log(3) - 1, abs=1e-15)
    assert g["A.mu"] == pytest.approx(0.25 + 0.75 * math.log(3), abs=1e-15)


@pytest.mark.parametrize("route", ["def", "fold_1", "fold_2", "fold_3"])
def test_example_b(oracle, route):
    g = _load()
    ex = _example_b()
    if route == "def":
        O, tO, LSE, MU = oracle.attn_jvp_def(**ex)
    else:
        O, tO, LSE, MU = oracle.attn_jvp_fold(**ex, Bc=int(route.split("_")[1]))
    want_O = np.array([[g["B.O00"], g["B.O01"]], [g["B.O10"], g["B.O11"]]])
    want_tO = np.array([[g["B.tO00"], g["B.tO01"]], [g["B.tO10"], g["B.tO11"]]])
    np.testing.assert_allclose(O, want_O, atol=1e-13, rtol=0)
    np.testing.assert_allclose(tO, want_tO, atol=1e-13, rtol=0)
    np.testing.assert_allclose(LSE, [g["B.LSE0"], g["B.LSE1"]], atol=1e-13, rtol=0)
    np.testing.assert_allclose(MU, [g["B.mu0"], g["B.mu1"]], atol=1e-13, rtol=0)


def test_example_b_transposed_operands_would_fail(oracle):
    """The example is asymmetric enough that swapping tQ<->Q in the tS term changes tO."""
    g = _load()
    ex = _example_b()
    ex["tQ"], ex["Q"] = ex["Q"], ex["tQ"]
    _, tO, _, _ = oracle.attn_jvp_def(**ex)
    assert abs(tO[0, 0] - g["B.tO00"]) > 1e-3
