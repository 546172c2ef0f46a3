"""Oracle vs PyTorch's built-in forward-mode operator (the routine the paper's kernel replaces,
Sec. 3.2) applied to a textbook softmax attention in fp64, and the bf16 [B][L][H][D] wrapper."""
import numpy as np
import pytest
import torch

from paper_2510_08431_b200 import synth


def _attn(q, k, v, s):
    return torch.softmax(s * q @ k.T, dim=-1) @ v


def _lse(q, k, s):
    return torch.logsumexp(s * q @ k.T, dim=-1)


@pytest.mark.parametrize("Lq,Lk,D,s", [(37, 53, 16, 0.25), (3, 5, 1, 1.0), (16, 700, 64, 0.125), (130, 129, 8, 0.3)])
def test_vs_torch_func_jvp(oracle, Lq, Lk, D, s):
    g = torch.Generator().manual_seed(Lq + Lk)
    r = lambda L: torch.randn(L, D, generator=g, dtype=torch.float64)
    Q, K, V, tQ, tK, tV = r(Lq), r(Lk), r(Lk), r(Lq), r(Lk), r(Lk)
    want_O, want_tO = torch.func.jvp(lambda a, b, c: _attn(a, b, c, s), (Q, K, V), (tQ, tK, tV))
    want_L, want_mu = torch.func.jvp(lambda a, b: _lse(a, b, s), (Q, K), (tQ, tK))
    for got in (oracle.attn_jvp_def(*[x.numpy() for x in (Q, K, V, tQ, tK, tV)], s),
                oracle.attn_jvp_fold(*[x.numpy() for x in (Q, K, V, tQ, tK, tV)], s, Bc=32)):
        O, tO, LSE, MU = got
        np.testing.assert_allclose(O, want_O.numpy(), atol=1e-13)
        np.testing.assert_allclose(tO, want_tO.numpy(), atol=1e-13)
        np.testing.assert_allclose(LSE, want_L.numpy(), atol=1e-13)
        np.testing.assert_allclose(MU, want_mu.numpy(), atol=1e-13)


@pytest.mark.parametrize("tangent_free", [False, True])
def test_bf16_blhd_rows_wrapper(oracle, tangent_free):
    """The strided bf16 wrapper picks the right (b, h, i) slices and widens bf16 exactly."""
    B, H, Lq, Lk, D = 2, 3, 10, 17, 8
    x = synth.make_inputs(B, H, Lq, Lk, D, 1.0, 0.5, seed=5, kv_tangent_free=tangent_free)
    s = 0.37
    rows = [0, 7, 29, 30, 59, 13, 41]  # unsorted on purpose
    bits = {k: (None if v is None else synth.bf16_bits(v)) for k, v in x.items()}
    O, tO, LSE, MU = oracle.attn_jvp_def_bf16_rows(bits["q"], bits["k"], bits["v"], bits["tq"], bits["tk"],
                                                   bits["tv"], B, H, Lq, Lk, D, s, rows)
    for n, r in enumerate(rows):
        bh, i = divmod(r, Lq)
        b, h = divmod(bh, H)
        sl = lambda t: None if t is None else t[b, :, h, :].to(torch.float64)
        Q, K, V, tQ = sl(x["q"])[i:i + 1], sl(x["k"]), sl(x["v"]), sl(x["tq"])[i:i + 1]
        tK = torch.zeros_like(K) if tangent_free else sl(x["tk"])
        tV = torch.zeros_like(V) if tangent_free else sl(x["tv"])
        wO, wtO = torch.func.jvp(lambda a, b_, c: _attn(a, b_, c, s), (Q, K, V), (tQ, tK, tV))
        wL, wmu = torch.func.jvp(lambda a, b_: _lse(a, b_, s), (Q, K), (tQ, tK))
        np.testing.assert_allclose(O[n], wO[0].numpy(), atol=1e-13)
        np.testing.assert_allclose(tO[n], wtO[0].numpy(), atol=1e-13)
        assert abs(LSE[n] - wL.item()) < 1e-13 and abs(MU[n] - wmu.item()) < 1e-13


def test_synth_is_deterministic_and_bf16():
    a = synth.make_inputs(1, 2, 5, 7, 8, seed=3)
    b = synth.make_inputs(1, 2, 5, 7, 8, seed=3)
    for k in a:
        assert a[k].dtype == torch.bfloat16 and torch.equal(a[k], b[k])
    assert a["q"].shape == (1, 5, 2, 8) and a["k"].shape == (1, 7, 2, 8)
    rows = synth.sample_rows(1, 2, 300, n_random_per_head=3, tile=128, full_tiles=(0,), heads_full=(0,))
    assert set(range(256, 300)) <= set(rows) and set(range(0, 128)) <= set(rows)
    assert rows == sorted(rows) and max(rows) < 600
