"""The chunk-merge identity used by the split-KV entry point, pinned on the CPU: running the oracle on chunks of
the keys and merging must reproduce the oracle on all keys (both are exact in real arithmetic)."""
import numpy as np
import pytest


@pytest.mark.parametrize("cuts", [[17], [1, 2], [10, 30, 31], [5, 6, 7, 8, 9]])
def test_chunk_merge_reproduces_full_result(oracle, cuts):
    rng = np.random.default_rng(len(cuts))
    Lq, Lk, D, s = 9, 40, 6, 0.4
    f = lambda L: rng.standard_normal((L, D))
    Q, K, V, tQ, tK, tV = f(Lq) * 2, f(Lk), f(Lk), f(Lq), f(Lk), f(Lk)
    ref = oracle.attn_jvp_def(Q, K, V, tQ, tK, tV, s)
    edges = [0] + cuts + [Lk]
    parts = [oracle.attn_jvp_def(Q, K[a:b], V[a:b], tQ, tK[a:b], tV[a:b], s) for a, b in zip(edges[:-1], edges[1:])]
    got = oracle.splitkv_merge([p[0] for p in parts], [p[1] for p in parts], [p[2] for p in parts], [p[3] for p in parts])
    for u, v in zip(ref, got):
        np.testing.assert_allclose(v, u, atol=1e-12, rtol=0)


def test_merge_of_one_chunk_is_identity(oracle):
    rng = np.random.default_rng(0)
    f = lambda L: rng.standard_normal((L, 4))
    ref = oracle.attn_jvp_def(f(3), f(5), f(5), f(3), f(5), f(5), 1.0)
    got = oracle.splitkv_merge([ref[0]], [ref[1]], [ref[2]], [ref[3]])
    for u, v in zip(ref, got):
        np.testing.assert_allclose(v, u, atol=1e-15, rtol=0)
