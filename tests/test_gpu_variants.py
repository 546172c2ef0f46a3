"""The kernel variants behind one entry point: one or two softmax warpgroups per CTA, and one CTA per query tile
or a CTA pair per 256-row query block (attn_jvp_set_tuning).  Every variant must pass the same oracle gates; with one
softmax group the pair and the single-CTA kernels run the same arithmetic in the same order and must agree to the
bit.  Shapes cover an odd number of query tiles (the pair's second CTA then has no rows), ragged tails, many short
work items per persistent CTA, and back-to-back launches without a host synchronisation in between."""
import numpy as np
import pytest
import torch

from paper_2510_08431_b200 import synth
from tests import gpu_util as U

pytestmark = pytest.mark.gpu

GROUPS, PAIR = 1, 2     # knobs of attn_jvp_set_tuning


@pytest.fixture(scope="module")
def aj():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2510_08431_b200 import build
    build.build_library()
    import paper_2510_08431_b200 as aj
    aj.load()
    yield aj
    aj.attn_jvp_set_tuning(GROUPS, 0)
    aj.attn_jvp_set_tuning(PAIR, 0)


def _run(aj, g, scale, mode, groups, pair):
    assert aj.attn_jvp_set_tuning(GROUPS, groups) == 0 and aj.attn_jvp_set_tuning(PAIR, pair) == 0
    try:
        return U.run(aj, g, scale, fwd_only=(mode == "fwd"))
    finally:
        aj.attn_jvp_set_tuning(GROUPS, 0)
        aj.attn_jvp_set_tuning(PAIR, 0)


@pytest.mark.parametrize("mode", ["jvp", "kv_free", "fwd"])
@pytest.mark.parametrize("shape", [(1, 2, 300, 1000), (2, 3, 129, 65), (1, 3, 128 * 7 + 5, 64 * 9 + 1), (1, 2, 2048, 4096)])
def test_every_variant_against_the_oracle(aj, oracle, mode, shape):
    B, H, Lq, Lk = shape
    D = 128
    x = synth.make_inputs(B, H, Lq, Lk, D, 1.0, 0.5, seed=300 + Lq, kv_tangent_free=(mode != "jvp"))
    g = U.to_gpu(x)
    scale = D ** -0.5
    rows = np.arange(B * H * Lq) if B * H * Lq <= 2048 else np.arange(0, B * H * Lq, 7)
    ref = None
    for groups in (1, 2):
        for pair in (1, 2):
            o, to, lse = _run(aj, g, scale, mode, groups, pair)
            U.check_all(oracle, aj, x, B, H, Lq, Lk, D, scale, rows, o, to, lse)
            if groups == 1:
                if ref is None:
                    ref = (o, to, lse)
                elif mode == "fwd":
                    # the forward-only kernel takes 128 keys per tile on one CTA and 64 in the pair: another order
                    # of summation, equal to one bf16 ulp
                    assert (o.float() - ref[0].float()).abs().max().item() <= 2.0 ** -7 * ref[0].float().abs().max().item()
                    assert (lse - ref[2]).abs().max().item() <= 1e-5
                else:   # same arithmetic, same order: the CTA pair only changes who issues the MMAs
                    assert torch.equal(o, ref[0]) and torch.equal(lse, ref[2])
                    assert to is None or torch.equal(to, ref[1])


def test_d64_groups_against_the_oracle(aj, oracle):
    B, H, Lq, Lk, D = 1, 3, 700, 1300, 64
    x = synth.make_inputs(B, H, Lq, Lk, D, 1.0, 0.5, seed=311)
    g = U.to_gpu(x)
    for groups in (1, 2):
        o, to, lse = _run(aj, g, D ** -0.5, "jvp", groups, 0)
        U.check_all(oracle, aj, x, B, H, Lq, Lk, D, D ** -0.5, np.arange(B * H * Lq), o, to, lse)


@pytest.mark.parametrize("groups,pair", [(2, 1), (1, 2), (2, 2)])
def test_many_short_items_back_to_back(aj, groups, pair):
    """Persistent CTAs (and CTA pairs) walking dozens of short work items each, several launches queued without a
    host synchronisation: every launch must complete (no bounded wait may expire) and reproduce the first result."""
    B, H, Lq, Lk, D = 1, 8, 128 * 148 + 300, 448, 128
    x = synth.make_inputs(B, H, Lq, Lk, D, 1.0, 0.5, seed=320)
    g = U.to_gpu(x)
    assert aj.attn_jvp_set_tuning(GROUPS, groups) == 0 and aj.attn_jvp_set_tuning(PAIR, pair) == 0
    try:
        first = aj.attention_jvp(g["q"], g["k"], g["v"], g["tq"], g["tk"], g["tv"])
        outs = [aj.attention_jvp(g["q"], g["k"], g["v"], g["tq"], g["tk"], g["tv"]) for _ in range(12)]
        torch.cuda.synchronize()
        st = aj.attn_jvp_device_status()
        assert st == 0, (aj.attn_jvp_strerror(st), aj.attn_jvp.attn_jvp_debug_timeout_info())
        for o, to, lse in outs:
            assert torch.equal(o, first[0]) and torch.equal(to, first[1]) and torch.equal(lse, first[2])
    finally:
        aj.attn_jvp_set_tuning(GROUPS, 0)
        aj.attn_jvp_set_tuning(PAIR, 0)


def test_unknown_knobs_are_refused(aj):
    assert aj.attn_jvp_set_tuning(99, 1) != 0 and aj.attn_jvp_set_tuning(GROUPS, 3) != 0 and aj.attn_jvp_set_tuning(PAIR, -1) != 0
