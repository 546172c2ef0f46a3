"""Persistent CTAs: several work items per CTA with very few key tiles each.

With one to nine 64-key tiles per item the hand-over between items (shared-memory ring running on across items,
staging slots for the output tiles interleaved with the next item's loads, reuse of the accumulators) makes up
most of what a CTA does, and every ring position is reused after a different predecessor than in long items.
Every item is checked against the fp64 oracle on a few of its rows.
"""
import numpy as np
import pytest
import torch

from paper_2510_08431_b200 import synth
from tests import gpu_util as U

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def aj():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2510_08431_b200 import build
    build.build_library()
    import paper_2510_08431_b200 as aj
    aj.load()
    return aj


def _rows_touching_every_item(B, H, Lq, stride=37):
    rows = set(range(0, B * H * Lq, stride))
    for bh in range(B * H):                      # first and last (partial) query tile of every head in full
        rows.update(range(bh * Lq, bh * Lq + min(128, Lq)))
        rows.update(range(bh * Lq + (Lq - 1) // 128 * 128, (bh + 1) * Lq))
    return np.array(sorted(rows))


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("mode", ["jvp", "kv_free", "fwd"])
@pytest.mark.parametrize("n_tiles", [1, 2, 3, 4, 6, 8, 9])
def test_many_short_items_per_cta(aj, oracle, D, mode, n_tiles):
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    B, H = 1, 3
    q_tiles = sms + 3                      # items = 3 * (sms + 3): three to four items per CTA
    Lq = 128 * (q_tiles - 1) + 17          # last query tile partial
    Lk = 64 * n_tiles - 7                  # last key tile partial
    x = synth.make_inputs(B, H, Lq, Lk, D, 1.0, 0.5, seed=700 + n_tiles, kv_tangent_free=(mode != "jvp"))
    g = U.to_gpu(x)
    scale = D ** -0.5
    # run twice into poisoned outputs: the second launch must not depend on what the first left behind
    for _ in range(2):
        o = torch.full((B, Lq, H, D), float("nan"), dtype=torch.bfloat16, device="cuda")
        to = torch.full_like(o, float("nan"))
        lse = torch.full((B, H, Lq), float("nan"), dtype=torch.float32, device="cuda")
        o, to_out, lse = U.run(aj, g, scale, fwd_only=(mode == "fwd"), out=(o, None if mode == "fwd" else to, lse))
    assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all()
    if mode != "fwd":
        assert torch.isfinite(to_out.float()).all()
    rows = _rows_touching_every_item(B, H, Lq)
    U.check_all(oracle, aj, x, B, H, Lq, Lk, D, scale, rows, o, to_out, lse)


def test_fewer_items_than_sms_and_exactly_one_round(aj, oracle):
    """Grid smaller than the GPU, and a grid where every CTA gets exactly one item (no hand-over at all)."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    for B, H, q_tiles in ((1, 1, 5), (1, 2, sms // 2), (2, 1, sms // 2 + 1)):
        Lq, Lk, D = 128 * q_tiles - 3, 200, 128
        x = synth.make_inputs(B, H, Lq, Lk, D, 1.0, 0.5, seed=800 + q_tiles)
        o, to, lse = U.run(aj, U.to_gpu(x), D ** -0.5)
        U.check_all(oracle, aj, x, B, H, Lq, Lk, D, D ** -0.5, _rows_touching_every_item(B, H, Lq, 53), o, to, lse)
