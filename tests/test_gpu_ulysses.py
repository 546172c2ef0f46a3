"""The Ulysses wrapper on one GPU: with a group of one rank nothing is exchanged and the results are the direct
call's, bit for bit (the multi-rank data flow is covered on the CPU by tests/test_ulysses_gloo.py)."""
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


def test_group_of_one_is_the_direct_call(aj):
    from paper_2510_08431_b200.ulysses import UlyssesAttentionJVP
    B, H, Lq, Lk, D = 1, 4, 300, 520, 128
    x = synth.make_inputs(B, H, Lq, Lk, D, 1.0, 0.5, seed=90)
    g = U.to_gpu(x)
    layer = UlyssesAttentionJVP(scale=D ** -0.5)
    o, to, lse, mu = layer(g["q"], g["k"], g["v"], g["tq"], g["tk"], g["tv"], return_mu=True)
    ro, rto, rlse, rmu = aj.attention_jvp(g["q"], g["k"], g["v"], g["tq"], g["tk"], g["tv"], scale=D ** -0.5,
                                          return_mu=True)
    torch.cuda.synchronize()
    assert aj.attn_jvp_device_status() == 0
    assert torch.equal(o, ro) and torch.equal(to, rto) and torch.equal(lse, rlse) and torch.equal(mu, rmu)
    # cross-attention on a replicated context, and the plain forward
    o2, to2, _ = layer(g["q"], g["k"], g["v"], g["tq"], kv_replicated=True)
    r2 = aj.attention_jvp(g["q"], g["k"], g["v"], g["tq"], None, None, scale=D ** -0.5)
    o3, to3, _ = layer(g["q"], g["k"], g["v"])
    r3 = aj.attention_jvp(g["q"], g["k"], g["v"], None, None, None, scale=D ** -0.5, fwd_only=True)
    torch.cuda.synchronize()
    assert torch.equal(o2, r2[0]) and torch.equal(to2, r2[1])
    assert to3 is None and torch.equal(o3, r3[0])
