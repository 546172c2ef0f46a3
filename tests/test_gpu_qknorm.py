"""RMS-norm JVP kernel vs its fp64 oracle (through the C ABI), and the chain qknorm -> attention JVP."""
import numpy as np
import pytest
import torch

from paper_2510_08431_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def aj():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2510_08431_b200 import build
    build.build_library()
    import paper_2510_08431_b200 as aj
    aj.load()
    return aj


def _check(got, ref):
    # outputs are fp32 results rounded to bf16 (8 significant bits: half an ulp is at most 2^-8 of the value,
    # 3.9e-3); inputs are exact bf16; the fp32 arithmetic in between adds ~1e-6
    got = got.float().cpu().double().numpy().reshape(ref.shape)
    assert np.isfinite(got).all()
    assert (np.abs(got - ref) <= 4.0e-3 * np.abs(ref) + 1e-5).all(), np.abs(got - ref).max()


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("rows", [1, 15, 16, 17, 33, 4097])
@pytest.mark.parametrize("with_tangent", [True, False])
def test_qknorm_matches_oracle(aj, oracle, D, rows, with_tangent):
    g = torch.Generator().manual_seed(rows + D)
    x = (torch.randn(rows, D, generator=g) * 1.5).to(torch.bfloat16)
    tx = (torch.randn(rows, D, generator=g) * 0.5).to(torch.bfloat16) if with_tangent else None
    w = torch.randn(D, generator=g).float() * 0.2 + 1.0
    y, ty = aj.qknorm_jvp(x.cuda(), None if tx is None else tx.cuda(), w.cuda(), eps=1e-6)
    torch.cuda.synchronize()
    ry, rty = oracle.rmsnorm_jvp(x.double().numpy(), None if tx is None else tx.double().numpy(), w.double().numpy(), 1e-6)
    _check(y, ry)
    if with_tangent:
        _check(ty, rty)
    else:
        assert ty is None


def test_qknorm_feeds_the_attention_kernel(aj, oracle):
    """q, k, tq, tk produced by the norm kernel go straight into the attention JVP (BLHD, bf16)."""
    B, H, L, D = 1, 2, 200, 128
    x = synth.make_inputs(B, H, L, L, D, 2.0, 1.0, seed=80)
    w = torch.ones(D, device="cuda")
    q, tq = aj.qknorm_jvp(x["q"].cuda(), x["tq"].cuda(), w)
    k, tk = aj.qknorm_jvp(x["k"].cuda(), x["tk"].cuda(), w)
    assert q.shape == (B, L, H, D) and abs(q.float().pow(2).mean().item() - 1.0) < 0.02
    o, to, lse = aj.attention_jvp(q, k, x["v"].cuda(), tq, tk, x["tv"].cuda())
    torch.cuda.synchronize()
    assert aj.attn_jvp_device_status() == 0
    y = dict(q=q.cpu(), k=k.cpu(), v=x["v"], tq=tq.cpu(), tk=tk.cpu(), tv=x["tv"])
    from tests import gpu_util as U
    U.check_all(oracle, aj, y, B, H, L, L, D, D ** -0.5, np.arange(B * H * L), o, to, lse)


def test_qknorm_rejects_bad_arguments(aj):
    x = torch.zeros(4, 96, dtype=torch.bfloat16, device="cuda")
    w = torch.ones(96, device="cuda")
    with pytest.raises(aj.AttnJvpError) as e:
        aj.qknorm_jvp(x, None, w)
    assert e.value.code == 3
    x = torch.zeros(4, 128, dtype=torch.bfloat16, device="cuda")
    assert aj.attn_jvp_qknorm_fwd(x, x, torch.ones(128, device="cuda"), x, None, 4, 128, 1e-6, None) == 1
    assert aj.attn_jvp_qknorm_fwd(x, None, torch.ones(128, device="cuda"), x, None, 4, 128, 1e-6, None) == 7
