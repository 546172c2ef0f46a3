"""Split-KV entry point and the mu side output vs the fp64 oracle (through the C ABI)."""
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


def _run(aj, g, scale, **kw):
    res = aj.attention_jvp(g["q"], g["k"], g["v"], g["tq"], g["tk"], g["tv"], scale=scale, **kw)
    torch.cuda.synchronize()
    st = aj.attn_jvp_device_status()
    assert st == 0, aj.attn_jvp_strerror(st)
    return res


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("kv_free", [False, True])
def test_mu_side_output(aj, oracle, D, kv_free):
    B, H, Lq, Lk = 1, 3, 200, 333
    x = synth.make_inputs(B, H, Lq, Lk, D, 1.0, 0.5, seed=60, kv_tangent_free=kv_free)
    o, to, lse, mu = _run(aj, U.to_gpu(x), D ** -0.5, return_mu=True)
    rows = np.arange(B * H * Lq)
    U.check_all(oracle, aj, x, B, H, Lq, Lk, D, D ** -0.5, rows, o, to, lse)
    _, _, _, rMU = U.oracle_rows(oracle, x, B, H, Lq, Lk, D, D ** -0.5, rows)
    gMU = mu.cpu().reshape(-1).double().numpy()
    # mu is an fp32 sum of bf16-operand products: same error model as LSE, scaled by |tS| ~ O(1)
    assert np.abs(gMU - rMU).max() <= 2e-3 * (1 + np.abs(rMU).max())


@pytest.mark.parametrize("shape", [(1, 2, 130, 1000, 128), (2, 2, 70, 513, 64), (1, 1, 128, 64 * 7, 128)])
@pytest.mark.parametrize("splits", [2, 3, 16])
@pytest.mark.parametrize("mode", ["jvp", "kv_free", "fwd"])
def test_splitkv_matches_oracle_and_single_pass(aj, oracle, shape, splits, mode):
    B, H, Lq, Lk, D = shape
    x = synth.make_inputs(B, H, Lq, Lk, D, 1.0, 0.5, seed=61, kv_tangent_free=(mode != "jvp"))
    g = U.to_gpu(x)
    scale = D ** -0.5
    o, to, lse, mu = _run(aj, g, scale, fwd_only=(mode == "fwd"), return_mu=True, splits=splits)
    rows = np.arange(B * H * Lq)
    U.check_all(oracle, aj, x, B, H, Lq, Lk, D, scale, rows, o, to, lse)
    if mode != "fwd":
        _, _, _, rMU = U.oracle_rows(oracle, x, B, H, Lq, Lk, D, scale, rows)
        assert np.abs(mu.cpu().reshape(-1).double().numpy() - rMU).max() <= 2e-3 * (1 + np.abs(rMU).max())
    # against the single-pass kernel: same math up to rounding of the partials
    o1, to1, lse1 = _run(aj, g, scale, fwd_only=(mode == "fwd"))
    assert (o.float() - o1.float()).abs().max() <= 4e-3
    if mode != "fwd":
        assert (to.float() - to1.float()).abs().max() <= 8e-3
    assert (lse - lse1).abs().max() <= 1e-5


def test_splitkv_workspace_checks(aj):
    B, H, Lq, Lk, D = 1, 2, 128, 640, 128
    x = synth.make_inputs(B, H, Lq, Lk, D, seed=62)
    g = U.to_gpu(x)
    need = aj.attn_jvp_splitkv_workspace_bytes(B, H, Lq, Lk, D, 4)
    n_eff = 4  # 10 tiles -> 3 per chunk -> 4 chunks
    assert need == n_eff * (2 * B * Lq * H * D * 4 + 2 * B * H * Lq * 4)
    assert aj.attn_jvp_splitkv_workspace_bytes(B, H, Lq, Lk, D, 1) == 0
    assert aj.attn_jvp_splitkv_workspace_bytes(B, H, Lq, 64, D, 8) == 0      # one tile: nothing to split
    small = torch.empty(need - 16, dtype=torch.uint8, device="cuda")
    with pytest.raises(aj.AttnJvpError) as e:
        aj.attention_jvp(g["q"], g["k"], g["v"], g["tq"], g["tk"], g["tv"], splits=4, workspace=small)
    assert e.value.code == 12
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    o, to, lse = aj.attention_jvp(g["q"], g["k"], g["v"], g["tq"], g["tk"], g["tv"], splits=4, workspace=ws)
    o1, to1, lse1 = aj.attention_jvp(g["q"], g["k"], g["v"], g["tq"], g["tk"], g["tv"])
    torch.cuda.synchronize()
    assert (o.float() - o1.float()).abs().max() <= 4e-3 and (to.float() - to1.float()).abs().max() <= 8e-3


def test_layer_front_end_matches_direct_calls(aj):
    """The withT protocol of the layer wrapper is argument routing only."""
    B, H, Lq, Lk, D = 1, 2, 200, 300, 128
    x = synth.make_inputs(B, H, Lq, Lk, D, 1.0, 0.5, seed=63)
    g = U.to_gpu(x)
    layer = aj.AttentionCoreJVP(scale=0.1, keep_mu=True)
    o_plain = layer(g["q"], g["k"], g["v"])
    o, to = layer((g["q"], g["tq"]), (g["k"], g["tk"]), (g["v"], g["tv"]), withT=True)
    lse, mu = layer.last_lse, layer.last_mu
    oc, toc = layer((g["q"], g["tq"]), g["k"], g["v"], withT=True)          # constant context
    ro, rto, rlse, rmu = aj.attention_jvp(g["q"], g["k"], g["v"], g["tq"], g["tk"], g["tv"], scale=0.1, return_mu=True)
    rco, rcto, _ = aj.attention_jvp(g["q"], g["k"], g["v"], g["tq"], None, None, scale=0.1)
    rpo, _, _ = aj.attention_jvp(g["q"], g["k"], g["v"], None, None, None, scale=0.1, fwd_only=True)
    torch.cuda.synchronize()
    assert torch.equal(o, ro) and torch.equal(to, rto) and torch.equal(lse, rlse) and torch.equal(mu, rmu)
    assert torch.equal(o_plain, rpo) and torch.equal(oc, rco) and torch.equal(toc, rcto)
    # (the plain forward runs on its own kernel variant: equal to the JVP call's O to one bf16 ulp)
    assert (o_plain.float() - ro.float()).abs().max().item() <= 2.0 ** -7 * ro.float().abs().max().item()
    with pytest.raises(ValueError):
        layer((g["q"], g["tq"]), (g["k"], g["tk"]), g["v"], withT=True)


def test_suggested_splits_fill_one_wave_and_give_the_same_result(aj, oracle):
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    # plenty of query tiles: no split
    assert aj.attn_jvp_suggest_splits(1, 40, 32760, 32760, 128) == 1
    assert aj.attn_jvp_suggest_splits(2, 8, 2048, 4096, 128) == 1
    # few query tiles: the largest chunk count that fits one wave, at least four key tiles per chunk
    B, H, Lq, Lk, D = 1, 8, 512, 8192, 128
    items = (Lq + 127) // 128 * H * B
    want = max(1, min(sms // items, (Lk + 63) // 64 // 4))
    assert aj.attn_jvp_suggest_splits(B, H, Lq, Lk, D) == want
    assert aj.attn_jvp_suggest_splits(1, 1, 64, 1024, 64) == 4          # 16 key tiles: four per chunk
    x = synth.make_inputs(B, H, Lq, Lk, D, 1.0, 0.5, seed=77)
    g = U.to_gpu(x)
    o, to, lse = aj.attention_jvp(g["q"], g["k"], g["v"], g["tq"], g["tk"], g["tv"], splits=0)
    torch.cuda.synchronize()
    assert aj.attn_jvp_device_status() == 0
    rows = synth.sample_rows(B, H, Lq, n_random_per_head=8, seed=3)
    U.check_all(oracle, aj, x, B, H, Lq, Lk, D, D ** -0.5, rows, o, to, lse)
