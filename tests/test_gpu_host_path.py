"""attn_jvp_fwd_host: host tensors in, host tensors out, heads pipelined in groups through a device workspace.

A head's result does not depend on the other heads, so the host path must reproduce the device-resident call
bit for bit; one case is also checked against the fp64 oracle directly.
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


def _device_result(aj, x, scale, mode):
    g = U.to_gpu(x)
    o, to, lse = U.run(aj, g, scale, fwd_only=(mode == "fwd"))
    return o.cpu(), None if to is None else to.cpu(), lse.cpu()


CASES = [
    # B, H, Lq, Lk, D, mode, heads_per_stage, pinned
    (2, 5, 300, 200, 128, "jvp", 2, True),       # groups of 2, 2, 1 heads; two batches
    (1, 7, 129, 513, 64, "kv_free", 0, True),    # library default grouping
    (1, 3, 257, 130, 128, "fwd", 1, False),      # pageable host memory, one head per stage
    (2, 4, 64, 64, 64, "jvp", 4, True),          # a single stage
    (1, 6, 1000, 700, 128, "jvp", 0, True),
    (1, 9, 200, 333, 128, "kv_free", 4, True),   # 4, 4, 1
]


@pytest.mark.parametrize("B,H,Lq,Lk,D,mode,hps,pinned", CASES)
def test_host_path_equals_device_path(aj, B, H, Lq, Lk, D, mode, hps, pinned):
    x = synth.make_inputs(B, H, Lq, Lk, D, 1.0, 0.5, seed=900 + H, kv_tangent_free=(mode != "jvp"),
                          pin_memory=pinned)
    scale = D ** -0.5
    ro, rto, rl = _device_result(aj, x, scale, mode)
    tq = None if mode == "fwd" else x["tq"]
    o, to, lse = aj.attention_jvp_host(x["q"], x["k"], x["v"], tq, x["tk"], x["tv"], scale=scale,
                                       fwd_only=(mode == "fwd"), heads_per_stage=hps)
    assert torch.equal(o.view(torch.int16), ro.view(torch.int16))
    assert torch.equal(lse, rl)
    if mode == "fwd":
        assert to is None
    else:
        assert torch.equal(to.view(torch.int16), rto.view(torch.int16))


def test_host_path_against_oracle_and_reuse_of_workspace(aj, oracle):
    """Two different problems through one workspace and one set of output tensors, back to back."""
    B, H, Lq, Lk, D = 1, 5, 391, 450, 128
    scale = D ** -0.5
    need = aj.attn_jvp_host_workspace_bytes(B, H, Lq, Lk, D, 2)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    out = (torch.empty((B, Lq, H, D), dtype=torch.bfloat16, pin_memory=True),
           torch.empty((B, Lq, H, D), dtype=torch.bfloat16, pin_memory=True),
           torch.empty((B, H, Lq), dtype=torch.float32, pin_memory=True))
    for seed in (31, 32):
        x = synth.make_inputs(B, H, Lq, Lk, D, 1.0, 0.5, seed=seed, pin_memory=True)
        for t in out:
            t.fill_(float("nan"))
        o, to, lse = aj.attention_jvp_host(x["q"], x["k"], x["v"], x["tq"], x["tk"], x["tv"], scale=scale, out=out,
                                           workspace=ws, heads_per_stage=2)
        U.check_all(oracle, aj, x, B, H, Lq, Lk, D, scale, np.arange(B * H * Lq), o, to, lse)


def test_host_path_argument_errors(aj):
    B, H, Lq, Lk, D = 1, 4, 128, 128, 128
    x = synth.make_inputs(B, H, Lq, Lk, D, 1.0, 0.5, seed=5, pin_memory=True)
    o = torch.empty((B, Lq, H, D), dtype=torch.bfloat16, pin_memory=True)
    to = torch.empty_like(o).pin_memory()
    lse = torch.empty((B, H, Lq), dtype=torch.float32, pin_memory=True)
    need = aj.attn_jvp_host_workspace_bytes(B, H, Lq, Lk, D, 0)
    assert need > 0 and aj.attn_jvp_host_workspace_bytes(B, H, Lq, Lk, 96, 0) == 0
    ws = torch.empty(need + 256, dtype=torch.uint8, device="cuda")
    args = (x["q"], x["k"], x["v"], x["tq"], x["tk"], x["tv"], o, to, lse, B, H, Lq, Lk, D, D ** -0.5, 0, 0)
    assert aj.attn_jvp_fwd_host(*args, ws, need - 1, None) == 12            # workspace too small
    assert aj.attn_jvp_fwd_host(*args, ws.data_ptr() + 16, need, None) == 4  # workspace not 256-byte aligned
    assert aj.attn_jvp_fwd_host(*args, None, need, None) == 1
    bad = list(args)
    bad[0] = None
    assert aj.attn_jvp_fwd_host(*bad, ws, need, None) == 1                   # q missing
    bad = list(args)
    bad[15] = 0x8
    assert aj.attn_jvp_fwd_host(*bad, ws, need, None) == 5                   # unknown flag
    bad = list(args)
    bad[16] = -1
    assert aj.attn_jvp_fwd_host(*bad, ws, need, None) == 2                   # negative heads_per_stage
    torch.cuda.synchronize()
    assert aj.attn_jvp_fwd_host(*args, ws, need, None) == 0
    torch.cuda.synchronize()
    assert aj.attn_jvp_device_status() == 0
