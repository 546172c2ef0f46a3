"""The allocation-free split-KV entry point (attn_jvp_fwd_splitkv_static) against the workspace-taking one.

Some callers may not allocate GPU memory at all: serving loops whose memory was fixed at start-up and which
cannot take the device-wide synchronisation of an allocation, processes where a framework allocator owns every
byte.  For them the
library carries a 32 MiB scratch buffer of its own.  This file is collected last on purpose, so that a run that
stops at the first failure has already been through every other test; it also passes when run alone in a fresh
process (then its first call is the very first use of the library on the device).
"""
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


def _buffers(B, H, Lq, D, fill):
    o = torch.full((B, Lq, H, D), fill, dtype=torch.bfloat16, device="cuda")
    to = torch.full((B, Lq, H, D), fill, dtype=torch.bfloat16, device="cuda")
    lse = torch.full((B, H, Lq), fill, dtype=torch.float32, device="cuda")
    mu = torch.full((B, H, Lq), fill, dtype=torch.float32, device="cuda")
    return o, to, lse, mu


def _both_ways(aj, shape, splits, seed, flags=0):
    B, H, Lq, Lk, D = shape
    x = synth.make_inputs(B, H, Lq, Lk, D, 1.0, 0.5, seed=seed, kv_tangent_free=bool(flags & aj.KV_TANGENT_FREE))
    g = {k: (None if t is None else t.cuda()) for k, t in x.items()}
    scale = D ** -0.5
    stream = torch.cuda.current_stream().cuda_stream
    # the new entry point: all device memory it touches besides inputs and outputs is the library's own buffer
    so, sto, slse, smu = _buffers(B, H, Lq, D, 3.0)
    rc = aj.attn_jvp_fwd_splitkv_static(g["q"], g["k"], g["v"], g["tq"], g["tk"], g["tv"], so, sto, slse, smu,
                                        B, H, Lq, Lk, D, scale, flags, splits, stream)
    assert rc == 0, aj.attn_jvp_strerror(rc)
    # the existing entry point with a caller-allocated workspace
    need = aj.attn_jvp_splitkv_workspace_bytes(B, H, Lq, Lk, D, splits)
    ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda")
    wo, wto, wlse, wmu = _buffers(B, H, Lq, D, 5.0)
    rc = aj.attn_jvp_fwd_splitkv(g["q"], g["k"], g["v"], g["tq"], g["tk"], g["tv"], wo, wto, wlse, wmu,
                                 B, H, Lq, Lk, D, scale, flags, splits, ws, ws.numel(), stream)
    assert rc == 0, aj.attn_jvp_strerror(rc)
    torch.cuda.synchronize()
    assert aj.attn_jvp_device_status() == 0
    # same kernels, same order of operations: the two must agree to the bit, which is well inside the
    # tolerance the parity tests use (2e-2 * (1 + |ref|))
    tol = 2e-2
    for name, a, b in (("O", so, wo), ("tO", sto, wto), ("LSE", slse, wlse), ("mu", smu, wmu)):
        a, b = a.float(), b.float()
        assert torch.isfinite(a).all(), name
        assert ((a - b).abs() <= tol * (1 + b.abs())).all(), name
        assert torch.equal(a, b), name


def test_static_scratch_matches_workspace_version_twice_in_a_row(aj):
    # two calls in a row with different shapes and chunk counts: the second one finds the first one's
    # leftovers in the shared buffer and must not be affected by them
    _both_ways(aj, (1, 4, 300, 2000, 128), splits=4, seed=70)
    _both_ways(aj, (2, 2, 130, 700, 64), splits=3, seed=71, flags=aj.KV_TANGENT_FREE)
    _both_ways(aj, (1, 4, 300, 2000, 128), splits=4, seed=72)


def test_static_call_leaves_device_memory_in_use_unchanged(aj):
    """What the entry point is for, observed rather than read from its source: after one warm-up call (module
    loading and the address look-up happen there) the free device memory reported by the driver is the same
    before and after a call."""
    B, H, Lq, Lk, D, splits = 1, 4, 300, 2000, 128, 4
    x = synth.make_inputs(B, H, Lq, Lk, D, 1.0, 0.5, seed=73)
    g = {k: t.cuda() for k, t in x.items()}
    o, to, lse, mu = _buffers(B, H, Lq, D, 0.0)
    stream = torch.cuda.current_stream().cuda_stream

    def call():
        rc = aj.attn_jvp_fwd_splitkv_static(g["q"], g["k"], g["v"], g["tq"], g["tk"], g["tv"], o, to, lse, mu,
                                            B, H, Lq, Lk, D, D ** -0.5, 0, splits, stream)
        assert rc == 0, aj.attn_jvp_strerror(rc)
        torch.cuda.synchronize()

    call()
    free_before, _ = torch.cuda.mem_get_info()
    call()
    call()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, (free_before, free_after)
    assert aj.attn_jvp_device_status() == 0


def test_static_scratch_refuses_oversized_calls(aj):
    B, H, Lq, Lk, D, splits = 1, 8, 4096, 8192, 128, 8
    assert aj.attn_jvp_splitkv_workspace_bytes(B, H, Lq, Lk, D, splits) > aj.attn_jvp.STATIC_SCRATCH_BYTES
    q = torch.zeros(16, dtype=torch.bfloat16, device="cuda")   # never touched: the call is refused up front
    rc = aj.attn_jvp_fwd_splitkv_static(q, q, q, q, q, q, q, q, q, q, B, H, Lq, Lk, D, 0.1, 0, splits, None)
    assert rc == aj.attn_jvp.ERR_STATIC_SCRATCH
    assert "built-in" in aj.attn_jvp_strerror(rc)
