"""Ulysses exchange around the attention core with two (and four) gloo ranks on the CPU.

Checked here: the pack / exchange / unpack permutation equals a single-process reshape of the whole tensor, it
round-trips, heads that do not divide by the group size are refused, and the whole wrapper (exchange, attention
on this rank's heads, exchange back) reproduces the result computed on the whole sequence at once.  The kernel
itself needs a GPU, so for the last check the call into the CUDA library is replaced, inside the test only, by
the fp64 oracle.
"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _whole(B, L, H, D, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(B, L, H, D, generator=g, dtype=torch.float64)


def _oracle_attention(q, k, v, tq=None, tk=None, tv=None, scale=None, fwd_only=False, return_mu=False, **_):
    """Stand-in for the CUDA call with the same signature and layouts, built on the fp64 oracle (test only)."""
    from oracle import attn_jvp_oracle as orc
    B, Lq, H, D = q.shape
    o = torch.empty_like(q); to = torch.empty_like(q)
    lse = torch.empty(B, H, Lq, dtype=q.dtype); mu = torch.empty(B, H, Lq, dtype=q.dtype)
    z = lambda t, b, h: None if t is None else t[b, :, h, :].numpy()
    for b in range(B):
        for h in range(H):
            tqh = np.zeros((Lq, D)) if tq is None else z(tq, b, h)
            O, tO, L, M = orc.attn_jvp_def(z(q, b, h), z(k, b, h), z(v, b, h), tqh, z(tk, b, h), z(tv, b, h),
                                           D ** -0.5 if scale is None else scale)
            o[b, :, h, :] = torch.from_numpy(O); to[b, :, h, :] = torch.from_numpy(tO)
            lse[b, h] = torch.from_numpy(L); mu[b, h] = torch.from_numpy(M)
    res = (o, None if fwd_only else to, lse)
    return res + (mu,) if return_mu else res


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2510_08431_b200 import ulysses
    try:
        B, L, H, D = 2, 8 * world, 4 * world if world > 2 else 4, 8
        Ls, Hp = L // world, H // world
        x = _whole(B, L, H, D, 0)
        mine = x[:, rank * Ls:(rank + 1) * Ls].contiguous()
        # 1. exchange == single-process reshape: whole sequence of this rank's heads
        got = ulysses.seq_to_heads(mine)
        assert got.shape == (B, L, Hp, D)
        assert torch.equal(got, x[:, :, rank * Hp:(rank + 1) * Hp, :])
        # 2. round trip
        assert torch.equal(ulysses.heads_to_seq(got), mine)
        # 3. per-row statistics [B][Hp][L] -> [B][H][Ls]
        stat = torch.arange(B * H * L, dtype=torch.float64).view(B, H, L)
        back = ulysses.stats_heads_to_seq(stat[:, rank * Hp:(rank + 1) * Hp, :].contiguous())
        assert torch.equal(back, stat[:, :, rank * Ls:(rank + 1) * Ls])
        # 4. replicated context: a slice of the heads, no exchange
        assert torch.equal(ulysses.local_heads(x), x[:, :, rank * Hp:(rank + 1) * Hp, :])
        # 5. heads not divisible by the group size
        bad = torch.zeros(1, 4, world + 1, 8, dtype=torch.float64)
        for fn in (ulysses.seq_to_heads, ulysses.local_heads):
            try:
                fn(bad)
                raise AssertionError("indivisible head count accepted")
            except ValueError:
                pass
        # 6. the whole wrapper against the whole-sequence result (oracle in place of the CUDA call)
        ulysses._binding.attention_jvp = _oracle_attention
        full = {n: _whole(B, L, H, D, s) for s, n in enumerate(("q", "k", "v", "tq", "tk", "tv"), start=1)}
        ref = _oracle_attention(*[full[n] for n in ("q", "k", "v", "tq", "tk", "tv")], return_mu=True)
        sl = lambda t: t[:, rank * Ls:(rank + 1) * Ls].contiguous()
        layer = ulysses.UlyssesAttentionJVP()
        o, to, lse, mu = layer(*[sl(full[n]) for n in ("q", "k", "v", "tq", "tk", "tv")], return_mu=True)
        assert torch.allclose(o, sl(ref[0]), atol=1e-12) and torch.allclose(to, sl(ref[1]), atol=1e-12)
        assert torch.allclose(lse, ref[2][:, :, rank * Ls:(rank + 1) * Ls], atol=1e-12)
        assert torch.allclose(mu, ref[3][:, :, rank * Ls:(rank + 1) * Ls], atol=1e-12)
        # cross-attention: replicated constant context, tangent-free
        ctx_k, ctx_v = _whole(B, 5, H, D, 11), _whole(B, 5, H, D, 12)
        ref_c = _oracle_attention(full["q"], ctx_k, ctx_v, full["tq"])
        o, to, lse = layer(sl(full["q"]), ctx_k, ctx_v, sl(full["tq"]), kv_replicated=True)
        assert torch.allclose(o, sl(ref_c[0]), atol=1e-12) and torch.allclose(to, sl(ref_c[1]), atol=1e-12)
        # plain forward
        o, to, lse = layer(sl(full["q"]), sl(full["k"]), sl(full["v"]))
        assert to is None and torch.allclose(o, sl(ref[0]), atol=1e-12)
        out.put((rank, "ok"))
    except Exception as e:   # noqa: BLE001 -- reported to the parent, which fails the test
        out.put((rank, f"{type(e).__name__}: {e}"))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 4])
def test_exchange_and_wrapper_with_gloo_ranks(world):
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == [(r, "ok") for r in range(world)], res


def test_single_process_is_identity():
    from paper_2510_08431_b200 import ulysses
    x = _whole(1, 6, 3, 4, 0)
    assert ulysses.seq_to_heads(x) is x and ulysses.heads_to_seq(x) is x and ulysses.local_heads(x) is x
    with pytest.raises(ValueError):
        ulysses.check_divisible(40, 3)
