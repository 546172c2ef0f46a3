"""Ulysses context parallelism around the attention-JVP kernel (Sec. 3.2, "CP").

Outside attention every rank of a context-parallel group holds a slice of the sequence, [B][L/P][H][D].
Attention needs whole sequences, so around it the tensors are exchanged all-to-all: every rank gives away its
sequence slice of all heads and receives the whole sequence of its own H/P heads, [B][L][H/P][D].  In JVP mode
the tangents travel the same way as the primals (tQ, tK, tV in; tO out), which is all the paper changes about
the scheme.  The exchange lands in this GPU's own memory; the kernel then runs unchanged on H/P heads, and its
outputs are exchanged back.  The C library stays free of collectives: the exchange is
``torch.distributed.all_to_all_single`` (NCCL over NVLink on GPUs).

Layout of the exchange (P ranks, rank r, Ls = L/P, Hp = H/P):

    seq_to_heads   [B][Ls][H][D]  --view-->  [B][Ls][P][Hp][D]  --send block p to rank p-->
                   received block s = rank s's slice of my heads  -->  [B][P*Ls][Hp][D], sequence in rank order
    heads_to_seq   the inverse; for the per-row statistics (LSE, mu) the same with [B][Hp][L] <-> [B][H][Ls].
"""
from __future__ import annotations

from typing import Optional

import torch
import torch.distributed as dist

from . import attn_jvp as _binding


def _group_size(group) -> int:
    return dist.get_world_size(group) if dist.is_initialized() else 1


def check_divisible(H: int, P: int) -> None:
    if P < 1 or H % P != 0:
        raise ValueError(f"the number of heads ({H}) must be a multiple of the context-parallel size ({P})")


def seq_to_heads(x: torch.Tensor, group=None) -> torch.Tensor:
    """[B][Ls][H][D] on every rank (sequence slices in rank order) -> [B][P*Ls][H/P][D] (this rank's heads)."""
    P = _group_size(group)
    B, Ls, H, D = x.shape
    check_divisible(H, P)
    if P == 1:
        return x
    Hp = H // P
    send = x.view(B, Ls, P, Hp, D).permute(2, 0, 1, 3, 4).contiguous()       # [P][B][Ls][Hp][D], block p -> rank p
    recv = torch.empty_like(send)
    dist.all_to_all_single(recv, send, group=group)                           # block s <- rank s
    return recv.permute(1, 0, 2, 3, 4).reshape(B, P * Ls, Hp, D)              # a view when B == 1


def heads_to_seq(x: torch.Tensor, group=None) -> torch.Tensor:
    """[B][P*Ls][H/P][D] (this rank's heads, whole sequence) -> [B][Ls][H][D] (this rank's sequence slice)."""
    P = _group_size(group)
    if P == 1:
        return x
    B, L, Hp, D = x.shape
    if L % P != 0:
        raise ValueError(f"the sequence length ({L}) must be a multiple of the context-parallel size ({P})")
    Ls = L // P
    send = x.view(B, P, Ls, Hp, D).permute(1, 0, 2, 3, 4).contiguous()        # [P][B][Ls][Hp][D], block s -> rank s
    recv = torch.empty_like(send)
    dist.all_to_all_single(recv, send, group=group)                           # block p <- rank p: head group p
    return recv.permute(1, 2, 0, 3, 4).reshape(B, Ls, P * Hp, D)


def stats_heads_to_seq(x: torch.Tensor, group=None) -> torch.Tensor:
    """Per-row statistics [B][H/P][P*Ls] (this rank's heads) -> [B][H][Ls] (this rank's sequence slice)."""
    P = _group_size(group)
    if P == 1:
        return x
    B, Hp, L = x.shape
    Ls = L // P
    send = x.view(B, Hp, P, Ls).permute(2, 0, 1, 3).contiguous()              # [P][B][Hp][Ls]
    recv = torch.empty_like(send)
    dist.all_to_all_single(recv, send, group=group)
    return recv.permute(1, 0, 2, 3).reshape(B, P * Hp, Ls)


def local_heads(x: torch.Tensor, group=None) -> torch.Tensor:
    """This rank's head group of a tensor that every rank holds in full, [B][L][H][D] -> [B][L][H/P][D]
    (the context of cross-attention is replicated, so nothing is exchanged for it)."""
    P = _group_size(group)
    H = x.shape[2]
    check_divisible(H, P)
    if P == 1:
        return x
    r = dist.get_rank(group)
    Hp = H // P
    return x[:, :, r * Hp:(r + 1) * Hp, :].contiguous()


class UlyssesAttentionJVP(torch.nn.Module):
    """The attention core under Ulysses context parallelism, forward or JVP mode.

    ``forward(q, k, v, tq=None, tk=None, tv=None)`` takes this rank's sequence slices [B][L/P][H][D]
    (bf16 CUDA tensors) and returns (O, tO, LSE) for the same slice: O, tO [B][L/P][H][D], LSE [B][H][L/P].
    ``tq is None`` runs the plain forward (tO is None).  ``kv_replicated=True``: k, v (and no tangents) are the
    full context [B][Lk][H][D] held by every rank (cross-attention); they are not exchanged and the
    tangent-free kernel path is used.  ``return_mu`` adds mu = rowsum(P . tS) [B][H][L/P] as a fourth result.
    """

    def __init__(self, group=None, scale: Optional[float] = None):
        super().__init__()
        self.group = group
        self.scale = scale

    def forward(self, q, k, v, tq=None, tk=None, tv=None, kv_replicated: bool = False, return_mu: bool = False):
        P = _group_size(self.group)
        check_divisible(q.shape[2], P)
        fwd_only = tq is None
        if kv_replicated and (tk is not None or tv is not None):
            raise ValueError("a replicated context is constant: it has no tangents")
        if (tk is None) != (tv is None):
            raise ValueError("tk and tv must both be given or both be None")
        g = self.group
        qh = seq_to_heads(q, g)
        tqh = None if fwd_only else seq_to_heads(tq, g)
        if kv_replicated:
            kh, vh, tkh, tvh = local_heads(k, g), local_heads(v, g), None, None
        else:
            kh, vh = seq_to_heads(k, g), seq_to_heads(v, g)
            tkh = None if (fwd_only or tk is None) else seq_to_heads(tk, g)
            tvh = None if (fwd_only or tv is None) else seq_to_heads(tv, g)
        res = _binding.attention_jvp(qh, kh, vh, tqh, tkh, tvh, scale=self.scale, fwd_only=fwd_only,
                                     return_mu=return_mu)
        o = heads_to_seq(res[0], g)
        to = None if fwd_only else heads_to_seq(res[1], g)
        lse = stats_heads_to_seq(res[2], g)
        if return_mu:
            return o, to, lse, stats_heads_to_seq(res[3], g)
        return o, to, lse
