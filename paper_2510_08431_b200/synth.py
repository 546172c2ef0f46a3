"""Seeded synthetic workloads (inputs only -- none of the method's arithmetic).

The shapes stand in for the attention calls of the image / video diffusion
transformers the paper distils (Sec. 5: 832x480x81 video => 21 latent frames
x 30 x 52 patches = 32760 tokens; ~4k tokens for 1024px image latents).
Unit-variance q,k with scale 1/sqrt(D) stand for QK-normalised projections
(Sec. 3.1); tangents of standard deviation 0.5 reflect the cos(t)sin(t) <= 1/2
pre-scaling of the tangent inputs (Algorithm 1, line 4).

Both the CPU oracle and the CUDA path are fed from here, so that they see the
same bits: tensors are drawn in fp32 on the CPU generator in the fixed order
Q, K, V, tQ, tK, tV, scaled, and rounded to bf16 (round-to-nearest-even).
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    Lq: int
    Lk: int
    D: int
    sigma_primal: float
    sigma_tangent: float
    seed: int
    kv_tangent_free: bool = False

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.D)

    @property
    def flops(self) -> int:
        """The metric's flop count: 12*B*H*Lq*Lk*D (six 2*D-flop contractions per score)."""
        return 12 * self.B * self.H * self.Lq * self.Lk * self.D

    @property
    def executed_flops(self) -> int:
        """Flops actually executed: 8*... when tK = tV = 0 drops two contractions."""
        per = 8 if self.kv_tangent_free else 12
        return per * self.B * self.H * self.Lq * self.Lk * self.D


WORKLOADS = {
    "tiny": Workload("tiny", 1, 2, 256, 256, 64, 1.0, 1.0, 0),
    "image_dit_2b": Workload("image_dit_2b", 2, 16, 4096, 4096, 128, 1.0, 0.5, 1),
    "video_dit_1p3b": Workload("video_dit_1p3b", 1, 12, 32760, 32760, 128, 1.0, 1.0, 2),
    "video_dit_14b": Workload("video_dit_14b", 1, 40, 32760, 32760, 128, 1.0, 0.5, 3),
    "cross_attn_14b": Workload("cross_attn_14b", 1, 40, 32760, 512, 128, 1.0, 1.0, 4,
                               kv_tangent_free=True),
    # not one of the five benchmark configs: few queries against a long key sequence, the case the
    # split-KV entry point exists for (32 query tiles x heads CTAs would fill a fifth of the GPU)
    "few_q_long_k": Workload("few_q_long_k", 1, 8, 512, 32760, 128, 1.0, 0.5, 5),
    # head dimension 64 (the library's other supported D) at the image and the video sequence lengths
    "image_dit_d64": Workload("image_dit_d64", 2, 24, 4096, 4096, 64, 1.0, 0.5, 6),
    "video_dit_d64": Workload("video_dit_d64", 1, 24, 32760, 32760, 64, 1.0, 0.5, 7),
}


def make_inputs(B, H, Lq, Lk, D, sigma_primal=1.0, sigma_tangent=1.0, seed=0,
                kv_tangent_free=False, pin_memory=False):
    """Returns dict q,k,v,tq,tk,tv of bf16 CPU tensors in [B][L][H][D] layout.

    With ``kv_tangent_free`` the tK / tV entries are None (and no random numbers
    are drawn for them).
    """
    g = torch.Generator(device="cpu").manual_seed(int(seed))

    def draw(L, sigma):
        x = torch.randn((B, L, H, D), generator=g, dtype=torch.float32)
        if sigma != 1.0:
            x.mul_(sigma)
        x = x.to(torch.bfloat16)
        return x.pin_memory() if pin_memory else x

    out = {}
    out["q"] = draw(Lq, sigma_primal)
    out["k"] = draw(Lk, sigma_primal)
    out["v"] = draw(Lk, sigma_primal)
    out["tq"] = draw(Lq, sigma_tangent)
    out["tk"] = None if kv_tangent_free else draw(Lk, sigma_tangent)
    out["tv"] = None if kv_tangent_free else draw(Lk, sigma_tangent)
    return out


def make_workload(w: Workload, pin_memory=False):
    return make_inputs(w.B, w.H, w.Lq, w.Lk, w.D, w.sigma_primal, w.sigma_tangent, w.seed,
                       w.kv_tangent_free, pin_memory=pin_memory)


def bf16_bits(t: torch.Tensor):
    """bf16 tensor -> numpy uint16 array of its bit patterns (same shape)."""
    return t.contiguous().view(torch.uint16).numpy()


def sample_rows(B, H, Lq, n_random_per_head=4, tile=128, full_tiles=(0,), heads_full=(0,), seed=0):
    """Deterministic sample of flat query-row indices (b*H + h)*Lq + i.

    Always contains the whole last (possibly partial) ``tile``-row tile and the
    listed full tiles of the heads in ``heads_full``, plus a few seeded random
    rows of every head.
    """
    g = torch.Generator(device="cpu").manual_seed(1000 + int(seed))
    rows = set()
    n_tiles = (Lq + tile - 1) // tile
    for bh in heads_full:
        if bh >= B * H:
            continue
        for t in set(list(full_tiles) + [n_tiles - 1]):
            if 0 <= t < n_tiles:
                for i in range(t * tile, min(Lq, (t + 1) * tile)):
                    rows.add(bh * Lq + i)
    for bh in range(B * H):
        idx = torch.randint(0, Lq, (n_random_per_head,), generator=g).tolist()
        for i in idx:
            rows.add(bh * Lq + i)
    return sorted(rows)
