"""Layer-level front end: an attention core that runs either as a plain forward or in JVP mode.

The paper restructures every network layer so that one call can carry primals alone or (primal, tangent)
pairs, selected by a ``withT`` keyword (Appendix C.2, "Network Restructuring"); all layers use PyTorch's
forward-mode operator for the JVP branch except the attention core, which calls the fused kernel
(Appendix C.1).  This module is that attention core for [B][L][H][D] bf16 tensors.  It holds no
parameters and does no arithmetic itself: both branches are calls into the CUDA library.
"""
from __future__ import annotations

from typing import Optional, Tuple, Union

import torch

from . import attn_jvp as _binding

TensorWithT = Tuple[torch.Tensor, torch.Tensor]   # (primal, tangent)


class AttentionCoreJVP(torch.nn.Module):
    """softmax(s q k^T) v with an optional tangent channel.

    ``forward(q, k, v)`` returns O.  ``forward(q, k, v, withT=True)`` takes q as a (primal, tangent) pair and
    k, v either as pairs (self-attention: their tangents matter) or as plain tensors (cross-attention on a
    context that does not depend on the differentiated input, so tK = tV = 0), and returns (O, tO).
    The log-sum-exp of the last call is kept in ``self.last_lse`` (and mu, the tangent of the LSE, in
    ``self.last_mu`` when ``keep_mu`` is set).
    """

    def __init__(self, scale: Optional[float] = None, keep_mu: bool = False):
        super().__init__()
        self.scale = scale
        self.keep_mu = keep_mu
        self.last_lse = None
        self.last_mu = None

    def forward(self, q, k, v, withT: bool = False):
        if withT:
            return self._forward_jvp(q, k, v)
        return self._forward(q, k, v)

    def _forward(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor) -> torch.Tensor:
        o, _, lse = _binding.attention_jvp(q, k, v, scale=self.scale, fwd_only=True)
        self.last_lse, self.last_mu = lse, None
        return o

    def _forward_jvp(self, q: TensorWithT, k: Union[TensorWithT, torch.Tensor],
                     v: Union[TensorWithT, torch.Tensor]) -> TensorWithT:
        qp, qt = q
        k_pair, v_pair = isinstance(k, (tuple, list)), isinstance(v, (tuple, list))
        if k_pair != v_pair:
            raise ValueError("k and v must both carry tangents (self-attention) or both be constant (context)")
        if k_pair:
            (kp, kt), (vp, vt) = k, v
        else:
            kp, kt, vp, vt = k, None, v, None
        res = _binding.attention_jvp(qp, kp, vp, qt.detach(), None if kt is None else kt.detach(),
                                     None if vt is None else vt.detach(), scale=self.scale,
                                     return_mu=self.keep_mu)
        self.last_lse = res[2]
        self.last_mu = res[3] if self.keep_mu else None
        return res[0], res[1]
