"""``torch.autograd`` entry point of the MALA attention path (marshalling only: Algorithm 1 in the forward, Algorithm 2
in the backward, both in the library's kernels; the saved tensors are q, k, v, o and the log-normalizer, nothing else).

Note that, as the paper states in Section 2.2, the backward is Algorithm 2 on the LSE-derived support, not the exact
derivative of the forward's output; at tau = 0 it is the exact FullAttn gradient.
"""
from __future__ import annotations

import math
from typing import Optional

import torch

from . import mala


class _MalaAttention(torch.autograd.Function):
    @staticmethod
    def forward(ctx, q, k, v, tau: float, scale: float, causal: bool):
        o, lse, _ = mala.fwd(q, k, v, scale, tau, causal=causal)
        ctx.save_for_backward(q, k, v, o, lse)
        ctx.tau, ctx.scale, ctx.causal = tau, scale, causal
        return o

    @staticmethod
    def backward(ctx, do):
        q, k, v, o, lse = ctx.saved_tensors
        if do.stride(-1) != 1:
            do = do.contiguous()
        dq, dk, dv, _ = mala.bwd(q, k, v, o, do, lse, ctx.scale, ctx.tau, causal=ctx.causal)
        return dq, dk, dv, None, None, None


def mala_attention(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, tau: float, scale: Optional[float] = None,
                   causal: bool = True) -> torch.Tensor:
    """MALA attention of bf16 q [B,N,Hq,d] against k, v [B,N,Hkv,d] on a B200 (tau = 0: FullAttn), differentiable
    with respect to q, k and v.  ``scale`` defaults to 1 / sqrt(d)."""
    if scale is None:
        scale = 1.0 / math.sqrt(q.shape[-1])
    return _MalaAttention.apply(q, k, v, float(tau), float(scale), bool(causal))
