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
        o, lse, _ = mala.fwd_chunk(q, k, v, scale, tau, causal=causal)
        ctx.save_for_backward(q, k, v, o, lse)
        ctx.tau, ctx.scale, ctx.causal = tau, scale, causal
        return o

    @staticmethod
    def backward(ctx, do):
        q, k, v, o, lse = ctx.saved_tensors
        if do.stride(-1) != 1:
            do = do.contiguous()
        dq, dk, dv, _ = mala.bwd_chunk(q, k, v, o, do, lse, ctx.scale, ctx.tau, causal=ctx.causal)
        return dq, dk, dv, None, None, None


class _MalaAttentionPacked(torch.autograd.Function):
    @staticmethod
    def forward(ctx, q, k, v, cu_q, cu_k, max_q: int, max_k: int, tau: float, scale: float, causal: bool):
        o, lse, _ = mala.fwd_varlen_prefix(q, k, v, cu_q, cu_k, max_q, max_k, scale, tau, causal=causal)
        ctx.save_for_backward(q, k, v, o, lse, cu_q, cu_k)
        ctx.args = (max_q, max_k, scale, tau, causal)
        return o

    @staticmethod
    def backward(ctx, do):
        q, k, v, o, lse, cu_q, cu_k = ctx.saved_tensors
        max_q, max_k, scale, tau, causal = ctx.args
        if do.stride(-1) != 1:
            do = do.contiguous()
        dq, dk, dv, _ = mala.bwd_varlen_prefix(q, k, v, o, do, lse, cu_q, cu_k, max_q, max_k, scale, tau, causal=causal)
        return dq, dk, dv, None, None, None, None, None, None, None


def mala_attention(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, tau: float, scale: Optional[float] = None,
                   causal: bool = True) -> torch.Tensor:
    """MALA attention of bf16 q [B,Nq,Hq,d] against k, v [B,Nk,Hkv,d] on a B200 (tau = 0: FullAttn), differentiable
    with respect to q, k and v.  Causal: the queries are the last Nq of the Nk positions (Nq = Nk: self attention).
    ``scale`` defaults to 1 / sqrt(d)."""
    if scale is None:
        scale = 1.0 / math.sqrt(q.shape[-1])
    return _MalaAttention.apply(q, k, v, float(tau), float(scale), bool(causal))


def mala_attention_packed(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, cu_seqlens_q: torch.Tensor,
                          cu_seqlens_k: torch.Tensor, max_seqlen_q: int, max_seqlen_k: int, tau: float,
                          scale: Optional[float] = None, causal: bool = True) -> torch.Tensor:
    """MALA attention on packed sequences: q [1,total_q,Hq,d], k, v [1,total_k,Hkv,d], sequence b in the rows
    cu_seqlens_q[b] .. cu_seqlens_q[b+1]-1 of q and cu_seqlens_k[b] .. of k, v (int32 on the device; pass the same
    tensor twice for self attention).  Differentiable with respect to q, k and v."""
    if scale is None:
        scale = 1.0 / math.sqrt(q.shape[-1])
    return _MalaAttentionPacked.apply(q, k, v, cu_seqlens_q, cu_seqlens_k, int(max_seqlen_q), int(max_seqlen_k),
                                      float(tau), float(scale), bool(causal))
