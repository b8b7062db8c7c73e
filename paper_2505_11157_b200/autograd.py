"""A thin ``torch.autograd.Function`` over the C-ABI calls, for dropping the operator into a PyTorch graph.

Nothing is computed here: forward calls ``sna_forward_ex`` (keeping out and lse), backward calls
``sna_backward_ex`` with a workspace tensor.  Tensors are [B, H, nlat, nlon, C] fp32 CUDA, channels last.
"""
from __future__ import annotations

import torch

from . import sna


class _SphericalNeighborhoodAttention(torch.autograd.Function):
    @staticmethod
    def forward(ctx, plan: "sna.Plan", q, k, v):
        if q.dtype != torch.float32 or k.dtype != torch.float32 or v.dtype != torch.float32:
            raise ValueError("spherical_neighborhood_attention computes in float32: cast q, k, v first "
                             "(autocast does not apply to this operator)")
        q, k, v = q.contiguous(), k.contiguous(), v.contiguous()
        out, lse = plan.forward(q, k, v, return_lse=True)
        ctx.plan = plan
        ctx.save_for_backward(q, k, v, out, lse)
        return out

    @staticmethod
    def backward(ctx, dout):
        q, k, v, out, lse = ctx.saved_tensors
        dq, dk, dv = ctx.plan.backward(q, k, v, dout.contiguous().float(), out=out, lse=lse)
        return None, dq, dk, dv


def spherical_neighborhood_attention(plan: "sna.Plan", q: torch.Tensor, k: torch.Tensor, v: torch.Tensor) -> torch.Tensor:
    """out = NAttn_{S^2}[q, k, v] on the grids and cutoff of ``plan`` (differentiable in q, k, v)."""
    return _SphericalNeighborhoodAttention.apply(plan, q, k, v)


class _SphericalNeighborhoodAttentionCF(torch.autograd.Function):
    @staticmethod
    def forward(ctx, plan: "sna.Plan", heads: int, q, k, v):
        if q.dtype != torch.float32 or k.dtype != torch.float32 or v.dtype != torch.float32:
            raise ValueError("spherical_neighborhood_attention_cf computes in float32: cast q, k, v first")
        out, state = plan.forward_cf(q.contiguous(), k.contiguous(), v.contiguous(), heads)
        ctx.plan, ctx.heads, ctx.state = plan, heads, state
        return out

    @staticmethod
    def backward(ctx, dout):
        dq, dk, dv = ctx.plan.backward_cf(dout.contiguous().float(), ctx.state, ctx.heads)
        return None, None, dq, dk, dv


def spherical_neighborhood_attention_cf(plan: "sna.Plan", q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, heads: int = 1) -> torch.Tensor:
    """The same operator on channels-first tensors [B, heads*C, nlat, nlon], as a 2D convolutional network carries
    them; the layout change runs on the GPU inside the call (differentiable in q, k, v)."""
    return _SphericalNeighborhoodAttentionCF.apply(plan, heads, q, k, v)
