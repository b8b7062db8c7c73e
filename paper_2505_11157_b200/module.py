"""Multi-head spherical (neighborhood) attention as a ``torch.nn.Module`` on channels-first feature maps.

The paper's attention layer (Sec. 3.3, "spherical multi-head attention") projects a feature map to queries, keys and
values with pointwise (1x1) linear maps, splits the channels into heads, applies the attention operator and projects
the result back.  Only the attention operator is this package's subject: the four pointwise projections here are plain
``torch.nn.functional.conv2d`` calls (library GEMMs), and the operator is the channels-first entry point of the C ABI,
so no tensor is permuted in Python.
"""
from __future__ import annotations

import math

import torch

from . import sna
from .autograd import spherical_neighborhood_attention_cf


class SphericalNeighborhoodAttention(torch.nn.Module):
    """x_q [B, C_in, nlat_out, nlon_out], x_kv [B, C_in, nlat_in, nlon_in] -> [B, C_out, nlat_out, nlon_out].

    ``plan`` fixes grids and cutoff (``sna.Plan(..., global_attention=True)`` gives global spherical attention).
    ``embed_dim`` = heads * head_dim channels are used inside; head_dim must be a multiple of 4 up to 128.
    """

    def __init__(self, plan: "sna.Plan", in_channels: int, heads: int, head_dim: int, out_channels: int | None = None, bias: bool = True):
        super().__init__()
        if head_dim % 4 != 0 or not 4 <= head_dim <= 128:
            raise ValueError("head_dim must be a multiple of 4 between 4 and 128")
        self.plan, self.heads, self.head_dim = plan, heads, head_dim
        embed = heads * head_dim
        out_channels = in_channels if out_channels is None else out_channels
        make = lambda o, i: torch.nn.Parameter(torch.empty(o, i, 1, 1).uniform_(-1.0 / math.sqrt(i), 1.0 / math.sqrt(i)))
        self.wq, self.wk, self.wv, self.wo = make(embed, in_channels), make(embed, in_channels), make(embed, in_channels), make(out_channels, embed)
        self.bq = torch.nn.Parameter(torch.zeros(embed)) if bias else None
        self.bk = torch.nn.Parameter(torch.zeros(embed)) if bias else None
        self.bv = torch.nn.Parameter(torch.zeros(embed)) if bias else None
        self.bo = torch.nn.Parameter(torch.zeros(out_channels)) if bias else None

    def forward(self, x_q: torch.Tensor, x_kv: torch.Tensor | None = None) -> torch.Tensor:
        x_kv = x_q if x_kv is None else x_kv
        conv = torch.nn.functional.conv2d
        q = conv(x_q, self.wq, self.bq)          # channel h * head_dim + c is channel c of head h: the layout sna_forward_cf takes
        k = conv(x_kv, self.wk, self.bk)
        v = conv(x_kv, self.wv, self.bv)
        y = spherical_neighborhood_attention_cf(self.plan, q.float(), k.float(), v.float(), heads=self.heads)
        return conv(y.to(x_q.dtype), self.wo, self.bo)
