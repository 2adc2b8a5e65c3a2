"""torch.autograd glue for the Taylor linear attention (training-time use).

`linear_attention(q, k, v)` returns based_prefill's output from the empty state and, under
autograd, routes the output gradient through based_prefill_backward (with the saved forward
output, which lets the bf16 path merge two of its passes).  Only plumbing lives here:
both directions run in the library's kernels.
"""
from __future__ import annotations

import torch

from . import binding as _b


class _LinearAttention(torch.autograd.Function):
    @staticmethod
    def forward(ctx, q, k, v, numerator_only: bool):
        q, k, v = q.contiguous(), k.contiguous(), v.contiguous()
        flags = _b.BASED_NUMERATOR_ONLY if numerator_only else 0
        out = _b.based_prefill(q, k, v, flags=flags)
        ctx.save_for_backward(q, k, v, out)
        ctx.flags = flags
        return out

    @staticmethod
    def backward(ctx, dout):
        q, k, v, out = ctx.saved_tensors
        dq, dk, dv = _b.based_prefill_backward(q, k, v, dout.contiguous().to(q.dtype), flags=ctx.flags, out=out)
        return dq, dk, dv, None


def linear_attention(q, k, v, numerator_only: bool = False):
    """Causal Taylor linear attention of q, k [B,H,L,16] and v [B,H,L,d_v] (bf16 or fp32, CUDA),
    differentiable with respect to q, k and v."""
    return _LinearAttention.apply(q, k, v, numerator_only)
