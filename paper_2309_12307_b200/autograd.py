"""torch.autograd front end of S2-Attn (Algorithm 1 of the LongLoRA paper).

`s2_attn(q, k, v, G)` behaves like a differentiable function of q [B,N,H,d] and k, v [B,N,Hkv,d]
(bf16, CUDA, contiguous): the forward runs `s2a_fwd`, the backward `s2a_bwd`.  Everything is
computed by the CUDA library; torch only records the graph and owns the tensors.
"""
from __future__ import annotations

import torch

from . import binding


class _S2Attn(torch.autograd.Function):
    @staticmethod
    def forward(ctx, q, k, v, G):
        q, k, v = q.contiguous(), k.contiguous(), v.contiguous()
        o, lse = binding.s2a_fwd(q, k, v, G)
        ctx.save_for_backward(q, k, v, o, lse)
        ctx.G = G
        return o

    @staticmethod
    def backward(ctx, dO):
        q, k, v, o, lse = ctx.saved_tensors
        dq, dk, dv = binding.s2a_bwd(q, k, v, o, lse, dO.contiguous(), ctx.G)
        return dq, dk, dv, None


def s2_attn(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, G: int) -> torch.Tensor:
    """Shifted sparse attention: groups of G tokens, second half of the heads shifted by G/2."""
    return _S2Attn.apply(q, k, v, G)
