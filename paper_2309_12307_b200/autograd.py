"""torch.autograd front end of S2-Attn (Algorithm 1 of the LongLoRA paper).

`s2_attn(q, k, v, G)` behaves like a differentiable function of q [B,N,H,d] and k, v [B,N,Hkv,d]
(bf16, CUDA, contiguous): the forward runs `s2a_fwd_ex`, the backward `s2a_bwd_ex`.  Everything is
computed by the CUDA library; torch only records the graph and owns the tensors.
"""
from __future__ import annotations

import torch

from . import binding


class _S2Attn(torch.autograd.Function):
    @staticmethod
    def forward(ctx, q, k, v, G, opts, fast_backward):
        q, k, v = q.contiguous(), k.contiguous(), v.contiguous()
        o, lse = binding.s2a_fwd_ex(q, k, v, G, **opts)
        ctx.save_for_backward(q, k, v, o, lse)
        ctx.G, ctx.opts, ctx.fast_backward = G, opts, fast_backward
        return o

    @staticmethod
    def backward(ctx, dO):
        q, k, v, o, lse = ctx.saved_tensors
        dq, dk, dv = binding.s2a_bwd_ex(q, k, v, o, lse, dO.contiguous(), ctx.G, fast=ctx.fast_backward, **ctx.opts)
        return dq, dk, dv, None, None, None


def s2_attn(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, G: int, *, scale: float | None = None,
            n_unshifted: int | None = None, shift: int | None = None, leak_free: bool = False,
            swap_wrapped: bool = False, fast_backward: bool = True) -> torch.Tensor:
    """Shifted sparse attention: groups of G tokens, second half of the heads shifted by G/2.

    Keyword options as in `s2a_fwd_ex`: softmax scale (default 1/sqrt(d)), number of unshifted heads
    (default H/2), shift in tokens (default G/2), and variants 2 (`leak_free`) and 3 (`swap_wrapped`)
    of the paper's Appendix B.  With n_unshifted = H, shift = 0 and G = N it is ordinary causal attention.
    `fast_backward` chooses the backward's scratch: True allocates room for the spilled dS (2 bytes per
    attended pair of a tile, within half of the free device memory) so that dq is a plain product, False
    the minimum (4 bytes per query row; dq then recomputes the scores).
    """
    opts = dict(scale=scale, n_unshifted=n_unshifted, shift=shift, leak_free=leak_free, swap_wrapped=swap_wrapped)
    return _S2Attn.apply(q, k, v, G, opts, fast_backward)
