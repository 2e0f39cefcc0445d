"""Second formulation of S2-Attn: Algorithm 1 of the LongLoRA paper carried out
with materialised tensors (plain PyTorch CPU ops, fp64), gradients by autograd.

TEST INFRASTRUCTURE ONLY.  It exists to pin the index-form C oracle: the two
are written differently (explicit roll / reshape / dense masked attention here,
per-row index sums there; autograd here, hand-derived gradient sums there) and
must agree to rounding.

Steps, as the paper states them (Algorithm 1, Fig. 3 caption, Section 3.2):
  1. split the heads into two halves; roll the tokens of the second half by
     -G/2 along the sequence;
  2. cut the (rolled) sequence into N/G groups of G consecutive tokens and
     treat the groups as batch entries;
  3. standard causal softmax attention inside each group (Eq. 1, with the
     usual 1/sqrt(d) scale);
  4. undo the grouping, and roll the second half of the heads back by +G/2.
Grouped-query attention (not in Algorithm 1) is expressed by repeating each KV
head H/Hkv times before step 1, which is what the head mapping means.
"""
from __future__ import annotations

import math

import torch


def _roll_second_half(x: torch.Tensor, amount: int) -> torch.Tensor:
    """x: [B, N, H, d].  Roll tokens of heads H/2.. by `amount` along N."""
    H = x.shape[2]
    first, second = x[:, :, : H // 2], x[:, :, H // 2:]
    return torch.cat([first, torch.roll(second, shifts=amount, dims=1)], dim=2)


def _group_causal_attention(q, k, v, scale, extra_mask=None):
    """q, k, v: [Bg, G, H, d] -> out [Bg, G, H, d], lse [Bg, H, G]; causal inside the group.
    extra_mask [Bg, H, G, G] (True = hidden) adds to the causal mask."""
    G = q.shape[1]
    scores = torch.einsum("bxhc,byhc->bhxy", q, k) * scale
    future = torch.ones(G, G, dtype=torch.bool).triu(1)  # y > x
    scores = scores.masked_fill(future, float("-inf"))
    if extra_mask is not None:
        scores = scores.masked_fill(extra_mask, float("-inf"))
    lse = torch.logsumexp(scores, dim=-1)
    probs = torch.softmax(scores, dim=-1)
    out = torch.einsum("bhxy,byhc->bxhc", probs, v)
    return out, lse


def _swap_halves_of_wrapped_group(x, B, n_groups, H):
    """x: [B * n_groups, G, H, ...] in rolled, grouped order.  In the last group of every sequence
    (the one that wraps) exchange the first and the second half of the tokens of heads H/2.. ;
    applying it twice restores x."""
    G = x.shape[1]
    x = x.clone()
    last = (torch.arange(B) * n_groups + (n_groups - 1)).tolist()
    for bg in last:
        blk = x[bg, :, H // 2:]
        x[bg, :, H // 2:] = torch.cat([blk[G // 2:], blk[: G // 2]], dim=0)
    return x


def s2_attn(q, k, v, G, scale=None, leak_free=False, swap_wrapped=False):
    """q [B,N,H,d], k/v [B,N,Hkv,d] (fp64) -> o [B,N,H,d], lse [B,H,N].
    leak_free: variant 2 of Appendix B (Table 8; done there by changing the attention mask): in the shifted
    heads the last group, which holds the sequence's last G/2 tokens followed by its first G/2 tokens,
    is treated as two groups, so the front tokens do not attend the tail tokens.
    swap_wrapped: variant 3 of Appendix B (Table 8; front and shifted tokens exchanged): in that same
    group the two halves change places before the attention and change back after it, so the group is
    attended in original token order (front tokens first)."""
    B, N, H, d = q.shape
    Hkv = k.shape[2]
    assert N % G == 0 and G % 2 == 0 and H % 2 == 0 and H % Hkv == 0
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    rep = H // Hkv
    k = k.repeat_interleave(rep, dim=2)
    v = v.repeat_interleave(rep, dim=2)
    # step 1
    q, k, v = (_roll_second_half(x, -(G // 2)) for x in (q, k, v))
    # step 2
    q, k, v = (x.reshape(B * (N // G), G, H, d) for x in (q, k, v))
    # step 3
    extra = None
    if leak_free:
        n_groups = N // G
        extra = torch.zeros(B * n_groups, H, G, G, dtype=torch.bool)
        last = torch.arange(B) * n_groups + (n_groups - 1)      # the wrapped group of every sequence
        # queries in the second half of that group (the front tokens) do not see its first half
        for bg in last.tolist():
            extra[bg, H // 2:, G // 2:, : G // 2] = True
    if swap_wrapped:
        assert not leak_free
        q, k, v = (_swap_halves_of_wrapped_group(x, B, N // G, H) for x in (q, k, v))
    out, lse = _group_causal_attention(q, k, v, scale, extra)
    if swap_wrapped:
        out = _swap_halves_of_wrapped_group(out, B, N // G, H)
        lse = _swap_halves_of_wrapped_group(lse.permute(0, 2, 1).unsqueeze(-1), B, N // G, H).squeeze(-1).permute(0, 2, 1)
    # step 4
    out = _roll_second_half(out.reshape(B, N, H, d), G // 2)
    lse = lse.reshape(B, N // G, H, G).permute(0, 2, 1, 3).reshape(B, H, N)  # rolled token order
    lse = _roll_second_half(lse.permute(0, 2, 1).unsqueeze(-1), G // 2).squeeze(-1).permute(0, 2, 1)
    return out, lse.contiguous()


def s2_attn_grads(q, k, v, dO, G, scale=None, leak_free=False, swap_wrapped=False):
    """Autograd gradients of sum(o * dO) w.r.t. q, k, v (all fp64)."""
    q = q.detach().clone().requires_grad_(True)
    k = k.detach().clone().requires_grad_(True)
    v = v.detach().clone().requires_grad_(True)
    o, _ = s2_attn(q, k, v, G, scale, leak_free, swap_wrapped)
    (o * dO).sum().backward()
    return q.grad, k.grad, v.grad
