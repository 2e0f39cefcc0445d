"""Seeded synthetic inputs for S2-Attn (shifted sparse attention).

This module only draws random tensors and names workload shapes.  It holds none
of the method's arithmetic, so both the CUDA path's tests and the CPU oracle's
tests may use it without sharing any computation.

The tensors stand in for post-RoPE Llama2 activations: i.i.d. N(0,1) values
drawn in fp32 and rounded to bf16 (round-to-nearest-even).  Only the shapes come
from the paper (context lengths of Tables 3-4, group size G = N/4 of Table 7,
per-device batch 1 of the experimental settings).
"""
from __future__ import annotations

from dataclasses import dataclass

import torch


@dataclass(frozen=True)
class Workload:
    """One S2-Attn problem shape.  Notation follows Algorithm 1 (B, N, G, H, D)."""

    name: str
    B: int
    N: int
    G: int
    H: int
    Hkv: int
    d: int

    @property
    def pairs(self) -> int:
        """(query, key) pairs attended: every group is causal inside itself."""
        return self.B * self.H * (self.N // self.G) * (self.G * (self.G + 1) // 2)

    @property
    def flops_fwd(self) -> int:
        return 4 * self.d * self.pairs

    @property
    def flops_bwd(self) -> int:
        return 10 * self.d * self.pairs

    @property
    def flops_fwd_bwd(self) -> int:
        return 14 * self.d * self.pairs


WORKLOADS = {
    "tiny": Workload("tiny", 1, 1024, 256, 4, 4, 64),
    "llama2_7b_8k": Workload("llama2_7b_8k", 1, 8192, 2048, 32, 32, 128),
    "llama2_7b_32k": Workload("llama2_7b_32k", 1, 32768, 8192, 32, 32, 128),
    "llama2_7b_100k": Workload("llama2_7b_100k", 1, 102400, 25600, 32, 32, 128),
    "llama2_70b_32k_gqa": Workload("llama2_70b_32k_gqa", 1, 32768, 8192, 64, 8, 128),
    # further context lengths and model sizes of Tables 3-4 (G = N/4 throughout)
    "llama2_7b_16k": Workload("llama2_7b_16k", 1, 16384, 4096, 32, 32, 128),
    "llama2_7b_64k": Workload("llama2_7b_64k", 1, 65536, 16384, 32, 32, 128),
    "llama2_13b_32k": Workload("llama2_13b_32k", 1, 32768, 8192, 40, 40, 128),
    # the literal 100,000-token context: G = 25,000 and G/2 = 12,500 are not multiples of the 128-token tile
    "llama2_7b_100000": Workload("llama2_7b_100000", 1, 100000, 25000, 32, 32, 128),
}


def make_inputs(B: int, N: int, H: int, Hkv: int, d: int, seed: int = 0):
    """Draw q, k, v, dO (in that order) from one CPU generator seeded with `seed`.

    Returns four bf16 CPU tensors: q [B,N,H,d], k [B,N,Hkv,d], v [B,N,Hkv,d],
    dO [B,N,H,d].  The same bits are meant to go to the GPU and, widened
    exactly, to the oracle.
    """
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    shapes = [(B, N, H, d), (B, N, Hkv, d), (B, N, Hkv, d), (B, N, H, d)]
    out = []
    for shp in shapes:
        x = torch.randn(shp, generator=gen, dtype=torch.float32)
        out.append(x.to(torch.bfloat16).contiguous())
    return tuple(out)


def make_inputs_periodic(B: int, N: int, H: int, Hkv: int, d: int, period: int, seed: int = 0):
    """Like make_inputs, but only `period` tokens per sequence are drawn and then repeated along N
    (N a multiple of `period`): a quick way to fill very large tensors, e.g. to exercise offsets
    beyond 2^31 elements.  Every batch entry gets its own draw."""
    assert N % period == 0
    q, k, v, dO = make_inputs(B, period, H, Hkv, d, seed)
    reps = N // period
    return tuple(x.repeat(1, reps, 1, 1).contiguous() for x in (q, k, v, dO))


def make_workload_inputs(w: Workload, seed: int = 0):
    return make_inputs(w.B, w.N, w.H, w.Hkv, w.d, seed)


def make_inputs_f64(B: int, N: int, H: int, Hkv: int, d: int, seed: int = 0):
    """fp64 draws for oracle-only tests (finite differences need fp64 inputs)."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    shapes = [(B, N, H, d), (B, N, Hkv, d), (B, N, Hkv, d), (B, N, H, d)]
    return tuple(torch.randn(s, generator=gen, dtype=torch.float64) for s in shapes)
