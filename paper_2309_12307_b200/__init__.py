"""B200-native shifted sparse attention (S2-Attn, LongLoRA Algorithm 1), forward and backward.

`inputs` (seeded synthetic tensors) is importable anywhere; `binding` loads the
CUDA library and raises if it has not been built.
"""
__all__ = ["inputs", "binding", "autograd", "replicas"]
