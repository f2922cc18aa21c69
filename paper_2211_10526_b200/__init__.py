"""B200-native linear-angular attention core (Castling-ViT inference attention).

The computation lives in the CUDA library built from ``csrc/``; ``binding`` marshals
arguments to its C ABI and ``CastlingAttn`` is a small convenience wrapper over torch
tensors.  Nothing here computes on the CPU.
"""
from . import binding
from .attn import CastlingAttn

__all__ = ["binding", "CastlingAttn"]
