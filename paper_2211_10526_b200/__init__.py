"""B200-native linear-angular attention core (Castling-ViT inference attention).

The computation lives in the CUDA library built from ``csrc/``; ``binding`` marshals
arguments to its C ABI and ``CastlingAttn`` is a small convenience wrapper over torch
tensors.  Nothing here computes on the CPU.  The library is loaded on first use of
``binding`` or ``CastlingAttn`` (so that ``python -m paper_2211_10526_b200.build`` can
run before it exists) and loading raises if it has not been built.
"""
import importlib

__all__ = ["binding", "CastlingAttn", "build", "sharded"]


def __getattr__(name):
    if name == "CastlingAttn":
        return importlib.import_module(".attn", __name__).CastlingAttn
    if name in ("binding", "build", "attn", "sharded"):
        return importlib.import_module("." + name, __name__)
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")
