"""Seeded synthetic inputs for the linear-angular attention core.

This module only draws random tensors and names shapes.  It holds none of the
method's arithmetic, so both the CPU oracle's tests and the CUDA path's tests
and benchmark can share it without sharing any computation.

Every workload is a list of calls; a call is one invocation of the attention
core on per-head tensors laid out ``[B, H, N, d]`` (d innermost, token index
``t = y * gridW + x``) with a depthwise filter bank ``[H*d, ksize, ksize]`` and
a bias ``[H*d]``.

The shapes stand in for the activations of the vision transformers the method
was evaluated in (Sec. 4.1): 14x14 / 7x7 / 4x4 token grids with 32-wide heads
are LeViT stages, 14x14 with 12 heads of width 64 is DeiT-Base at 224 px with
16 px patches, and the 64x64 ... 256x256 grids are the high-resolution /
small-patch regime of the appendix throughput tables.  No dataset or trained
weight is involved: values are i.i.d. Gaussian draws (with a per-token
log-normal scale on Q and K for the DeiT-shaped case, which exercises the
per-token L2 normalisation).

Draw order per call is fixed: q, k, v, dw_weight, dw_bias, then (if any) the
per-token scales of q and of k.  All draws are fp32 from one
``torch.Generator`` on the CPU and are then cast to the call's I/O dtype; the
oracle and the CUDA path both consume the *cast* values.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Iterator, List, Optional

import torch


@dataclass(frozen=True)
class CallShape:
    """Shape of one invocation of the attention core."""

    B: int
    H: int
    gridH: int
    gridW: int
    d: int
    ksize: int
    dtype: str  # "f32" or "bf16"
    w_std: float = 0.1
    qk_lognormal_sigma: float = 0.0  # > 0: per-token scale on q and k

    @property
    def N(self) -> int:
        return self.gridH * self.gridW

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    @property
    def image_tokens(self) -> int:
        """Tokens as an image model counts them: B * N."""
        return self.B * self.N

    @property
    def head_tokens(self) -> int:
        return self.B * self.H * self.N

    @property
    def algorithmic_bytes(self) -> int:
        """Q, K and V read once and the output written once, plus the filters."""
        e = self.elem_bytes
        return 4 * self.B * self.H * self.N * self.d * e + self.H * self.d * (self.ksize ** 2 + 1) * e

    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    def label(self) -> str:
        return (f"B{self.B}_H{self.H}_{self.gridH}x{self.gridW}_d{self.d}_k{self.ksize}_{self.dtype}")


@dataclass(frozen=True)
class Workload:
    name: str
    seed: int
    calls: List[CallShape] = field(default_factory=list)
    note: str = ""


def _sweep(side: int) -> CallShape:
    return CallShape(B=2, H=8, gridH=side, gridW=side, d=64, ksize=3, dtype="bf16")


WORKLOADS: Dict[str, Workload] = {
    # fp32 tiny case
    "c1_fp32_tiny": Workload("c1_fp32_tiny", 0, [CallShape(2, 4, 14, 14, 32, 3, "f32")],
                             "small case the oracle finishes at once"),
    # LeViT-stage shapes, three calls drawn one after another from one generator
    "c2_levit_bf16": Workload("c2_levit_bf16", 1, [
        CallShape(64, 4, 14, 14, 32, 3, "bf16"),
        CallShape(64, 8, 7, 7, 32, 3, "bf16"),
        CallShape(64, 12, 4, 4, 32, 3, "bf16"),
    ], "LeViT-stage shapes"),
    # DeiT-Base shaped, per-token log-normal scales on q and k
    "c3_deit_base_bf16": Workload("c3_deit_base_bf16", 2, [
        CallShape(64, 12, 14, 14, 64, 3, "bf16", qk_lognormal_sigma=0.5)], "DeiT-Base shaped"),
    # detection, high resolution, 5x5 filters with sigma 0.05
    "c4_detection_bf16": Workload("c4_detection_bf16", 3, [
        CallShape(8, 8, 64, 64, 32, 5, "bf16", w_std=0.05)], "detection high-res"),
    # long-sequence sweep: square grids, side doubling, drawn in increasing size
    "c5_sweep_bf16": Workload("c5_sweep_bf16", 4, [_sweep(32), _sweep(64), _sweep(128), _sweep(256)],
                              "long-sequence sweep"),
}


@dataclass
class CallInputs:
    shape: CallShape
    q: torch.Tensor
    k: torch.Tensor
    v: torch.Tensor
    dw_weight: torch.Tensor
    dw_bias: Optional[torch.Tensor]


def draw_call(shape: CallShape, gen: torch.Generator) -> CallInputs:
    """Draw one call's tensors (CPU) from ``gen`` in the fixed order."""
    dims = (shape.B, shape.H, shape.N, shape.d)
    q = torch.randn(dims, generator=gen, dtype=torch.float32)
    k = torch.randn(dims, generator=gen, dtype=torch.float32)
    v = torch.randn(dims, generator=gen, dtype=torch.float32)
    w = torch.randn((shape.H * shape.d, shape.ksize, shape.ksize), generator=gen,
                    dtype=torch.float32) * shape.w_std
    bias = torch.randn((shape.H * shape.d,), generator=gen, dtype=torch.float32) * shape.w_std
    if shape.qk_lognormal_sigma > 0.0:
        sq = torch.randn(dims[:3] + (1,), generator=gen, dtype=torch.float32)
        sk = torch.randn(dims[:3] + (1,), generator=gen, dtype=torch.float32)
        q = q * torch.exp(shape.qk_lognormal_sigma * sq)
        k = k * torch.exp(shape.qk_lognormal_sigma * sk)
    dt = shape.torch_dtype()
    return CallInputs(shape, q.to(dt), k.to(dt), v.to(dt), w.to(dt), bias.to(dt))


def iter_workload(name: str, only: Optional[List[int]] = None, seed_offset: int = 0) -> Iterator[CallInputs]:
    """Yield the calls of a workload in order.

    The generator always advances through every call of the workload so that a
    given call sees the same values whether or not earlier calls are consumed;
    ``only`` selects which call indices are yielded.  ``seed_offset`` gives
    independent replicas (one per rank) of the same workload.
    """
    wl = WORKLOADS[name]
    gen = torch.Generator(device="cpu")
    gen.manual_seed(wl.seed + seed_offset)
    for idx, shape in enumerate(wl.calls):
        if only is not None and idx not in only and max(only) < idx:
            return
        call = draw_call(shape, gen)
        if only is None or idx in only:
            yield call


def custom_call(B: int, H: int, gridH: int, gridW: int, d: int, ksize: int, dtype: str, seed: int,
                w_std: float = 0.1, qk_lognormal_sigma: float = 0.0) -> CallInputs:
    """One call of an arbitrary shape (edge-case and sweep tests)."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    return draw_call(CallShape(B, H, gridH, gridW, d, ksize, dtype, w_std, qk_lognormal_sigma), gen)
