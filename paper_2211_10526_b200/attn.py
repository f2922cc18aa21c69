"""Convenience wrapper: torch tensors in, torch tensor out, all arithmetic in the CUDA library."""
from __future__ import annotations

from typing import Optional

import torch

from . import binding as _b


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return _b.CASTLING_F32
    if t.dtype == torch.bfloat16:
        return _b.CASTLING_BF16
    raise TypeError(f"unsupported dtype {t.dtype}: the attention core takes float32 or bfloat16")


class CastlingAttn:
    """Owns one library handle (one stream at a time).

    ``forward`` takes device tensors ``[B, H, N, d]`` and enqueues on the current torch
    stream; ``forward_host`` takes CPU tensors (pinned for best speed) and returns after
    the result has been copied back.
    """

    def __init__(self, ksize: int = 3, eps: float = 0.0, force_path: int = _b.PATH_AUTO, max_workspace: int = 0):
        self.ksize = int(ksize)
        self._h = _b.castling_attn_create(ksize, eps, force_path, max_workspace)

    def close(self) -> None:
        if getattr(self, "_h", None):
            _b.castling_attn_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    @property
    def handle(self) -> int:
        return self._h

    def _check(self, q, k, v, w, bias, out, gridH, gridW, device_type):
        if q.dim() != 4 or q.shape != k.shape or q.shape != v.shape or q.shape != out.shape:
            raise ValueError("q, k, v, out must share one [B, H, N, d] shape")
        B, H, N, d = q.shape
        if N != gridH * gridW:
            raise ValueError("N != gridH * gridW")
        if tuple(w.shape) != (H * d, self.ksize, self.ksize):
            raise ValueError("dw_weight must be [H*d, ksize, ksize]")
        if bias is not None and tuple(bias.shape) != (H * d,):
            raise ValueError("dw_bias must be [H*d]")
        for t in (q, k, v, w, out) + ((bias,) if bias is not None else ()):
            if t.device.type != device_type:
                raise ValueError(f"expected {device_type} tensors")
            if not t.is_contiguous():
                raise ValueError("tensors must be contiguous")
            if t.dtype != q.dtype:
                raise TypeError("all tensors must share one dtype")
        return B, H, N, d

    def forward(self, q, k, v, dw_weight, dw_bias: Optional[torch.Tensor], gridH: int, gridW: int,
                out: Optional[torch.Tensor] = None) -> torch.Tensor:
        if out is None:
            out = torch.empty_like(q)
        B, H, N, d = self._check(q, k, v, dw_weight, dw_bias, out, gridH, gridW, "cuda")
        stream = torch.cuda.current_stream(q.device).cuda_stream
        rc = _b.castling_attn_forward(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), dw_weight.data_ptr(),
                                      None if dw_bias is None else dw_bias.data_ptr(), out.data_ptr(),
                                      B, H, gridH, gridW, d, _dtype_code(q), stream)
        if rc != _b.OK:
            raise _b.CastlingError(rc, "castling_attn_forward")
        return out

    def forward_host(self, q, k, v, dw_weight, dw_bias: Optional[torch.Tensor], gridH: int, gridW: int,
                     out: Optional[torch.Tensor] = None, stream: int = 0) -> torch.Tensor:
        if out is None:
            out = torch.empty_like(q)
        B, H, N, d = self._check(q, k, v, dw_weight, dw_bias, out, gridH, gridW, "cpu")
        rc = _b.castling_attn_forward_host(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), dw_weight.data_ptr(),
                                           None if dw_bias is None else dw_bias.data_ptr(), out.data_ptr(),
                                           B, H, gridH, gridW, d, _dtype_code(q), stream)
        if rc != _b.OK:
            raise _b.CastlingError(rc, "castling_attn_forward_host")
        return out

    def last_path(self):
        return _b.castling_attn_last_path(self._h)

    def device_status(self, stream: int = 0):
        return _b.castling_attn_device_status(self._h, stream)
