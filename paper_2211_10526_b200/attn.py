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


def _current_raw_stream(device: torch.device) -> int:
    """Handle of torch's current stream on ``device`` (the short route when torch offers it)."""
    raw = getattr(torch._C, "_cuda_getCurrentRawStream", None)
    if raw is not None and device.index is not None:
        return raw(device.index)
    return torch.cuda.current_stream(device).cuda_stream


class CastlingAttn:
    """Owns one library handle (one stream at a time).

    ``forward`` takes device tensors of shape ``[B, H, N, d]`` (contiguous, or any view whose
    last dimension has stride 1, e.g. ``x.view(B, N, H, d).permute(0, 2, 1, 3)``) and enqueues on
    the current torch stream; ``forward_host`` takes CPU tensors (pinned for best speed) and returns after
    the result has been copied back.
    """

    def __init__(self, ksize: int = 3, eps: float = 0.0, force_path: int = _b.PATH_AUTO, max_workspace: int = 0,
                 prefix_tokens: int = 0, normalize_rows: bool = False, exact_kernel: bool = False,
                 sparse_eps: Optional[float] = None):
        self.ksize = int(ksize)
        self.prefix_tokens = int(prefix_tokens)  # leading off-grid (class) tokens: N = prefix_tokens + gridH * gridW
        # variants: rows of attention weights divided by their sums; the exact angular kernel; the masked
        # softmax branch with threshold sparse_eps (None: off)
        self._h = _b.castling_attn_create(ksize, eps, force_path, max_workspace, prefix_tokens, normalize_rows,
                                          exact_kernel, sparse_eps)

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
        # straight-line on purpose: this runs on every call and small shapes are bound by host time
        shape = q.shape
        if len(shape) != 4 or k.shape != shape or v.shape != shape or out.shape != shape:
            raise ValueError("q, k, v, out must share one [B, H, N, d] shape")
        B, H, N, d = shape
        if N != self.prefix_tokens + gridH * gridW:
            raise ValueError("N != prefix_tokens + gridH * gridW")
        ks = self.ksize
        if w.shape != (H * d, ks, ks):
            raise ValueError("dw_weight must be [H*d, ksize, ksize]")
        dt = q.dtype
        if bias is not None:
            if bias.shape != (H * d,):
                raise ValueError("dw_bias must be [H*d]")
            if bias.device.type != device_type or not bias.is_contiguous() or bias.dtype != dt:
                raise ValueError(f"dw_bias must be a contiguous {device_type} tensor of the tensors' dtype")
        if not (q.device.type == k.device.type == v.device.type == w.device.type == out.device.type == device_type):
            raise ValueError(f"expected {device_type} tensors")
        if not w.is_contiguous():
            raise ValueError("dw_weight must be contiguous")
        if not (q.is_contiguous() and k.is_contiguous() and v.is_contiguous() and out.is_contiguous()):
            if device_type != "cuda":
                raise ValueError("host tensors must be contiguous")
            for t in (q, k, v, out):
                if t.stride(3) != 1:
                    raise ValueError("the d elements of a token must be contiguous (stride 1 in the last dimension)")
        if not (k.dtype == dt and v.dtype == dt and w.dtype == dt and out.dtype == dt):
            raise TypeError("all tensors must share one dtype")
        return B, H, N, d

    def forward(self, q, k, v, dw_weight, dw_bias: Optional[torch.Tensor], gridH: int, gridW: int,
                out: Optional[torch.Tensor] = None) -> torch.Tensor:
        if out is None:
            out = torch.empty_like(q)
        B, H, N, d = self._check(q, k, v, dw_weight, dw_bias, out, gridH, gridW, "cuda")
        stream = _current_raw_stream(q.device)
        bias_ptr = None if dw_bias is None else dw_bias.data_ptr()
        if q.is_contiguous() and k.is_contiguous() and v.is_contiguous() and out.is_contiguous():
            rc = _b.castling_attn_forward(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), dw_weight.data_ptr(),
                                          bias_ptr, out.data_ptr(), B, H, gridH, gridW, d, _dtype_code(q), stream)
        else:  # views of token-major or fused-projection buffers: pass their strides through
            strides = [s for t in (q, k, v, out) for s in t.stride()[:3]]
            rc = _b.castling_attn_forward_strided(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                                  dw_weight.data_ptr(), bias_ptr, out.data_ptr(), B, H, gridH, gridW,
                                                  d, _dtype_code(q), strides, stream)
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

    def shard_state(self, k, v, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Sums over this band's tokens (k, v: contiguous [B, H, n, d] on the device) -> fp32 [B*H, d*d + d]:
        K^^T V row-major, then the token sum of V.  The states of the bands of one sequence add up."""
        if k.shape != v.shape or k.dim() != 4 or not (k.is_contiguous() and v.is_contiguous()) or k.dtype != v.dtype:
            raise ValueError("k, v: contiguous [B, H, n, d] tensors of one dtype")
        B, H, n, d = k.shape
        if out is None:
            out = torch.empty(B * H, _b.castling_attn_state_words(d), dtype=torch.float32, device=k.device)
        rc = _b.castling_attn_shard_state(self._h, k.data_ptr(), v.data_ptr(), out.data_ptr(), B, H, n, d, _dtype_code(k),
                                          _current_raw_stream(k.device))
        if rc != _b.OK:
            raise _b.CastlingError(rc, "castling_attn_shard_state")
        return out

    def shard_apply(self, q, v_halo, dw_weight, dw_bias: Optional[torch.Tensor], state, gridH_local: int, gridW: int,
                    halo_top: int, halo_bottom: int, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Output rows of one band of grid rows from a state summed over all bands; v_halo holds the band's rows of
        V between halo_top rows of the band above and halo_bottom rows of the band below."""
        B, H, n, d = q.shape
        rows = halo_top + gridH_local + halo_bottom
        if n != gridH_local * gridW or tuple(v_halo.shape) != (B, H, rows * gridW, d):
            raise ValueError("q: [B, H, gridH_local*gridW, d]; v_halo: [B, H, (halo_top+gridH_local+halo_bottom)*gridW, d]")
        if not (q.is_contiguous() and v_halo.is_contiguous() and dw_weight.is_contiguous() and state.is_contiguous()):
            raise ValueError("contiguous tensors expected")
        if tuple(state.shape) != (B * H, _b.castling_attn_state_words(d)) or state.dtype != torch.float32:
            raise ValueError("state: fp32 [B*H, d*d + d]")
        if out is None:
            out = torch.empty_like(q)
        rc = _b.castling_attn_shard_apply(self._h, q.data_ptr(), v_halo.data_ptr(), dw_weight.data_ptr(),
                                          None if dw_bias is None else dw_bias.data_ptr(), state.data_ptr(), out.data_ptr(),
                                          B, H, gridH_local, gridW, halo_top, halo_bottom, d, _dtype_code(q),
                                          _current_raw_stream(q.device))
        if rc != _b.OK:
            raise _b.CastlingError(rc, "castling_attn_shard_apply")
        return out

    def last_path(self):
        return _b.castling_attn_last_path(self._h)

    def device_status(self, stream: int = 0):
        return _b.castling_attn_device_status(self._h, stream)
