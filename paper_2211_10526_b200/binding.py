"""ctypes binding of ``include/castling_attn.h``: argument marshalling only.

Function names mirror the C ABI.  Tensors are passed as raw addresses
(``tensor.data_ptr()``); PyTorch is used by callers for device memory and streams, never
for arithmetic.  Importing this module loads the compiled CUDA library and raises if it
is missing: there is no CPU or PyTorch fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcastling_attn.so")

CASTLING_F32, CASTLING_BF16 = 0, 1
PATH_AUTO, PATH_SIMT, PATH_TENSOR = 0, 1, 2
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_ARCH, ERR_CUDA, ERR_OOM, ERR_DEVICE = 0, -1, -2, -3, -4, -5, -6, -7
ERR_SCRATCH_LIMIT = -8
STATIC_SCRATCH_BYTES = 4 << 20


class castling_attn_config_t(ctypes.Structure):
    _fields_ = [("ksize", ctypes.c_int), ("eps", ctypes.c_double), ("force_path", ctypes.c_int),
                ("max_workspace", ctypes.c_size_t), ("prefix_tokens", ctypes.c_int),
                ("normalize_rows", ctypes.c_int), ("exact_kernel", ctypes.c_int), ("sparse_branch", ctypes.c_int),
                ("sparse_eps", ctypes.c_double)]


class castling_attn_layout_t(ctypes.Structure):
    _fields_ = [(f"{t}_{s}", ctypes.c_longlong) for t in ("q", "k", "v", "out") for s in ("batch", "head", "token")]


class CastlingError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {error_string(code)} (code {code})")
        self.code = code


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is not built; run `python -m paper_2211_10526_b200.build` "
                          "(needs nvcc; there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    lib.castling_attn_create.restype = i
    lib.castling_attn_create.argtypes = [ctypes.POINTER(castling_attn_config_t), ctypes.POINTER(vp)]
    fwd_args = [vp] * 7 + [i] * 5 + [i, vp]
    lib.castling_attn_forward.restype = i
    lib.castling_attn_forward.argtypes = fwd_args
    lib.castling_attn_forward_host.restype = i
    lib.castling_attn_forward_host.argtypes = fwd_args
    lib.castling_attn_forward_strided.restype = i
    lib.castling_attn_forward_strided.argtypes = [vp] * 7 + [i] * 5 + [i, ctypes.POINTER(castling_attn_layout_t), vp]
    lib.castling_attn_destroy.restype = i
    lib.castling_attn_destroy.argtypes = [vp]
    lib.castling_attn_workspace_bytes.restype = sz
    lib.castling_attn_workspace_bytes.argtypes = [i] * 6
    lib.castling_attn_error_string.restype = ctypes.c_char_p
    lib.castling_attn_error_string.argtypes = [i]
    lib.castling_attn_last_cuda_error.restype = i
    lib.castling_attn_last_cuda_error.argtypes = [vp]
    lib.castling_attn_last_path.restype = i
    lib.castling_attn_last_path.argtypes = [vp, ctypes.POINTER(i)]
    lib.castling_attn_device_status.restype = i
    lib.castling_attn_device_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_uint)]
    lib.castling_attn_state_words.restype = sz
    lib.castling_attn_state_words.argtypes = [i]
    lib.castling_attn_shard_state.restype = i
    lib.castling_attn_shard_state.argtypes = [vp] * 4 + [i] * 4 + [i, vp]
    lib.castling_attn_shard_apply.restype = i
    lib.castling_attn_shard_apply.argtypes = [vp] * 7 + [i] * 7 + [i, vp]
    lib.castling_attn_selftest_wait.restype = i
    lib.castling_attn_selftest_wait.argtypes = [vp, ctypes.c_uint, vp]
    lib.castling_attn_set_profiling.restype = i
    lib.castling_attn_set_profiling.argtypes = [vp, i]
    lib.castling_attn_kernel_times.restype = i
    lib.castling_attn_kernel_times.argtypes = [vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_char_p), i]
    lib.castling_attn_forward_static.restype = i
    lib.castling_attn_forward_static.argtypes = [vp] * 6 + [i] * 6 + [ctypes.c_double, i, vp]
    return lib


lib = _load()


def error_string(code: int) -> str:
    return lib.castling_attn_error_string(int(code)).decode()


def castling_attn_create(ksize: int = 3, eps: float = 0.0, force_path: int = PATH_AUTO,
                         max_workspace: int = 0, prefix_tokens: int = 0, normalize_rows: bool = False,
                         exact_kernel: bool = False, sparse_eps: Optional[float] = None) -> int:
    """Returns the handle (an integer address); raises CastlingError on failure.  ``sparse_eps`` other than
    None switches the masked softmax branch on with that threshold."""
    cfg = castling_attn_config_t(int(ksize), float(eps), int(force_path), int(max_workspace), int(prefix_tokens),
                                 int(bool(normalize_rows)), int(bool(exact_kernel)), int(sparse_eps is not None),
                                 float(sparse_eps if sparse_eps is not None else 0.0))
    h = ctypes.c_void_p()
    rc = lib.castling_attn_create(ctypes.byref(cfg), ctypes.byref(h))
    if rc != OK:
        raise CastlingError(rc, "castling_attn_create")
    return h.value


def castling_attn_forward(handle, q: int, k: int, v: int, dw_weight: int, dw_bias: Optional[int], out: int,
                          B: int, H: int, gridH: int, gridW: int, d: int, dtype: int, stream: int = 0) -> int:
    """Raw call on device addresses; returns the C return code."""
    return lib.castling_attn_forward(handle, q, k, v, dw_weight, dw_bias, out, B, H, gridH, gridW, d, dtype,
                                     stream or None)


def castling_attn_forward_strided(handle, q: int, k: int, v: int, dw_weight: int, dw_bias: Optional[int], out: int,
                                  B: int, H: int, gridH: int, gridW: int, d: int, dtype: int, strides,
                                  stream: int = 0) -> int:
    """Raw call on device base addresses; ``strides`` holds the twelve element strides
    (q, k, v, out) x (batch, head, token) in that order.  Returns the C return code."""
    layout = castling_attn_layout_t(*[int(x) for x in strides])
    return lib.castling_attn_forward_strided(handle, q, k, v, dw_weight, dw_bias, out, B, H, gridH, gridW, d, dtype,
                                             ctypes.byref(layout), stream or None)


def castling_attn_forward_host(handle, q: int, k: int, v: int, dw_weight: int, dw_bias: Optional[int], out: int,
                               B: int, H: int, gridH: int, gridW: int, d: int, dtype: int, stream: int = 0) -> int:
    """Raw call on host addresses (copies in, computes, copies out, synchronises)."""
    return lib.castling_attn_forward_host(handle, q, k, v, dw_weight, dw_bias, out, B, H, gridH, gridW, d, dtype,
                                          stream or None)


def castling_attn_destroy(handle) -> int:
    return lib.castling_attn_destroy(handle)


def castling_attn_workspace_bytes(B, H, gridH, gridW, d, dtype) -> int:
    return lib.castling_attn_workspace_bytes(B, H, gridH, gridW, d, dtype)


def castling_attn_last_cuda_error(handle) -> int:
    return lib.castling_attn_last_cuda_error(handle)


def castling_attn_last_path(handle):
    n = ctypes.c_int(0)
    path = lib.castling_attn_last_path(handle, ctypes.byref(n))
    return path, n.value


def castling_attn_device_status(handle, stream: int = 0):
    raw = ctypes.c_uint(0)
    rc = lib.castling_attn_device_status(handle, stream or None, ctypes.byref(raw))
    return rc, raw.value


def castling_attn_state_words(d: int) -> int:
    return int(lib.castling_attn_state_words(int(d)))


def castling_attn_shard_state(handle, k: int, v: int, state_out: int, B: int, H: int, n_tokens: int, d: int, dtype: int,
                              stream: int = 0) -> int:
    return lib.castling_attn_shard_state(handle, k, v, state_out, B, H, n_tokens, d, dtype, stream or None)


def castling_attn_shard_apply(handle, q: int, v_halo: int, dw_weight: int, dw_bias: Optional[int], state: int, out: int,
                              B: int, H: int, gridH_local: int, gridW: int, halo_top: int, halo_bottom: int, d: int,
                              dtype: int, stream: int = 0) -> int:
    return lib.castling_attn_shard_apply(handle, q, v_halo, dw_weight, dw_bias, state, out, B, H, gridH_local, gridW,
                                         halo_top, halo_bottom, d, dtype, stream or None)


def castling_attn_selftest_wait(handle, limit_us: int = 2000, stream: int = 0) -> int:
    """Runs the kernel whose bounded wait must give up; returns the C return code (OK when it did)."""
    return lib.castling_attn_selftest_wait(handle, int(limit_us), stream or None)


def castling_attn_set_profiling(handle, enable: bool) -> int:
    return lib.castling_attn_set_profiling(handle, 1 if enable else 0)


def castling_attn_kernel_times(handle):
    """[(kernel name, milliseconds)] of the handle's most recent forward (empty when profiling is off)."""
    cap = 8
    ms = (ctypes.c_float * cap)()
    names = (ctypes.c_char_p * cap)()
    n = lib.castling_attn_kernel_times(handle, ms, names, cap)
    if n < 0:
        raise CastlingError(n, "castling_attn_kernel_times")
    return [(names[i].decode(), float(ms[i])) for i in range(n)]


def castling_attn_forward_static(q: int, k: int, v: int, dw_weight: int, dw_bias: Optional[int], out: int,
                                 B: int, H: int, gridH: int, gridW: int, d: int, ksize: int, eps: float,
                                 dtype: int, stream: int = 0) -> int:
    """Forward pass that allocates nothing (scratch is a fixed array inside the library); raw device
    addresses in, C return code out.  See the header for the size limit and the sharing rules."""
    return lib.castling_attn_forward_static(q, k, v, dw_weight, dw_bias, out, B, H, gridH, gridW, d, ksize,
                                            float(eps), dtype, stream or None)
