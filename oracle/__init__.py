"""Python face of the CPU oracle (test infrastructure, not product code).

Builds ``castling_oracle.c`` with gcc into a shared object beside it and calls
it through ctypes on float64 numpy arrays.  Nothing here touches CUDA or the
``paper_2211_10526_b200`` package, and that package never imports this one.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may use
this module.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "castling_oracle.c")
_LIB = os.path.join(_HERE, "libcastling_oracle.so")
_lib = None

DEFAULT_EPS = 1e-12

_dp = ctypes.POINTER(ctypes.c_double)


def build(force: bool = False, src: str = _SRC, lib: str = _LIB) -> str:
    """Compile the C oracle (-O2, no fast-math) if it is missing or stale."""
    if force or not os.path.exists(lib) or os.path.getmtime(lib) < os.path.getmtime(src):
        tmp = f"{lib}.{os.getpid()}.tmp"
        subprocess.run(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-o", tmp, src, "-lm"], check=True)
        os.replace(tmp, lib)
    return lib


def _declare(lib: ctypes.CDLL) -> ctypes.CDLL:
    i, dbl = ctypes.c_int, ctypes.c_double
    lib.castling_oracle_forward.restype = i
    lib.castling_oracle_forward.argtypes = [_dp] * 6 + [i] * 6 + [dbl, i, i]
    lib.castling_oracle_forward_prefix.restype = i
    lib.castling_oracle_forward_prefix.argtypes = [_dp] * 6 + [i] * 7 + [dbl, i, i]
    lib.castling_oracle_forward_bruteforce.restype = i
    lib.castling_oracle_forward_bruteforce.argtypes = [_dp] * 6 + [i] * 6 + [dbl]
    lib.castling_oracle_similarity.restype = i
    lib.castling_oracle_similarity.argtypes = [_dp] * 3 + [i, i, dbl]
    lib.castling_oracle_forward_rownorm.restype = i
    lib.castling_oracle_forward_rownorm.argtypes = [_dp] * 6 + [i] * 7 + [dbl, i, i]
    lib.castling_oracle_attention_weights.restype = i
    lib.castling_oracle_attention_weights.argtypes = [_dp] * 3 + [i, i, dbl, i, i, i, dbl]
    lib.castling_oracle_forward_matrix.restype = i
    lib.castling_oracle_forward_matrix.argtypes = [_dp] * 6 + [i] * 6 + [dbl, i, i, i, dbl, i, i]
    lib.castling_oracle_softmax_probs.restype = i
    lib.castling_oracle_softmax_probs.argtypes = [_dp] * 3 + [i, i, dbl]
    lib.castling_oracle_angular_exact.restype = dbl
    lib.castling_oracle_angular_exact.argtypes = [dbl]
    lib.castling_oracle_angular_series.restype = dbl
    lib.castling_oracle_angular_series.argtypes = [dbl, i]
    lib.castling_oracle_angular_series_coeff.restype = dbl
    lib.castling_oracle_angular_series_coeff.argtypes = [i]
    return lib


def load(path: Optional[str] = None) -> ctypes.CDLL:
    """Load (building first if needed) the oracle library; ``path`` loads another build of it."""
    global _lib
    if path is not None:
        return _declare(ctypes.CDLL(path))
    if _lib is None:
        _lib = _declare(ctypes.CDLL(build()))
    return _lib


def _f64(a) -> np.ndarray:
    """float64, C-contiguous numpy view/copy of a numpy array or a CPU torch tensor."""
    if hasattr(a, "detach"):  # torch tensor, any float dtype
        a = a.detach().cpu().double().numpy()
    return np.ascontiguousarray(a, dtype=np.float64)


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(_dp)


def _check_shapes(q, k, v, w, bias, gridH, gridW, ksize, prefix=0):
    if q.ndim != 4 or q.shape != k.shape or q.shape != v.shape:
        raise ValueError("q, k, v must share one [B, H, N, d] shape")
    B, H, N, d = q.shape
    if N != prefix + gridH * gridW:
        raise ValueError("N != prefix + gridH * gridW")
    if w.shape != (H * d, ksize, ksize):
        raise ValueError("dw_weight must be [H*d, ksize, ksize]")
    if bias is not None and bias.shape != (H * d,):
        raise ValueError("dw_bias must be [H*d]")
    return B, H, N, d


def forward(q, k, v, dw_weight, dw_bias, gridH: int, gridW: int, ksize: int,
            eps: float = DEFAULT_EPS, threads: int = 1, lib: Optional[ctypes.CDLL] = None,
            prefix: int = 0) -> np.ndarray:
    """Linear-angular attention core, re-associated form, float64.  Returns [B,H,N,d].

    ``threads`` > 1 splits the independent (b,h) heads over host threads; each
    thread runs the same single-threaded C routine on its own slice.  ``prefix`` > 0:
    the first ``prefix`` tokens of every sequence are off-grid (class tokens): they take
    part in the attention terms but not in the depthwise convolution.
    """
    lib = lib or load()
    q, k, v, w = _f64(q), _f64(k), _f64(v), _f64(dw_weight)
    bias = None if dw_bias is None else _f64(dw_bias)
    B, H, N, d = _check_shapes(q, k, v, w, bias, gridH, gridW, ksize, prefix)
    out = np.empty_like(q)
    BH = B * H
    threads = max(1, min(int(threads), BH))

    def run(lo: int, hi: int) -> int:
        if prefix:
            return lib.castling_oracle_forward_prefix(_ptr(q), _ptr(k), _ptr(v), _ptr(w), _ptr(bias), _ptr(out),
                                                      B, H, int(prefix), gridH, gridW, d, ksize, float(eps), lo, hi)
        return lib.castling_oracle_forward(_ptr(q), _ptr(k), _ptr(v), _ptr(w), _ptr(bias), _ptr(out),
                                           B, H, gridH, gridW, d, ksize, float(eps), lo, hi)

    if threads == 1:
        rcs = [run(0, BH)]
    else:
        cuts = [BH * t // threads for t in range(threads + 1)]
        with ThreadPoolExecutor(max_workers=threads) as pool:
            rcs = list(pool.map(lambda ab: run(*ab), zip(cuts[:-1], cuts[1:])))
    if any(rcs):
        raise RuntimeError("castling_oracle_forward failed")
    return out


def forward_bruteforce(q, k, v, dw_weight, dw_bias, gridH: int, gridW: int, ksize: int,
                       eps: float = DEFAULT_EPS, lib: Optional[ctypes.CDLL] = None) -> np.ndarray:
    """Same result from the explicit N x N similarity matrix (Eq. 8 then Eq. 9); small N only."""
    lib = lib or load()
    q, k, v, w = _f64(q), _f64(k), _f64(v), _f64(dw_weight)
    bias = None if dw_bias is None else _f64(dw_bias)
    B, H, N, d = _check_shapes(q, k, v, w, bias, gridH, gridW, ksize)
    out = np.empty_like(q)
    rc = lib.castling_oracle_forward_bruteforce(_ptr(q), _ptr(k), _ptr(v), _ptr(w), _ptr(bias), _ptr(out),
                                                B, H, gridH, gridW, d, ksize, float(eps))
    if rc:
        raise RuntimeError("castling_oracle_forward_bruteforce failed")
    return out


def similarity(q, k, eps: float = DEFAULT_EPS, lib: Optional[ctypes.CDLL] = None) -> np.ndarray:
    """Explicit similarity matrix 1/2 + q^.k^/pi of one head; q, k are [N, d]."""
    lib = lib or load()
    q, k = _f64(q), _f64(k)
    N, d = q.shape
    sim = np.empty((N, N), dtype=np.float64)
    if lib.castling_oracle_similarity(_ptr(q), _ptr(k), _ptr(sim), N, d, float(eps)):
        raise RuntimeError("castling_oracle_similarity failed")
    return sim


def angular_exact(x: float) -> float:
    """Eq. 5 on a cosine: 1 - arccos(x)/pi."""
    return load().castling_oracle_angular_exact(float(x))


def angular_series(x: float, kmax: int) -> float:
    """Eq. 8 truncated after the k = kmax residual term (kmax = 0: the kept linear part)."""
    return load().castling_oracle_angular_series(float(x), int(kmax))


def angular_series_coeff(k: int) -> float:
    """Eq. 8's coefficient (2k)! / (2^(2k) (k!)^2 (2k+1))."""
    return load().castling_oracle_angular_series_coeff(int(k))


def _threaded(run, BH: int, threads: int, what: str) -> None:
    threads = max(1, min(int(threads), BH))
    if threads == 1:
        rcs = [run(0, BH)]
    else:
        cuts = [BH * t // threads for t in range(threads + 1)]
        with ThreadPoolExecutor(max_workers=threads) as pool:
            rcs = list(pool.map(lambda ab: run(*ab), zip(cuts[:-1], cuts[1:])))
    if any(rcs):
        raise RuntimeError(f"{what} failed")


def forward_rownorm(q, k, v, dw_weight, dw_bias, gridH: int, gridW: int, ksize: int,
                    eps: float = DEFAULT_EPS, threads: int = 1, lib: Optional[ctypes.CDLL] = None,
                    prefix: int = 0) -> np.ndarray:
    """The core with every row of attention weights divided by its sum (Eq. 3's denominator applied to
    the kept kernel of Eq. 8), linear in the number of tokens; the convolution is added unchanged."""
    lib = lib or load()
    q, k, v, w = _f64(q), _f64(k), _f64(v), _f64(dw_weight)
    bias = None if dw_bias is None else _f64(dw_bias)
    B, H, N, d = _check_shapes(q, k, v, w, bias, gridH, gridW, ksize, prefix)
    out = np.empty_like(q)
    _threaded(lambda lo, hi: lib.castling_oracle_forward_rownorm(
        _ptr(q), _ptr(k), _ptr(v), _ptr(w), _ptr(bias), _ptr(out), B, H, int(prefix), gridH, gridW, d, ksize,
        float(eps), lo, hi), B * H, threads, "castling_oracle_forward_rownorm")
    return out


KERNEL_LINEAR, KERNEL_EXACT = 0, 1


def attention_weights(q, k, kernel: int = KERNEL_LINEAR, rownorm: bool = False, sparse_eps: Optional[float] = None,
                      eps: float = DEFAULT_EPS, lib: Optional[ctypes.CDLL] = None) -> np.ndarray:
    """Explicit [N,N] attention weights of one head (q, k: [N,d]): the kept kernel of Eq. 8 or the exact
    angular kernel of Eq. 5, optionally with rows divided by their sums, optionally plus the masked softmax
    of Eq. 10 with threshold ``sparse_eps``."""
    lib = lib or load()
    q, k = _f64(q), _f64(k)
    N, d = q.shape
    wts = np.empty((N, N), dtype=np.float64)
    rc = lib.castling_oracle_attention_weights(_ptr(q), _ptr(k), _ptr(wts), N, d, float(eps), int(kernel), int(bool(rownorm)),
                                               int(sparse_eps is not None), float(sparse_eps or 0.0))
    if rc:
        raise RuntimeError("castling_oracle_attention_weights failed")
    return wts


def forward_matrix(q, k, v, dw_weight, dw_bias, gridH: int, gridW: int, ksize: int, kernel: int = KERNEL_LINEAR,
                   rownorm: bool = False, sparse_eps: Optional[float] = None, eps: float = DEFAULT_EPS,
                   threads: int = 1, lib: Optional[ctypes.CDLL] = None) -> np.ndarray:
    """weights . V + DWConv(V) with the explicit weight matrix of ``attention_weights``; O(N^2 d) per head."""
    lib = lib or load()
    q, k, v, w = _f64(q), _f64(k), _f64(v), _f64(dw_weight)
    bias = None if dw_bias is None else _f64(dw_bias)
    B, H, N, d = _check_shapes(q, k, v, w, bias, gridH, gridW, ksize)
    out = np.empty_like(q)
    _threaded(lambda lo, hi: lib.castling_oracle_forward_matrix(
        _ptr(q), _ptr(k), _ptr(v), _ptr(w), _ptr(bias), _ptr(out), B, H, gridH, gridW, d, ksize, float(eps),
        int(kernel), int(bool(rownorm)), int(sparse_eps is not None), float(sparse_eps or 0.0), lo, hi),
        B * H, threads, "castling_oracle_forward_matrix")
    return out


def softmax_probs(q, k, eps: float = DEFAULT_EPS, lib: Optional[ctypes.CDLL] = None) -> np.ndarray:
    """Softmax over the keys of the cosines of one head (q, k: [N,d]) -> [N,N]."""
    lib = lib or load()
    q, k = _f64(q), _f64(k)
    N, d = q.shape
    p = np.empty((N, N), dtype=np.float64)
    if lib.castling_oracle_softmax_probs(_ptr(q), _ptr(k), _ptr(p), N, d, float(eps)):
        raise RuntimeError("castling_oracle_softmax_probs failed")
    return p
