"""The allocation-free entry point against the ordinary one.

`castling_attn_forward_static` serves callers that are not allowed to allocate device memory
while they run (a serving loop that must not hit cudaMalloc's implicit synchronisation, a
plug-in living inside another program's fixed memory budget): it keeps the state that passes
between its kernels in an array built into the library.  This file calls it through the C ABI,
twice in a row per case, and requires the result to agree with `castling_attn_forward` within
the tolerances the parity tests use, and with the float64 CPU oracle within the same bound.  It is
named to be collected last, so a run that stops at
the first failure has already run every other test.
"""
from __future__ import annotations

import numpy as np
import pytest
import torch

import oracle
import workloads

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "bf16": 2e-2}


def _rel(a: torch.Tensor, b: torch.Tensor) -> float:
    a64, b64 = a.double(), b.double()
    return float((a64 - b64).abs().max() / b64.abs().max().clamp_min(1e-30))


CASES = [
    # B, H, gridH, gridW, d, ksize, dtype
    (2, 4, 14, 14, 32, 3, "f32"),      # the small fp32 configuration
    (2, 3, 9, 11, 64, 3, "bf16"),      # the ordinary entry point runs its tensor-core kernels here
    (1, 2, 48, 50, 32, 5, "f32"),      # token range split: partial states in the scratch too
    (4, 12, 14, 14, 64, 3, "bf16"),
    (200, 1, 32, 32, 64, 3, "bf16"),   # the split partial states would not fit the array: one split per plane instead
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: "x".join(map(str, c)))
def test_static_entry_point_matches_handle_entry_point(case):
    from paper_2211_10526_b200 import CastlingAttn, binding as b
    B, H, gh, gw, d, ks, dtype = case
    dev = torch.device("cuda:0")
    code = b.CASTLING_F32 if dtype == "f32" else b.CASTLING_BF16
    stream = torch.cuda.current_stream(dev).cuda_stream
    with CastlingAttn(ksize=ks) as attn:
        for rep, seed in enumerate((900 + sum(case[:6]), 901 + sum(case[:6]))):  # two calls in a row, new data each
            c = workloads.custom_call(B, H, gh, gw, d, ks, dtype, seed=seed)
            q, k, v, w, bias = (t.to(dev) for t in (c.q, c.k, c.v, c.dw_weight, c.dw_bias))
            want = attn.forward(q, k, v, w, bias, gh, gw)
            got = torch.full_like(q, float("nan"))
            rc = b.castling_attn_forward_static(q.data_ptr(), k.data_ptr(), v.data_ptr(), w.data_ptr(),
                                                bias.data_ptr(), got.data_ptr(), B, H, gh, gw, d, ks, 0.0, code, stream)
            assert rc == b.OK, b.error_string(rc)
            torch.cuda.synchronize()
            assert torch.isfinite(got.float()).all()
            err = _rel(got, want)
            assert err <= TOL[dtype], f"call {rep}: max-rel difference {err:.3e}"
            ref = oracle.forward(c.q, c.k, c.v, c.dw_weight, c.dw_bias, gh, gw, ks, threads=8)
            err = float(np.max(np.abs(got.double().cpu().numpy() - ref)) / np.max(np.abs(ref)))
            assert err <= TOL[dtype], f"call {rep}: max-rel error against the oracle {err:.3e}"


def test_static_entry_point_rejects_what_does_not_fit():
    from paper_2211_10526_b200 import binding as b
    dev = torch.device("cuda:0")
    # B*H*(d*d + d)*4 bytes must fit the built-in array: 260 heads of width 64 do not
    B, H, gh, gw, d = 260, 1, 2, 2, 64
    assert B * H * (d * d + d) * 4 > b.STATIC_SCRATCH_BYTES
    x = torch.zeros((B, H, gh * gw, d), dtype=torch.bfloat16, device=dev)
    out = torch.empty_like(x)
    w = torch.zeros((H * d, 3, 3), dtype=torch.bfloat16, device=dev)
    rc = b.castling_attn_forward_static(x.data_ptr(), x.data_ptr(), x.data_ptr(), w.data_ptr(), None, out.data_ptr(),
                                        B, H, gh, gw, d, 3, 0.0, b.CASTLING_BF16, 0)
    assert rc == b.ERR_SCRATCH_LIMIT
    assert "static scratch" in b.error_string(rc)
    # argument checks come first and launch nothing
    assert b.castling_attn_forward_static(None, x.data_ptr(), x.data_ptr(), w.data_ptr(), None, out.data_ptr(),
                                          1, 1, 2, 2, 64, 3, 0.0, b.CASTLING_BF16, 0) == b.ERR_INVALID_ARG
    assert b.castling_attn_forward_static(x.data_ptr(), x.data_ptr(), x.data_ptr(), w.data_ptr(), None, out.data_ptr(),
                                          1, 1, 2, 2, 64, 4, 0.0, b.CASTLING_BF16, 0) == b.ERR_INVALID_ARG
    # the output may overlap none of the inputs, the filters and the bias included
    big = torch.zeros(4 * 64 + 64 * 9, dtype=torch.bfloat16, device=dev)
    assert b.castling_attn_forward_static(x.data_ptr(), x.data_ptr(), x.data_ptr(), big[128:].data_ptr(), None,
                                          big.data_ptr(), 1, 1, 2, 2, 64, 3, 0.0, b.CASTLING_BF16, 0) == b.ERR_INVALID_ARG
    assert b.castling_attn_forward_static(x.data_ptr(), x.data_ptr(), x.data_ptr(), w.data_ptr(), big[64:].data_ptr(),
                                          big.data_ptr(), 1, 1, 2, 2, 64, 3, 0.0, b.CASTLING_BF16, 0) == b.ERR_INVALID_ARG
    torch.cuda.synchronize()
