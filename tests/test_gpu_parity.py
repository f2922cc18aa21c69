"""GPU parity: the CUDA library against the float64 CPU oracle, through the C ABI.

Error metric (both tolerances come with the method's acceptance bar): per call,
``max_i |gpu_i - ref_i| / max_i |ref_i|`` must be <= 1e-5 for fp32 I/O and <= 2e-2 for
bf16 I/O.  The oracle consumes the already-rounded fp32/bf16 inputs widened to float64
and its output is not rounded.  Term-isolation cases make one term of Eq. 9 the whole
output so that a defect in a small term cannot hide under a large one.
"""
from __future__ import annotations

import numpy as np
import pytest
import torch

import oracle
import workloads

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "bf16": 2e-2}


def _lib():
    import paper_2211_10526_b200 as pkg
    return pkg


def rel_err(got: torch.Tensor, ref: np.ndarray) -> float:
    g = got.detach().double().cpu().numpy()
    assert np.all(np.isfinite(g)), "non-finite GPU output"
    return float(np.max(np.abs(g - ref)) / max(np.max(np.abs(ref)), 1e-30))


def run_gpu(call: workloads.CallInputs, force_path: int = 0, bias: bool = True) -> torch.Tensor:
    pkg = _lib()
    s = call.shape
    dev = torch.device("cuda:0")
    q, k, v, w = (t.to(dev) for t in (call.q, call.k, call.v, call.dw_weight))
    b = call.dw_bias.to(dev) if (bias and call.dw_bias is not None) else None
    with pkg.CastlingAttn(ksize=s.ksize, force_path=force_path) as attn:
        out = attn.forward(q, k, v, w, b, s.gridH, s.gridW)
        torch.cuda.synchronize()
        rc, raw = attn.device_status()
        assert rc == 0, f"device status word {raw:#x}"
    return out


def run_oracle(call: workloads.CallInputs, bias: bool = True, threads: int = 8) -> np.ndarray:
    s = call.shape
    return oracle.forward(call.q, call.k, call.v, call.dw_weight, call.dw_bias if bias else None,
                          s.gridH, s.gridW, s.ksize, threads=threads)


def check(call, force_path=0, bias=True, tol=None):
    ref = run_oracle(call, bias)
    got = run_gpu(call, force_path, bias)
    err = rel_err(got, ref)
    tol = TOL[call.shape.dtype] if tol is None else tol
    assert err <= tol, f"{call.shape.label()}: max-rel error {err:.3e} > {tol:.1e}"
    return err


# ---------------------------------------------------------------------------
# the five configurations
# ---------------------------------------------------------------------------
CONFIG_CALLS = [("c1_fp32_tiny", 0), ("c2_levit_bf16", 0), ("c2_levit_bf16", 1), ("c2_levit_bf16", 2),
                ("c3_deit_base_bf16", 0), ("c4_detection_bf16", 0), ("c5_sweep_bf16", 0), ("c5_sweep_bf16", 1)]


@pytest.mark.parametrize("name,idx", CONFIG_CALLS, ids=[f"{n}-{i}" for n, i in CONFIG_CALLS])
def test_config_parity(name, idx):
    (call,) = list(workloads.iter_workload(name, only=[idx]))
    check(call)


@pytest.mark.parametrize("idx", [2, 3], ids=["side128", "side256"])
def test_long_sequence_full_size(idx):
    """Largest sweep points, every element compared."""
    (call,) = list(workloads.iter_workload("c5_sweep_bf16", only=[idx]))
    check(call)


# ---------------------------------------------------------------------------
# term isolation (Eq. 9 one term at a time)
# ---------------------------------------------------------------------------
def _iso_call(dtype, seed, B=2, H=3, gh=9, gw=11, d=32, ks=3):
    return workloads.custom_call(B, H, gh, gw, d, ks, dtype, seed)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("d", [32, 64])
def test_linear_term_alone(dtype, d):
    """Zero filters, zero bias and V with zero token-sum: only (1/pi) q^ (K^^T V) is left."""
    c = _iso_call(dtype, 201, d=d)
    v = c.v.float()
    v = v - v.mean(dim=2, keepdim=True)
    c.v = v.to(c.v.dtype)
    c.dw_weight.zero_(); c.dw_bias.zero_()
    check(c)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_half_sum_term_alone(dtype):
    """Constant V: output is c (N/2 + q^ . sum k^ / pi); dominated by the 1/2 term."""
    c = _iso_call(dtype, 202)
    c.v[:] = c.v[:, :, :1, :].clone()
    c.dw_weight.zero_(); c.dw_bias.zero_()
    check(c)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("ks", [3, 5])
def test_conv_term_alone(dtype, ks):
    """K = 0 (cosine 0) and zero-sum V: attention part vanishes, the convolution is the output."""
    c = _iso_call(dtype, 203, ks=ks)
    v = c.v.float()
    v = v - v.mean(dim=2, keepdim=True)
    c.v = v.to(c.v.dtype)
    # the token sum of the rounded V is not exactly zero; make the conv term dominate it
    c.dw_weight = (c.dw_weight.float() * 30).to(c.dw_weight.dtype)
    c.k.zero_()
    check(c)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_delta_filter_is_identity(dtype):
    c = _iso_call(dtype, 204)
    c.dw_weight.zero_(); c.dw_weight[:, 1, 1] = 1.0
    c.dw_bias.zero_()
    c.k.zero_()
    v = c.v.float(); v = v - v.mean(dim=2, keepdim=True); c.v = v.to(c.v.dtype)
    got = run_gpu(c).double().cpu().numpy()
    half_sum = 0.5 * c.v.double().sum(dim=2, keepdim=True).numpy()
    np.testing.assert_allclose(got, c.v.double().numpy() + half_sum, rtol=0, atol=2e-2 if dtype == "bf16" else 1e-5)


# ---------------------------------------------------------------------------
# shapes, edges
# ---------------------------------------------------------------------------
EDGE = [
    # B, H, gridH, gridW, d, ksize
    (1, 1, 1, 1, 32, 3), (1, 1, 1, 1, 16, 7), (1, 2, 4, 4, 32, 5), (2, 1, 2, 2, 64, 7), (1, 3, 3, 17, 32, 3),
    (1, 1, 13, 5, 64, 3), (3, 2, 8, 8, 16, 1), (1, 1, 33, 31, 64, 3), (2, 2, 5, 13, 48, 5), (1, 2, 7, 9, 80, 3),
    (1, 1, 6, 11, 96, 3), (1, 2, 10, 3, 112, 3), (1, 1, 12, 12, 128, 3), (1, 1, 65, 63, 32, 5), (1, 1, 40, 52, 64, 7),
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", EDGE, ids=lambda s: "x".join(map(str, s)))
def test_edge_shapes(shape, dtype):
    c = workloads.custom_call(*shape, dtype, seed=300 + sum(shape))
    check(c)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_no_bias(dtype):
    c = workloads.custom_call(2, 2, 6, 7, 32, 3, dtype, seed=310)
    check(c, bias=False)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_zero_rows(dtype):
    """A zero query or key row has cosine 0 with everything (eps floor), never NaN."""
    c = workloads.custom_call(1, 2, 5, 5, 32, 3, dtype, seed=311)
    c.q[0, 0, 3] = 0
    c.k[0, 1, 7] = 0
    c.k[0, 0, 0] = 0
    check(c)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_scale_invariance_large_dynamic_range(dtype):
    """Per-token scales over several orders of magnitude leave the result unchanged."""
    c = workloads.custom_call(1, 2, 8, 8, 64, 3, dtype, seed=312, qk_lognormal_sigma=3.0)
    check(c)


def test_many_heads_small_grid():
    c = workloads.custom_call(32, 12, 4, 4, 32, 3, "bf16", seed=313)
    check(c)


def test_split_state_path_fp32():
    """N large enough that the state kernel splits the token range (partials + reduce)."""
    c = workloads.custom_call(1, 2, 48, 50, 32, 3, "f32", seed=314)
    check(c)
    c = workloads.custom_call(1, 1, 70, 77, 64, 5, "f32", seed=315)
    check(c)


# Many planes of few tokens: the CUDA-core path runs its single-launch kernel (one CTA per (b,h),
# the whole plane in shared memory).  B, H, gridH, gridW, d, ksize
FUSED_SHAPES = [(16, 4, 1, 1, 32, 3), (8, 8, 1, 1, 16, 7), (32, 2, 4, 4, 32, 5), (16, 4, 2, 2, 64, 7),
                (64, 1, 3, 17, 32, 3), (8, 8, 13, 5, 64, 3), (64, 2, 8, 8, 16, 1), (4, 16, 5, 13, 48, 5),
                (16, 4, 7, 9, 80, 3), (64, 1, 4, 8, 96, 3), (8, 8, 3, 5, 112, 3), (16, 4, 4, 4, 128, 3),
                (8, 8, 14, 14, 32, 3), (8, 8, 16, 16, 16, 5)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", FUSED_SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_single_launch_kernel_parity(shape, dtype):
    pkg = _lib()
    c = workloads.custom_call(*shape, dtype, seed=330 + sum(shape))
    s = c.shape
    ref = run_oracle(c)
    dev = torch.device("cuda:0")
    q, k, v, w, b = (t.to(dev) for t in (c.q, c.k, c.v, c.dw_weight, c.dw_bias))
    with pkg.CastlingAttn(ksize=s.ksize, force_path=pkg.binding.PATH_SIMT) as attn:
        out = attn.forward(q, k, v, w, b, s.gridH, s.gridW)
        torch.cuda.synchronize()
        assert attn.last_path() == (pkg.binding.PATH_SIMT, 1), "expected the one-launch kernel"
        out_nb = attn.forward(q, k, v, w, None, s.gridH, s.gridW)
        torch.cuda.synchronize()
    assert rel_err(out, ref) <= TOL[dtype]
    ref_nb = run_oracle(c, bias=False)
    assert rel_err(out_nb, ref_nb) <= TOL[dtype]


def test_single_launch_kernel_zero_rows_and_few_planes():
    """Zero q/k rows in the one-launch kernel; and with few planes the three-kernel path is kept."""
    pkg = _lib()
    c = workloads.custom_call(16, 4, 5, 5, 32, 3, "f32", seed=331)
    c.q[0, 0, 3] = 0
    c.k[3, 1, 7] = 0
    c.k[15, 3, 24] = 0
    check(c)
    few = workloads.custom_call(2, 4, 14, 14, 32, 3, "f32", seed=332)
    dev = torch.device("cuda:0")
    with pkg.CastlingAttn(ksize=3) as attn:
        attn.forward(*(t.to(dev) for t in (few.q, few.k, few.v, few.dw_weight, few.dw_bias)), 14, 14)
        torch.cuda.synchronize()
        assert attn.last_path() == (pkg.binding.PATH_SIMT, 2)


# ---------------------------------------------------------------------------
# leading off-grid tokens (class tokens): in the attention terms, not in the convolution
# ---------------------------------------------------------------------------
def _prefix_call(B, H, P, gh, gw, d, ks, dtype, seed):
    """Inputs for sequences of P + gh*gw tokens (drawn as one row of that many tokens)."""
    c = workloads.custom_call(B, H, 1, P + gh * gw, d, ks, dtype, seed=seed)
    return c


# B, H, prefix, gridH, gridW, d, ksize, dtype, layout, kernel family expected, launches expected
PREFIX_CASES = [
    (2, 3, 1, 5, 7, 32, 3, "f32", "head_major", 1, 2),       # CUDA cores, three-kernel path (no split)
    (1, 2, 2, 40, 33, 48, 5, "f32", "head_major", 1, 3),     # CUDA cores, token range split
    (16, 4, 1, 7, 7, 32, 3, "bf16", "head_major", 1, 1),     # CUDA cores, single-launch kernel (odd N)
    (4, 12, 1, 14, 14, 64, 3, "bf16", "head_major", 2, 1),   # DeiT-shaped with a class token: single tensor-core kernel
    (2, 3, 2, 15, 16, 64, 5, "bf16", "head_major", 2, 1),    # 242 tokens, 5 x 5
    (2, 2, 1, 24, 20, 64, 3, "bf16", "head_major", 2, 3),    # state + apply + leading rows
    (1, 2, 3, 37, 53, 64, 5, "bf16", "head_major", 2, 3),
    (2, 2, 2, 24, 20, 32, 3, "bf16", "head_major", 2, 1),    # width 32, even N: token pairs, single kernel (241 rows)
    (2, 2, 2, 40, 30, 32, 5, "bf16", "head_major", 2, 3),    # ... state + apply + leading rows
    (2, 2, 1, 24, 20, 32, 3, "bf16", "head_major", 1, 3),    # width 32, odd N: CUDA cores (P = 2 splits)
    (2, 4, 1, 24, 20, 32, 5, "bf16", "token_major", 2, 3),   # width 32 token-major: head pairs
    (2, 4, 1, 12, 12, 32, 3, "bf16", "token_major", 2, 1),   # ... in the single-kernel forward
    (2, 3, 1, 14, 14, 64, 3, "bf16", "token_major", 2, 1),
    (1, 2, 2, 30, 31, 64, 3, "bf16", "fused_qkv", 2, 3),
]


@pytest.mark.parametrize("case", PREFIX_CASES, ids=lambda c: "x".join(map(str, c[:9])))
def test_prefix_tokens(case):
    from paper_2211_10526_b200 import CastlingAttn, binding
    B, H, P, gh, gw, d, ks, dtype, layout, family, n_launch = case
    c = _prefix_call(B, H, P, gh, gw, d, ks, dtype, seed=900 + sum(case[:7]))
    dev = torch.device("cuda:0")
    if layout == "head_major":
        q, k, v = (t.to(dev) for t in (c.q, c.k, c.v))
        guard = torch.full((q.numel() + 4096,), 7.0, dtype=q.dtype, device=dev)
        out = guard[2048:2048 + q.numel()].view_as(q)
    else:
        q, k, v, out, _ = _strided_views(c, layout, dev)
        guard = None
    w, b = c.dw_weight.to(dev), c.dw_bias.to(dev)
    with CastlingAttn(ksize=ks, prefix_tokens=P) as attn:
        attn.forward(q, k, v, w, b, gh, gw, out=out)
        torch.cuda.synchronize()
        assert attn.device_status() == (0, 0)
        assert attn.last_path() == (family, n_launch)
        out_nb = attn.forward(q, k, v, w, None, gh, gw)
        torch.cuda.synchronize()
    if guard is not None:
        assert bool((guard[:2048] == 7.0).all()) and bool((guard[-2048:] == 7.0).all()), "wrote outside the output"
    ref = oracle.forward(c.q, c.k, c.v, c.dw_weight, c.dw_bias, gh, gw, ks, threads=8, prefix=P)
    assert rel_err(out, ref) <= TOL[dtype]
    ref_nb = oracle.forward(c.q, c.k, c.v, c.dw_weight, None, gh, gw, ks, threads=8, prefix=P)
    assert rel_err(out_nb, ref_nb) <= TOL[dtype]


def test_prefix_tokens_conv_term_alone():
    """Only the convolution (with a bias of about 3) left: the leading rows stay near zero (what is left of
    1/2 sum V after rounding), the grid rows are the filtered grid."""
    from paper_2211_10526_b200 import CastlingAttn
    dev = torch.device("cuda:0")
    for dtype, shape in (("f32", (2, 2, 2, 9, 11, 32, 3)), ("bf16", (2, 2, 1, 24, 20, 64, 3)), ("bf16", (2, 2, 1, 12, 16, 64, 5))):
        B, H, P, gh, gw, d, ks = shape
        c = _prefix_call(B, H, P, gh, gw, d, ks, dtype, seed=950 + sum(shape))
        v = c.v.float(); c.v = (v - v.mean(dim=2, keepdim=True)).to(c.v.dtype)
        c.k.zero_()
        c.dw_weight = (c.dw_weight.float() * 30).to(c.v.dtype)
        c.dw_bias = (c.dw_bias.float() + 3).to(c.v.dtype)   # a bias that would show on a leading row
        with CastlingAttn(ksize=ks, prefix_tokens=P) as attn:
            out = attn.forward(*(t.to(dev) for t in (c.q, c.k, c.v, c.dw_weight, c.dw_bias)), gh, gw)
            torch.cuda.synchronize()
        ref = oracle.forward(c.q, c.k, c.v, c.dw_weight, c.dw_bias, gh, gw, ks, threads=8, prefix=P)
        assert rel_err(out, ref) <= TOL[dtype]
        lead = out[:, :, :P].float().abs().max().item()
        assert lead < 0.5, f"leading rows carry {lead}: the convolution or its bias leaked"


# ---------------------------------------------------------------------------
# strided layouts: token-major [B,N,H,d], a fused [B,N,3,H,d] projection buffer, padded token rows
# ---------------------------------------------------------------------------
def _strided_views(call, layout, dev):
    """q, k, v, out as [B,H,N,d] views of differently laid out device buffers, plus the buffer that holds out."""
    s = call.shape
    B, H, N, d = s.B, s.H, s.N, s.d
    dt = s.torch_dtype()
    if layout == "token_major":
        mk = lambda t: t.permute(0, 2, 1, 3).contiguous().to(dev).permute(0, 2, 1, 3)
        q, k, v = mk(call.q), mk(call.k), mk(call.v)
        obuf = torch.full((B, N, H, d), 7.0, dtype=dt, device=dev)
        out = obuf.permute(0, 2, 1, 3)
    elif layout == "fused_qkv":
        qkv = torch.stack([t.permute(0, 2, 1, 3) for t in (call.q, call.k, call.v)], dim=2).contiguous().to(dev)  # [B,N,3,H,d]
        q, k, v = (qkv[:, :, i].permute(0, 2, 1, 3) for i in range(3))
        obuf = torch.full((B, N, H, d), 7.0, dtype=dt, device=dev)
        out = obuf.permute(0, 2, 1, 3)
    else:  # "padded": head-major with token rows twice as long as d
        def mk(t):
            buf = torch.full((B, H, N, 2 * d), 7.0, dtype=dt, device=dev)
            buf[..., :d] = t.to(dev)
            return buf[..., :d]
        q, k, v = mk(call.q), mk(call.k), mk(call.v)
        obuf = torch.full((B, H, N, 2 * d), 7.0, dtype=dt, device=dev)
        out = obuf[..., :d]
    return q, k, v, out, obuf


# B, H, gridH, gridW, d, ksize, dtype, kernel family expected for the token-major layout
LAYOUT_CASES = [(2, 3, 9, 11, 32, 3, "f32", 1), (2, 4, 14, 14, 64, 3, "bf16", 2), (2, 3, 24, 20, 64, 3, "bf16", 2),
                (1, 2, 37, 53, 64, 5, "bf16", 2), (2, 4, 14, 14, 32, 3, "bf16", 1), (64, 2, 7, 7, 32, 3, "bf16", 1),
                (1, 1, 7, 8, 64, 3, "bf16", 2), (3, 1, 8, 16, 64, 3, "bf16", 2), (2, 2, 40, 66, 32, 5, "bf16", 1),
                (2, 6, 33, 21, 32, 3, "bf16", 1), (3, 3, 16, 16, 32, 3, "bf16", 1), (1, 8, 5, 7, 32, 5, "bf16", 1),
                (8, 8, 64, 64, 32, 5, "bf16", 1)]


@pytest.mark.parametrize("layout", ["token_major", "fused_qkv", "padded"])
@pytest.mark.parametrize("case", LAYOUT_CASES, ids=lambda c: "x".join(map(str, c[:7])))
def test_strided_layouts(case, layout):
    from paper_2211_10526_b200 import CastlingAttn, binding
    *shape, dtype, family = case
    c = workloads.custom_call(*shape, dtype, seed=800 + sum(shape))
    s = c.shape
    dev = torch.device("cuda:0")
    q, k, v, out, obuf = _strided_views(c, layout, dev)
    assert not out.is_contiguous() or s.H == 1 or s.N == 1
    w, b = c.dw_weight.to(dev), c.dw_bias.to(dev)
    with CastlingAttn(ksize=s.ksize) as attn:
        attn.forward(q, k, v, w, b, s.gridH, s.gridW, out=out)
        torch.cuda.synchronize()
        assert attn.device_status() == (0, 0)
        used, _ = attn.last_path()
    if layout == "padded":
        assert bool((obuf[..., s.d:] == 7.0).all()), "wrote into the padding between token rows"
    if s.d == 32 and dtype == "bf16":
        # token-major width-32 heads: two heads share a 128-byte row on the tensor-core path (even H, at least
        # 48 tokens); padded rows leave neither two tokens nor two heads side by side
        family = 2 if (layout != "padded" and s.H % 2 == 0 and s.N >= 48) else 1
    assert used == family, f"kernel family {used}, expected {family}"
    assert rel_err(out, run_oracle(c)) <= TOL[dtype]


@pytest.mark.parametrize("grid", [(12, 20), (24, 20)], ids=["one_kernel", "two_kernels"])
def test_token_major_head_pairs_term_isolation(grid):
    """Width-32 heads stored [B,N,H,32]: two heads share a 128-byte row on the tensor-core path.  With the
    other terms removed, any leak between the two heads of a row (the off-diagonal blocks of the paired
    state, a norm taken over the whole row) is the whole error."""
    from paper_2211_10526_b200 import CastlingAttn, binding
    gh, gw = grid
    dev = torch.device("cuda:0")

    def run(c):
        s = c.shape
        q, k, v, out, _ = _strided_views(c, "token_major", dev)
        with CastlingAttn(ksize=s.ksize) as attn:
            attn.forward(q, k, v, c.dw_weight.to(dev), c.dw_bias.to(dev), gh, gw, out=out)
            torch.cuda.synchronize()
            assert attn.device_status() == (0, 0)
            assert attn.last_path()[0] == binding.PATH_TENSOR
        err = rel_err(out, run_oracle(c))
        assert err <= TOL["bf16"], err

    base = lambda seed: workloads.custom_call(2, 4, gh, gw, 32, 3, "bf16", seed=seed)
    c = base(631)  # linear term alone, heads of very different scale
    v = c.v.float(); c.v = (v - v.mean(dim=2, keepdim=True)).to(torch.bfloat16)
    c.v[:, 1::2] *= 64
    c.q[:, 0::2] *= 1e-3; c.k[:, 1::2] *= 1e3
    c.dw_weight.zero_(); c.dw_bias.zero_()
    run(c)
    c = base(632)  # one head of each pair has all-zero keys: its linear term vanishes, its neighbour's does not
    v = c.v.float(); c.v = (v - v.mean(dim=2, keepdim=True)).to(torch.bfloat16)
    c.k[:, 0::2] = 0
    c.dw_weight.zero_(); c.dw_bias.zero_()
    run(c)
    c = base(633)  # 1/2 sum (constant V per head)
    c.v[:] = c.v[:, :, :1, :].clone()
    c.dw_weight.zero_(); c.dw_bias.zero_()
    run(c)
    c = base(634)  # convolution alone
    v = c.v.float(); c.v = (v - v.mean(dim=2, keepdim=True)).to(torch.bfloat16)
    c.dw_weight = (c.dw_weight.float() * 30).to(torch.bfloat16)
    c.k.zero_()
    run(c)


def _random_cases(n, seed):
    rng = np.random.default_rng(seed)
    cases = []
    for i in range(n):
        dtype = "bf16" if rng.random() < 0.7 else "f32"
        d = int(rng.choice([32, 64, 32, 64, 16, 48, 96, 128])) if dtype == "bf16" else int(rng.choice([16, 32, 64, 80]))
        ks = int(rng.choice([3, 5, 3, 5, 1, 7]))
        big = rng.random() < 0.3
        gh, gw = (int(rng.integers(1, 60)), int(rng.integers(1, 60))) if big else (int(rng.integers(1, 17)), int(rng.integers(1, 17)))
        B, H = (int(rng.integers(1, 3)), int(rng.integers(1, 5))) if big else (int(rng.integers(1, 40)), int(rng.integers(1, 7)))
        prefix = int(rng.choice([0, 0, 1, 2, 3]))
        layout = str(rng.choice(["head_major", "head_major", "token_major", "fused_qkv", "padded"]))
        cases.append((B, H, prefix, gh, gw, d, ks, dtype, layout, 1000 + i))
    return cases


@pytest.mark.parametrize("case", _random_cases(128, 20221118), ids=lambda c: "x".join(map(str, c[:9])))
def test_random_shapes_layouts_and_leading_tokens(case):
    """Seeded random shapes across dtypes, head widths, filter sizes, leading tokens and memory layouts:
    whatever kernel family the dispatcher picks, the result is the oracle's."""
    from paper_2211_10526_b200 import CastlingAttn
    B, H, P, gh, gw, d, ks, dtype, layout, seed = case
    c = _prefix_call(B, H, P, gh, gw, d, ks, dtype, seed=seed)
    dev = torch.device("cuda:0")
    if layout == "head_major":
        q, k, v = (t.to(dev) for t in (c.q, c.k, c.v))
        out = torch.empty_like(q)
    else:
        q, k, v, out, _ = _strided_views(c, layout, dev)
    bias = c.dw_bias.to(dev) if seed % 4 else None
    with CastlingAttn(ksize=ks, prefix_tokens=P) as attn:
        attn.forward(q, k, v, c.dw_weight.to(dev), bias, gh, gw, out=out)
        again = torch.empty_like(out)
        attn.forward(q, k, v, c.dw_weight.to(dev), bias, gh, gw, out=again)
        torch.cuda.synchronize()
        assert attn.device_status() == (0, 0)
    ref = oracle.forward(c.q, c.k, c.v, c.dw_weight, c.dw_bias if bias is not None else None, gh, gw, ks, threads=8, prefix=P)
    assert rel_err(out, ref) <= TOL[dtype]
    assert torch.equal(out, again), "two runs differ bitwise"


def test_strided_entry_point_rejects_bad_strides():
    from paper_2211_10526_b200 import binding
    c = workloads.custom_call(2, 2, 4, 4, 32, 3, "f32", seed=801)
    dev = torch.device("cuda:0")
    q, k, v, w, b = (t.to(dev) for t in (c.q, c.k, c.v, c.dw_weight, c.dw_bias))
    out = torch.empty_like(q)
    h = binding.castling_attn_create(3)
    good = [2 * 16 * 32, 16 * 32, 32] * 4
    call = lambda st, o=out: binding.castling_attn_forward_strided(
        h, q.data_ptr(), k.data_ptr(), v.data_ptr(), w.data_ptr(), b.data_ptr(), o.data_ptr(), 2, 2, 4, 4, 32,
        binding.CASTLING_F32, st)
    try:
        assert call(good) == binding.OK
        torch.cuda.synchronize()
        assert rel_err(out, run_oracle(c)) <= TOL["f32"]
        bad = list(good); bad[2] = 16          # token stride shorter than d
        assert call(bad) == binding.ERR_INVALID_ARG
        bad = list(good); bad[5] = 34          # not a multiple of 16 bytes
        assert call(bad) == binding.ERR_ALIGNMENT
        bad = list(good); bad[6] = 0           # B > 1 with batch stride 0
        assert call(bad) == binding.ERR_INVALID_ARG
        bad = list(good); bad[9] = -1024
        assert call(bad) == binding.ERR_INVALID_ARG
        assert call(good, q) == binding.ERR_INVALID_ARG  # out aliases an input
    finally:
        binding.castling_attn_destroy(h)


# ---------------------------------------------------------------------------
# kernel families: the tensor-core path must be the one that runs where it applies
# ---------------------------------------------------------------------------
TENSOR_SHAPES = [(2, 8, 32, 32, 64, 3), (1, 2, 8, 16, 64, 3), (1, 1, 1, 1, 64, 3), (2, 3, 14, 14, 64, 3),
                 (1, 2, 37, 53, 64, 3), (1, 2, 24, 40, 64, 5), (1, 1, 3, 130, 64, 3), (1, 1, 200, 5, 64, 5),
                 (3, 5, 64, 64, 64, 3),
                 # head width 32 on even-width grids: two tokens share a 128-byte row
                 (2, 4, 14, 14, 32, 3), (1, 2, 64, 64, 32, 5), (1, 3, 9, 22, 32, 3), (1, 1, 5, 2, 32, 5),
                 (2, 2, 40, 66, 32, 5), (1, 1, 1, 2, 32, 3), (1, 2, 33, 34, 32, 3), (64, 12, 4, 4, 32, 3)]


@pytest.mark.parametrize("shape", TENSOR_SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_tensor_path_parity(shape):
    from paper_2211_10526_b200 import CastlingAttn, binding
    c = workloads.custom_call(*shape, "bf16", seed=500 + sum(shape))
    ref = run_oracle(c)
    s = c.shape
    dev = torch.device("cuda:0")
    args = [t.to(dev) for t in (c.q, c.k, c.v, c.dw_weight, c.dw_bias)]
    errs = {}
    for path in (binding.PATH_TENSOR, binding.PATH_SIMT, binding.PATH_AUTO):
        with CastlingAttn(ksize=s.ksize, force_path=path) as attn:
            out = attn.forward(*args, s.gridH, s.gridW)
            torch.cuda.synchronize()
            assert attn.device_status() == (0, 0)
            used, launches = attn.last_path()
        if path != binding.PATH_AUTO:
            assert used == path
        else:
            rows = s.N if s.d == 64 else s.N // 2   # 128-byte rows per (b,h); tiny problems stay on CUDA cores
            want = binding.PATH_TENSOR if rows >= 48 else binding.PATH_SIMT
            assert used == want, "automatic dispatch picked the wrong kernel family"
        errs[path] = rel_err(out, ref)
    assert max(errs.values()) <= TOL["bf16"], errs


def test_tensor_path_term_isolation():
    """Each term of Eq. 9 alone, on the tensor-core kernels."""
    from paper_2211_10526_b200 import binding
    base = lambda seed: workloads.custom_call(2, 2, 24, 20, 64, 3, "bf16", seed=seed)
    # linear term alone
    c = base(601)
    v = c.v.float(); c.v = (v - v.mean(dim=2, keepdim=True)).to(torch.bfloat16)
    c.dw_weight.zero_(); c.dw_bias.zero_()
    check(c, force_path=binding.PATH_TENSOR)
    # 1/2 sum alone (plus its linear companion)
    c = base(602)
    c.v[:] = c.v[:, :, :1, :].clone()
    c.dw_weight.zero_(); c.dw_bias.zero_()
    check(c, force_path=binding.PATH_TENSOR)
    # convolution alone
    c = base(603)
    v = c.v.float(); c.v = (v - v.mean(dim=2, keepdim=True)).to(torch.bfloat16)
    c.dw_weight = (c.dw_weight.float() * 30).to(torch.bfloat16)
    c.k.zero_()
    check(c, force_path=binding.PATH_TENSOR)
    # zero rows
    c = base(604)
    c.q[0, 0, 5] = 0; c.k[1, 1, 17] = 0
    check(c, force_path=binding.PATH_TENSOR)


# Short sequences of width-64 heads (N <= 256): one tensor-core kernel does the whole pass.
# B, H, gridH, gridW, d, ksize
ONE_KERNEL_SHAPES = [(1, 1, 1, 1, 64, 3), (2, 3, 14, 14, 64, 3), (1, 2, 16, 16, 64, 3), (3, 2, 1, 129, 64, 3),
                     (2, 2, 3, 70, 64, 5), (1, 1, 128, 1, 64, 3), (1, 3, 9, 14, 64, 5), (5, 70, 8, 8, 64, 3),
                     (1, 1, 2, 128, 64, 5), (2, 1, 127, 1, 64, 5), (37, 9, 5, 7, 64, 3),
                     # width-32 heads, two tokens per row (even grid width, at most 512 tokens)
                     (2, 4, 14, 14, 32, 3), (1, 2, 16, 32, 32, 3), (3, 2, 1, 130, 32, 3), (2, 2, 3, 70, 32, 5),
                     (1, 1, 1, 2, 32, 3), (5, 70, 8, 8, 32, 3), (2, 3, 9, 22, 32, 5), (1, 2, 128, 4, 32, 3)]


@pytest.mark.parametrize("shape", ONE_KERNEL_SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_tensor_one_kernel_parity(shape):
    from paper_2211_10526_b200 import CastlingAttn, binding
    c = workloads.custom_call(*shape, "bf16", seed=700 + sum(shape))
    s = c.shape
    dev = torch.device("cuda:0")
    q, k, v, w, b = (t.to(dev) for t in (c.q, c.k, c.v, c.dw_weight, c.dw_bias))
    with CastlingAttn(ksize=s.ksize, force_path=binding.PATH_TENSOR) as attn:
        guard = torch.full((s.B * s.H * s.N * s.d + 4096,), 7.0, dtype=torch.bfloat16, device=dev)
        out = guard[2048:2048 + s.B * s.H * s.N * s.d].view(s.B, s.H, s.N, s.d)
        attn.forward(q, k, v, w, b, s.gridH, s.gridW, out=out)
        torch.cuda.synchronize()
        assert attn.device_status() == (0, 0)
        assert attn.last_path() == (binding.PATH_TENSOR, 1), "expected the single-kernel forward"
        assert bool((guard[:2048] == 7.0).all()) and bool((guard[-2048:] == 7.0).all()), "wrote outside the output"
        out_nb = attn.forward(q, k, v, w, None, s.gridH, s.gridW)
        out_again = attn.forward(q, k, v, w, b, s.gridH, s.gridW)
        torch.cuda.synchronize()
        assert attn.device_status() == (0, 0)
    assert rel_err(out, run_oracle(c)) <= TOL["bf16"]
    assert rel_err(out_nb, run_oracle(c, bias=False)) <= TOL["bf16"]
    assert torch.equal(out, out_again), "two runs differ bitwise"


def test_tensor_one_kernel_term_isolation():
    """Each term of Eq. 9 alone, on the single-kernel forward (240 tokens: two tiles, the second ragged)."""
    from paper_2211_10526_b200 import binding
    for ks in (3, 5):
        base = lambda seed: workloads.custom_call(3, 2, 12, 20, 64, ks, "bf16", seed=seed)
        c = base(621)  # linear term alone
        v = c.v.float(); c.v = (v - v.mean(dim=2, keepdim=True)).to(torch.bfloat16)
        c.dw_weight.zero_(); c.dw_bias.zero_()
        check(c, force_path=binding.PATH_TENSOR)
        c = base(622)  # 1/2 sum (constant V)
        c.v[:] = c.v[:, :, :1, :].clone()
        c.dw_weight.zero_(); c.dw_bias.zero_()
        check(c, force_path=binding.PATH_TENSOR)
        c = base(623)  # convolution alone
        v = c.v.float(); c.v = (v - v.mean(dim=2, keepdim=True)).to(torch.bfloat16)
        c.dw_weight = (c.dw_weight.float() * 30).to(torch.bfloat16)
        c.k.zero_()
        check(c, force_path=binding.PATH_TENSOR)
        c = base(624)  # zero rows
        c.q[0, 0, 5] = 0; c.k[1, 1, 17] = 0; c.k[2, 0, 239] = 0
        check(c, force_path=binding.PATH_TENSOR)
        c = workloads.custom_call(2, 2, 10, 10, 64, ks, "bf16", seed=625, qk_lognormal_sigma=3.0)  # row scales
        check(c, force_path=binding.PATH_TENSOR)


def test_tensor_path_term_isolation_head_width_32():
    from paper_2211_10526_b200 import binding
    base = lambda seed, ks: workloads.custom_call(2, 2, 24, 20, 32, ks, "bf16", seed=seed)
    for ks in (3, 5):
        c = base(611, ks)   # linear term alone
        v = c.v.float(); c.v = (v - v.mean(dim=2, keepdim=True)).to(torch.bfloat16)
        c.dw_weight.zero_(); c.dw_bias.zero_()
        check(c, force_path=binding.PATH_TENSOR)
        c = base(612, ks)   # 1/2 sum (constant V)
        c.v[:] = c.v[:, :, :1, :].clone()
        c.dw_weight.zero_(); c.dw_bias.zero_()
        check(c, force_path=binding.PATH_TENSOR)
        c = base(613, ks)   # convolution alone
        v = c.v.float(); c.v = (v - v.mean(dim=2, keepdim=True)).to(torch.bfloat16)
        c.dw_weight = (c.dw_weight.float() * 30).to(torch.bfloat16)
        c.k.zero_()
        check(c, force_path=binding.PATH_TENSOR)


def test_odd_grid_width_head_width_32_uses_cuda_cores():
    from paper_2211_10526_b200 import CastlingAttn, binding
    c = workloads.custom_call(2, 2, 7, 7, 32, 3, "bf16", seed=614)
    dev = torch.device("cuda:0")
    with CastlingAttn(ksize=3) as attn:
        attn.forward(*[t.to(dev) for t in (c.q, c.k, c.v, c.dw_weight, c.dw_bias)], 7, 7)
        torch.cuda.synchronize()
        assert attn.last_path()[0] == binding.PATH_SIMT
    check(c)


def test_tensor_path_rejects_what_it_cannot_take():
    from paper_2211_10526_b200 import CastlingAttn, binding
    c = workloads.custom_call(1, 1, 4, 4, 32, 3, "f32", seed=605)
    dev = torch.device("cuda:0")
    with CastlingAttn(ksize=3, force_path=binding.PATH_TENSOR) as attn:
        with pytest.raises(binding.CastlingError) as ei:
            attn.forward(*[t.to(dev) for t in (c.q, c.k, c.v, c.dw_weight, c.dw_bias)], 4, 4)
        assert ei.value.code == binding.ERR_UNSUPPORTED
