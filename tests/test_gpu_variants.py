"""GPU parity of the variants of the attention beyond the inference-time core, against the CPU oracle:

* rows of attention weights divided by their sums (Eq. 3's denominator on the kept kernel of Eq. 8),
* the exact angular kernel of Eq. 4-5 in place of its kept part,
* the masked softmax branch of training, Eq. 10,

on the named configurations (the quadratic variants up to 4096 tokens, the size their kernel is meant for,
and once at its limit of 16384), with the same bounds as the core: 1e-5 of the largest reference value for fp32,
2e-2 for bf16.  The mask of Eq. 10 compares a probability with a threshold; the kernel does that in fp32 and the
oracle in float64, so thresholds are placed in a gap of the oracle's probabilities wherever all of them can be
listed (then no comparison is close); elsewhere a borderline probability may fall on either side, which moves an
output by at most threshold * |v|, far inside the bf16 bound.
"""
from __future__ import annotations

import numpy as np
import pytest
import torch

import oracle
import workloads

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "bf16": 2e-2}


def gpu_forward(c, layout="head_major", prefix=0, grid=None, **variant):
    from paper_2211_10526_b200 import CastlingAttn
    s = c.shape
    gh, gw = grid if grid else (s.gridH, s.gridW)
    dev = torch.device("cuda:0")
    if layout == "head_major":
        q, k, v = (t.to(dev) for t in (c.q, c.k, c.v))
        out = torch.full_like(q, float("nan"))
    else:
        mk = lambda t: t.permute(0, 2, 1, 3).contiguous().to(dev).permute(0, 2, 1, 3)
        q, k, v = mk(c.q), mk(c.k), mk(c.v)
        out = torch.full((s.B, s.N, s.H, s.d), float("nan"), dtype=q.dtype, device=dev).permute(0, 2, 1, 3)
    with CastlingAttn(ksize=s.ksize, prefix_tokens=prefix, **variant) as attn:
        attn.forward(q, k, v, c.dw_weight.to(dev), c.dw_bias.to(dev), gh, gw, out=out)
        torch.cuda.synchronize()
        assert attn.device_status() == (0, 0)
    got = out.double().cpu().numpy()
    assert np.all(np.isfinite(got)), "an output element was never written"
    return got


def check(got, ref, dtype, what):
    scale = float(np.max(np.abs(ref)))
    err = float(np.max(np.abs(got - ref))) / scale
    assert err <= TOL[dtype], f"{what}: max-rel error {err:.3e} (largest reference value {scale:.3g})"


def gap_threshold(c, lo=0.1, hi=0.9, require=True):
    """A threshold inside the widest gap between neighbouring softmax probabilities (all planes) in the middle of
    their distribution: no probability is closer to it than half that gap.  With `require` the gap has to be
    wide against fp32 rounding (the fp32 cases, whose bound a single borderline probability would break)."""
    s = c.shape
    ps = [oracle.softmax_probs(c.q[b, h], c.k[b, h]).ravel() for b in range(s.B) for h in range(s.H)]
    p = np.sort(np.concatenate(ps))
    a, b = int(lo * p.size), int(hi * p.size)
    i = a + int(np.argmax(np.diff(p[a:b])))
    thr = 0.5 * (p[i] + p[i + 1])
    assert not require or (p[i + 1] - p[i]) / thr > 1e-5, "no usable gap"
    return float(thr)


CONFIG_CALLS = [("c1_fp32_tiny", 0), ("c2_levit_bf16", 0), ("c2_levit_bf16", 1), ("c2_levit_bf16", 2),
                ("c3_deit_base_bf16", 0), ("c4_detection_bf16", 0), ("c5_sweep_bf16", 0), ("c5_sweep_bf16", 1),
                ("c5_sweep_bf16", 2), ("c5_sweep_bf16", 3)]
IDS = [f"{n}-{i}" for n, i in CONFIG_CALLS]


@pytest.mark.parametrize("name,idx", CONFIG_CALLS, ids=IDS)
def test_row_normalised_configurations(name, idx):
    (c,) = list(workloads.iter_workload(name, only=[idx]))
    s = c.shape
    ref = oracle.forward_rownorm(c.q, c.k, c.v, c.dw_weight, c.dw_bias, s.gridH, s.gridW, s.ksize, threads=16)
    check(gpu_forward(c, normalize_rows=True), ref, s.dtype, f"{s.label()} row-normalised")


def test_row_normalised_attention_term_alone():
    """Zero filters and bias: the output is the normalised attention term, a weighted mean of V, on its own scale."""
    for dtype, shape in (("f32", (2, 3, 20, 24, 32, 3)), ("bf16", (2, 2, 48, 40, 64, 3))):
        c = workloads.custom_call(*shape, dtype, seed=8100)
        c.dw_weight.zero_(); c.dw_bias.zero_()
        s = c.shape
        ref = oracle.forward_rownorm(c.q, c.k, c.v, c.dw_weight, c.dw_bias, s.gridH, s.gridW, s.ksize, threads=8)
        check(gpu_forward(c, normalize_rows=True), ref, dtype, f"{s.label()} normalised attention term")
        # rows of weights sum to one: a constant V comes back
        c.v[:] = 1.25
        got = gpu_forward(c, normalize_rows=True)
        assert np.max(np.abs(got - 1.25)) <= (2e-6 if dtype == "f32" else 1e-2)


def test_row_normalised_with_leading_tokens_and_strides():
    c = workloads.custom_call(2, 4, 1, 2 + 9 * 10, 32, 3, "f32", seed=8101)
    ref = oracle.forward_rownorm(c.q, c.k, c.v, c.dw_weight, c.dw_bias, 9, 10, 3, prefix=2)
    check(gpu_forward(c, prefix=2, grid=(9, 10), normalize_rows=True), ref, "f32", "leading tokens")
    # bf16 with leading tokens on the tensor-core kernels: width 64, and width-32 token pairs (even number of leading tokens)
    for d, prefix, gh, gw in ((64, 1, 20, 24), (32, 2, 20, 24)):
        c = workloads.custom_call(2, 4, 1, prefix + gh * gw, d, 3, "bf16", seed=8103 + d)
        ref = oracle.forward_rownorm(c.q, c.k, c.v, c.dw_weight, c.dw_bias, gh, gw, 3, prefix=prefix)
        check(gpu_forward(c, prefix=prefix, grid=(gh, gw), normalize_rows=True, force_path=2), ref, "bf16", f"leading tokens, d={d}")
    c = workloads.custom_call(2, 4, 12, 14, 64, 5, "bf16", seed=8102)
    ref = oracle.forward_rownorm(c.q, c.k, c.v, c.dw_weight, c.dw_bias, 12, 14, 5)
    check(gpu_forward(c, layout="token_major", normalize_rows=True), ref, "bf16", "token-major")


@pytest.mark.parametrize("path", [1, 2], ids=["cuda-core", "tensor-core"])
@pytest.mark.parametrize("case", [(2, 8, 64, 64, 64, 3, "head_major"), (3, 4, 40, 56, 64, 5, "head_major"),
                                  (2, 4, 64, 64, 32, 3, "head_major"), (2, 6, 48, 64, 32, 5, "head_major"),
                                  (2, 6, 48, 64, 32, 3, "token_major")], ids=lambda t: "x".join(map(str, t)))
def test_row_normalised_on_both_kernel_families(case, path):
    """The row-sum division on the tensor-core kernels (sum of the unit key rows as one more accumulator column of the
    state contraction, q . sum k^ as one more column of the apply contraction) and on the CUDA-core kernels, for every
    packing of the tensor-core kernels; once with the filters and bias as drawn and once without them, so that the
    divided attention term is the whole output."""
    from paper_2211_10526_b200 import CastlingAttn
    *shape, layout = case
    for zero_conv in (False, True):
        c = workloads.custom_call(*shape, "bf16", seed=8150 + shape[2])
        if zero_conv:
            c.dw_weight.zero_(); c.dw_bias.zero_()
        s = c.shape
        ref = oracle.forward_rownorm(c.q, c.k, c.v, c.dw_weight, c.dw_bias, s.gridH, s.gridW, s.ksize, threads=16)
        dev = torch.device("cuda:0")
        if layout == "head_major":
            q, k, v = (t.to(dev) for t in (c.q, c.k, c.v))
            out = torch.full_like(q, float("nan"))
        else:
            mk = lambda t: t.permute(0, 2, 1, 3).contiguous().to(dev).permute(0, 2, 1, 3)
            q, k, v = mk(c.q), mk(c.k), mk(c.v)
            out = torch.full((s.B, s.N, s.H, s.d), float("nan"), dtype=q.dtype, device=dev).permute(0, 2, 1, 3)
        with CastlingAttn(ksize=s.ksize, normalize_rows=True, force_path=path) as attn:
            attn.forward(q, k, v, c.dw_weight.to(dev), c.dw_bias.to(dev), s.gridH, s.gridW, out=out)
            torch.cuda.synchronize()
            assert attn.device_status() == (0, 0)
            assert attn.last_path()[0] == path
        got = out.double().cpu().numpy()
        assert np.all(np.isfinite(got))
        check(got, ref, "bf16", f"{s.label()} {layout} path {path} zero_conv={zero_conv}")


QUAD_CALLS = [("c1_fp32_tiny", 0), ("c2_levit_bf16", 0), ("c2_levit_bf16", 1), ("c2_levit_bf16", 2),
              ("c3_deit_base_bf16", 0), ("c4_detection_bf16", 0), ("c5_sweep_bf16", 0), ("c5_sweep_bf16", 1)]
QUAD_IDS = [f"{n}-{i}" for n, i in QUAD_CALLS]


@pytest.mark.parametrize("name,idx", QUAD_CALLS, ids=QUAD_IDS)
def test_exact_angular_kernel_configurations(name, idx):
    (c,) = list(workloads.iter_workload(name, only=[idx]))
    s = c.shape
    ref = oracle.forward_matrix(c.q, c.k, c.v, c.dw_weight, c.dw_bias, s.gridH, s.gridW, s.ksize,
                                kernel=oracle.KERNEL_EXACT, threads=16)
    check(gpu_forward(c, exact_kernel=True), ref, s.dtype, f"{s.label()} exact kernel")


@pytest.mark.parametrize("path", [1, 2], ids=["cuda-core", "tensor-core"])
@pytest.mark.parametrize("case", [(2, 3, 16, 16, 64, 3, "head_major"), (1, 4, 25, 31, 64, 5, "head_major"),
                                  (2, 2, 40, 48, 64, 3, "token_major"), (1, 2, 9, 11, 64, 3, "head_major")],
                         ids=lambda t: "x".join(map(str, t)))
def test_exact_kernel_on_both_kernel_families(case, path):
    """The exact angular kernel on the tensor cores (cosines and weighted sums as UMMAs, weights through shared
    memory) and on the CUDA cores: whole tiles, a ragged last tile of queries and keys, a plane smaller than a tile,
    both filter sizes, a strided layout; with the filters as drawn, and without them, so that the attention term is
    the whole output."""
    from paper_2211_10526_b200 import CastlingAttn
    *shape, layout = case
    for zero_conv in (False, True):
        c = workloads.custom_call(*shape, "bf16", seed=8300 + shape[2])
        if zero_conv:
            c.dw_weight.zero_(); c.dw_bias.zero_()
        s = c.shape
        ref = oracle.forward_matrix(c.q, c.k, c.v, c.dw_weight, c.dw_bias, s.gridH, s.gridW, s.ksize,
                                    kernel=oracle.KERNEL_EXACT, threads=16)
        dev = torch.device("cuda:0")
        if layout == "head_major":
            q, k, v = (t.to(dev) for t in (c.q, c.k, c.v))
            out = torch.full_like(q, float("nan"))
        else:
            mk = lambda t: t.permute(0, 2, 1, 3).contiguous().to(dev).permute(0, 2, 1, 3)
            q, k, v = mk(c.q), mk(c.k), mk(c.v)
            out = torch.full((s.B, s.N, s.H, s.d), float("nan"), dtype=q.dtype, device=dev).permute(0, 2, 1, 3)
        with CastlingAttn(ksize=s.ksize, exact_kernel=True, force_path=path) as attn:
            attn.forward(q, k, v, c.dw_weight.to(dev), c.dw_bias.to(dev), s.gridH, s.gridW, out=out)
            torch.cuda.synchronize()
            assert attn.device_status() == (0, 0)
            assert attn.last_path() == (path, 1)
        got = out.double().cpu().numpy()
        assert np.all(np.isfinite(got))
        check(got, ref, "bf16", f"{s.label()} {layout} path {path} zero_conv={zero_conv}")


@pytest.mark.parametrize("path", [1, 2], ids=["cuda-core", "tensor-core"])
@pytest.mark.parametrize("exact", [False, True], ids=["kept-kernel", "exact-kernel"])
@pytest.mark.parametrize("case", [(2, 3, 2, 3, 64, 3), (2, 3, 4, 4, 64, 3), (1, 4, 5, 6, 64, 5), (2, 3, 16, 16, 64, 3),
                                  (1, 4, 25, 31, 64, 5)], ids=lambda t: "x".join(map(str, t)))
def test_sparse_branch_on_both_kernel_families(case, exact, path):
    """The masked softmax branch on the tensor cores (a first sweep over the keys for the denominators, the masked
    probabilities added to the weights in the second) and on the CUDA cores, on top of either base kernel.  The
    threshold sits in a gap of the oracle's probabilities; with bf16 cosines a probability next to it may still fall
    on the other side, which moves an output by at most the threshold times |v|."""
    from paper_2211_10526_b200 import CastlingAttn
    c = workloads.custom_call(*case, "bf16", seed=8400 + case[2])
    s = c.shape
    thr = gap_threshold(c, lo=0.0, hi=0.2, require=False)   # most probabilities pass
    ref = oracle.forward_matrix(c.q, c.k, c.v, c.dw_weight, c.dw_bias, s.gridH, s.gridW, s.ksize,
                                kernel=oracle.KERNEL_EXACT if exact else oracle.KERNEL_LINEAR, sparse_eps=thr, threads=16)
    base = oracle.forward_matrix(c.q, c.k, c.v, c.dw_weight, c.dw_bias, s.gridH, s.gridW, s.ksize,
                                 kernel=oracle.KERNEL_EXACT if exact else oracle.KERNEL_LINEAR, threads=16)
    # With unit rows a probability is about 1/N, so the branch is a small term of long sequences (the bound on the whole
    # output could hide it there); on the planes of a few tokens it is several times the bound, and a defect in the
    # denominators or the mask fails the comparison below.
    if s.N <= 32:
        assert np.max(np.abs(ref - base)) > 2.5 * TOL["bf16"] * np.max(np.abs(ref)), "the branch is too small to be seen"
    dev = torch.device("cuda:0")
    q, k, v = (t.to(dev) for t in (c.q, c.k, c.v))
    out = torch.full_like(q, float("nan"))
    with CastlingAttn(ksize=s.ksize, exact_kernel=exact, sparse_eps=thr, force_path=path) as attn:
        attn.forward(q, k, v, c.dw_weight.to(dev), c.dw_bias.to(dev), s.gridH, s.gridW, out=out)
        torch.cuda.synchronize()
        assert attn.device_status() == (0, 0)
        assert attn.last_path() == (path, 1)
    got = out.double().cpu().numpy()
    assert np.all(np.isfinite(got))
    check(got, ref, "bf16", f"{s.label()} exact={exact} path {path}")


@pytest.mark.parametrize("name,idx", QUAD_CALLS, ids=QUAD_IDS)
def test_sparse_branch_configurations(name, idx):
    (c,) = list(workloads.iter_workload(name, only=[idx]))
    s = c.shape
    # a threshold that keeps about half of the probabilities (the paper's 0.02 masks everything on such inputs:
    # with unit rows no probability exceeds e^2 / N); in a gap of all probabilities where they can be listed
    thr = gap_threshold(c, require=(s.dtype == "f32")) if s.B * s.H * s.N * s.N <= 4_000_000 else 1.0 / s.N
    ref = oracle.forward_matrix(c.q, c.k, c.v, c.dw_weight, c.dw_bias, s.gridH, s.gridW, s.ksize, sparse_eps=thr, threads=16)
    check(gpu_forward(c, sparse_eps=thr), ref, s.dtype, f"{s.label()} masked softmax branch, threshold {thr:.3e}")


def test_castling_all_zero_mask_is_the_inference_core():
    """With the paper's threshold the mask is empty on these inputs, and the explicit-weights kernel then computes
    the inference-time core: same result as the oracle's linear form, and as the linear kernels to rounding."""
    (c,) = list(workloads.iter_workload("c1_fp32_tiny", only=[0]))
    s = c.shape
    ref = oracle.forward(c.q, c.k, c.v, c.dw_weight, c.dw_bias, s.gridH, s.gridW, s.ksize)
    assert np.array_equal(oracle.forward_matrix(c.q, c.k, c.v, c.dw_weight, c.dw_bias, s.gridH, s.gridW, s.ksize, sparse_eps=0.02),
                          oracle.forward_matrix(c.q, c.k, c.v, c.dw_weight, c.dw_bias, s.gridH, s.gridW, s.ksize))
    quad = gpu_forward(c, sparse_eps=0.02)
    check(quad, ref, "f32", "empty mask")
    check(quad, gpu_forward(c), "f32", "explicit weights against the linear kernels")


def test_variant_terms_alone_fp32():
    """The masked softmax term and the high-order residual of the exact kernel, each as the difference of two fp32
    runs, on its own scale; thresholds in a gap of the probabilities."""
    c = workloads.custom_call(2, 3, 16, 16, 32, 3, "f32", seed=8103)
    s = c.shape
    core = gpu_forward(c, sparse_eps=2.0)      # explicit weights, empty mask
    thr = gap_threshold(c)
    o = lambda **kw: oracle.forward_matrix(c.q, c.k, c.v, c.dw_weight, c.dw_bias, s.gridH, s.gridW, s.ksize, threads=6, **kw)
    base = o()
    for what, got, ref in (("masked softmax term", gpu_forward(c, sparse_eps=thr) - core, o(sparse_eps=thr) - base),
                           ("plain softmax term", gpu_forward(c, sparse_eps=-1.0) - core, o(sparse_eps=-1.0) - base),
                           ("high-order residual", gpu_forward(c, exact_kernel=True) - core, o(kernel=oracle.KERNEL_EXACT) - base)):
        scale = float(np.max(np.abs(ref)))
        err = float(np.max(np.abs(got - ref)))
        # each run is good to 1e-5 of its own largest value, which is larger than this term's
        assert err <= 2e-5 * float(np.max(np.abs(base))), f"{what}: {err:.3e} on a term of size {scale:.3g}"
        assert err <= 5e-3 * scale, f"{what}: {err:.3e} on a term of size {scale:.3g}"


def test_all_variants_together_and_limits():
    from paper_2211_10526_b200 import CastlingAttn, binding as b
    c = workloads.custom_call(2, 2, 16, 20, 48, 5, "f32", seed=8104)
    s = c.shape
    thr = gap_threshold(c)
    ref = oracle.forward_matrix(c.q, c.k, c.v, c.dw_weight, c.dw_bias, s.gridH, s.gridW, s.ksize, kernel=oracle.KERNEL_EXACT,
                                rownorm=True, sparse_eps=thr)
    check(gpu_forward(c, exact_kernel=True, normalize_rows=True, sparse_eps=thr), ref, "f32", "all variants")
    ref = oracle.forward_matrix(c.q, c.k, c.v, c.dw_weight, c.dw_bias, s.gridH, s.gridW, s.ksize, rownorm=True, sparse_eps=thr)
    check(gpu_forward(c, normalize_rows=True, sparse_eps=thr), ref, "f32", "row sums and mask")
    # leading tokens and the quadratic variants do not combine; nor do more than 16384 tokens
    with pytest.raises(b.CastlingError):
        CastlingAttn(prefix_tokens=1, exact_kernel=True)
    dev = torch.device("cuda:0")
    with CastlingAttn(exact_kernel=True) as attn:
        t = torch.zeros(1, 1, 129 * 128, 32, dtype=torch.bfloat16, device=dev)
        w, bias = torch.zeros(32, 3, 3, dtype=torch.bfloat16, device=dev), torch.zeros(32, dtype=torch.bfloat16, device=dev)
        with pytest.raises(b.CastlingError):
            attn.forward(t, t, t, w, bias, 129, 128, out=torch.empty_like(t))


def test_exact_kernel_at_the_token_limit():
    c = workloads.custom_call(1, 2, 128, 128, 32, 3, "bf16", seed=8105)
    s = c.shape
    ref = oracle.forward_matrix(c.q, c.k, c.v, c.dw_weight, c.dw_bias, s.gridH, s.gridW, s.ksize, kernel=oracle.KERNEL_EXACT, threads=2)
    check(gpu_forward(c, exact_kernel=True), ref, "bf16", "16384 tokens")
    # the same limit on the tensor-core kernel (width-64 heads): 128 query tiles x 128 key tiles for one plane
    c = workloads.custom_call(1, 1, 128, 128, 64, 3, "bf16", seed=8106)
    s = c.shape
    ref = oracle.forward_matrix(c.q, c.k, c.v, c.dw_weight, c.dw_bias, s.gridH, s.gridW, s.ksize, kernel=oracle.KERNEL_EXACT, threads=2)
    check(gpu_forward(c, exact_kernel=True, force_path=2), ref, "bf16", "16384 tokens, tensor cores")
