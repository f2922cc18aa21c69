"""Pins for the CPU oracle: things the paper and the mathematics fix.

Each ``pin_*`` function takes a loaded oracle library and raises AssertionError
when that build of the oracle violates a fact that does not depend on the
oracle itself: values worked by hand from Eq. 8-9, the arcsin series of Eq. 8,
the range and special values of Eq. 5-6, brute force over the explicit N x N
similarity matrix, closed forms (constant V, equal keys, d = 1, zero rows),
filters whose convolution is known (delta, shift, box, zero), an explicit
M_DW matrix, a library convolution, scale invariance and linearity.

``test_pins_catch_planted_mistakes`` then rebuilds the oracle with one planted
mistake at a time (a dropped term, a wrong sign or index, a transposed
operand, a missing normalisation ...) and requires that some pin fails for
every one of them.
"""
from __future__ import annotations

import math
import os
import subprocess
from fractions import Fraction

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
PI = math.pi


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as fh:
        return [ln.split() for ln in fh if ln.strip() and not ln.lstrip().startswith("#")]


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def _problem(B, H, gh, gw, d, ks, seed, bias=True):
    rng = np.random.default_rng(seed)
    q, k, v = (rng.standard_normal((B, H, gh * gw, d)) for _ in range(3))
    w = 0.3 * rng.standard_normal((H * d, ks, ks))
    b = 0.3 * rng.standard_normal((H * d,)) if bias else None
    return q, k, v, w, b


def _zero_filter(H, d, ks):
    return np.zeros((H * d, ks, ks)), np.zeros((H * d,))


def _unit(x):
    return x / np.linalg.norm(x, axis=-1, keepdims=True)


def _close(a, b, tol=1e-12):
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    scale = max(1.0, float(np.max(np.abs(b))))
    err = float(np.max(np.abs(a - b)))
    assert np.all(np.isfinite(a)), "non-finite oracle output"
    assert err <= tol * scale, f"max abs diff {err:.3e} over scale {scale:.3e}"


# --------------------------------------------------------------------------
# golden fixtures
# --------------------------------------------------------------------------
def pin_worked_example(lib):
    """Hand-worked 1 x 2 grid instance of Eq. 8-9 (tests/golden/worked_example_1x2.txt)."""
    q = np.array([[3.0, 4.0], [0.0, 2.0]]).reshape(1, 1, 2, 2)
    k = np.array([[1.0, 0.0], [0.0, -5.0]]).reshape(1, 1, 2, 2)
    v = np.array([[1.0, 2.0], [3.0, 4.0]]).reshape(1, 1, 2, 2)
    w = np.array([[[9, 9, 9], [0.5, 1, 2], [9, 9, 9]], [[7, 7, 7], [-1, 0, 1], [7, 7, 7]]], dtype=np.float64)
    b = np.array([0.25, -0.5])
    expect = np.zeros((2, 2))
    for t, c, a, bb in _rows("worked_example_1x2.txt"):
        expect[int(t), int(c)] = float(a) + float(bb) / PI
    for fn in (oracle.forward, oracle.forward_bruteforce):
        out = fn(q, k, v, w, b, 1, 2, 3, lib=lib)
        _close(out[0, 0], expect, 1e-14)


def pin_series_coefficients(lib):
    """Eq. 8 coefficients against the hand-evaluated fractions."""
    for k, num, den in _rows("eq8_series_coefficients.txt"):
        got = lib.castling_oracle_angular_series_coeff(int(k))
        assert abs(got - float(Fraction(int(num), int(den)))) < 1e-15, (k, got)


def pin_angular_values(lib):
    """Eq. 4-6 special values of the exact kernel."""
    for x, num, den in _rows("angular_kernel_values.txt"):
        got = lib.castling_oracle_angular_exact(float(x))
        assert abs(got - int(num) / int(den)) < 1e-15, (x, got)


# --------------------------------------------------------------------------
# Eq. 8: series identities
# --------------------------------------------------------------------------
def pin_series_properties(lib):
    exact = lib.castling_oracle_angular_exact
    series = lib.castling_oracle_angular_series
    xs = np.linspace(-1.0, 1.0, 41)
    for x in xs:
        # first line of Eq. 8: 1 - acos(x)/pi == 1/2 + asin(x)/pi
        assert abs(exact(x) - (0.5 + math.asin(x) / PI)) < 1e-15
        # kept part is exactly 1/2 + x/pi
        assert abs(series(x, 0) - (0.5 + x / PI)) < 1e-16
        # range of Eq. 5
        assert -1e-16 <= exact(x) <= 1.0 + 1e-16
        # residual is odd in x
        r_pos = exact(x) - series(x, 0)
        r_neg = exact(-x) - series(-x, 0)
        assert abs(r_pos + r_neg) < 1e-15
    # residual at the ends is +-(1/2 - 1/pi)
    assert abs((exact(1.0) - series(1.0, 0)) - (0.5 - 1 / PI)) < 1e-15
    assert abs((exact(-1.0) - series(-1.0, 0)) + (0.5 - 1 / PI)) < 1e-15
    # partial sums converge to the exact kernel inside the unit interval
    for x in (-0.9, -0.5, 0.1, 0.7):
        prev = abs(exact(x) - series(x, 0))
        for kmax in (2, 8, 40, 200):
            cur = abs(exact(x) - series(x, kmax))
            assert cur <= prev + 1e-16
            prev = cur
        assert prev < 1e-12
    # slope at zero is 1/pi
    h = 1e-6
    assert abs((exact(h) - exact(-h)) / (2 * h) - 1 / PI) < 1e-9


# --------------------------------------------------------------------------
# Eq. 8-9: explicit similarity matrix against the re-associated form
# --------------------------------------------------------------------------
def pin_bruteforce_equals_linear(lib):
    for (B, H, gh, gw, d, ks, seed) in [(2, 3, 3, 4, 5, 3, 11), (1, 2, 5, 5, 8, 5, 12), (1, 1, 1, 1, 3, 3, 13),
                                        (1, 2, 2, 7, 4, 7, 14), (2, 4, 14, 14, 32, 3, 15)]:
        q, k, v, w, b = _problem(B, H, gh, gw, d, ks, seed)
        lin = oracle.forward(q, k, v, w, b, gh, gw, ks, lib=lib)
        bf = oracle.forward_bruteforce(q, k, v, w, b, gh, gw, ks, lib=lib)
        _close(lin, bf, 1e-12)


def pin_similarity_matrix(lib):
    """Range and diagonal of 1/2 + cos/pi, and A = Sim V with numpy doing the product."""
    N, d = 9, 6
    q, k, v = _rand((N, d), 21), _rand((N, d), 22), _rand((N, d), 23)
    sim = oracle.similarity(q, k, lib=lib)
    assert sim.min() >= 0.5 - 1 / PI - 1e-15 and sim.max() <= 0.5 + 1 / PI + 1e-15
    cos = _unit(q) @ _unit(k).T  # cosines by numpy, Eq. 4
    _close(sim, 0.5 + cos / PI, 1e-14)
    # Sim(x, x): the linear part gives 1/2 + 1/pi on the diagonal when k = q
    _close(np.diag(oracle.similarity(q, q, lib=lib)), np.full(N, 0.5 + 1 / PI), 1e-14)
    wz, bz = _zero_filter(1, d, 3)
    out = oracle.forward(q[None, None], k[None, None], v[None, None], wz, bz, 3, 3, 3, lib=lib)
    _close(out[0, 0], sim @ v, 1e-13)


# --------------------------------------------------------------------------
# closed forms
# --------------------------------------------------------------------------
def _box_counts(gh, gw, ks):
    r = (ks - 1) // 2
    cnt = np.zeros((gh, gw))
    for y in range(gh):
        for x in range(gw):
            cnt[y, x] = (min(gh - 1, y + r) - max(0, y - r) + 1) * (min(gw - 1, x + r) - max(0, x - r) + 1)
    return cnt


def pin_constant_v(lib):
    """v_j = c for all j: A_t = c (N/2 + q^_t . sum_j k^_j / pi); the 1/2 term is exactly N c / 2."""
    B, H, gh, gw, d, ks = 2, 2, 4, 5, 6, 3
    N = gh * gw
    q, k, _, _, _ = _problem(B, H, gh, gw, d, ks, 31)
    c = _rand((B, H, 1, d), 32)
    v = np.broadcast_to(c, (B, H, N, d)).copy()
    wz, bz = _zero_filter(H, d, ks)
    out = oracle.forward(q, k, v, wz, bz, gh, gw, ks, lib=lib)
    ksum = _unit(k).sum(axis=2, keepdims=True)                     # [B,H,1,d]
    coef = N / 2.0 + (_unit(q) * ksum).sum(-1, keepdims=True) / PI  # [B,H,N,1]
    _close(out, coef * c, 1e-13)
    # with q orthogonal to sum k^ only N c / 2 is left
    q_orth = q - (q * ksum).sum(-1, keepdims=True) / (ksum * ksum).sum(-1, keepdims=True) * ksum
    out = oracle.forward(q_orth, k, v, wz, bz, gh, gw, ks, lib=lib)
    _close(out, np.broadcast_to(N / 2.0 * c, out.shape), 1e-12)


def pin_equal_keys(lib):
    """All k^_j equal to one unit vector u: A_t = (1/2 + q^_t . u / pi) sum_j v_j."""
    B, H, gh, gw, d, ks = 1, 2, 3, 3, 5, 3
    N = gh * gw
    q, _, v, _, _ = _problem(B, H, gh, gw, d, ks, 41)
    u = _unit(_rand((B, H, 1, d), 42))
    scales = np.abs(_rand((B, H, N, 1), 43)) + 0.1
    k = u * scales
    wz, bz = _zero_filter(H, d, ks)
    out = oracle.forward(q, k, v, wz, bz, gh, gw, ks, lib=lib)
    coef = 0.5 + (_unit(q) * u).sum(-1, keepdims=True) / PI
    _close(out, coef * v.sum(axis=2, keepdims=True), 1e-13)


def pin_d_equals_one(lib):
    """d = 1: unit rows are signs, every similarity is 1/2 +- 1/pi."""
    gh, gw = 3, 4
    N = gh * gw
    q, k, v = _rand((1, 1, N, 1), 51), _rand((1, 1, N, 1), 52), _rand((1, 1, N, 1), 53)
    wz, bz = _zero_filter(1, 1, 3)
    out = oracle.forward(q, k, v, wz, bz, gh, gw, 3, lib=lib)
    sgn = np.sign(q[0, 0]) @ np.sign(k[0, 0]).T
    _close(out[0, 0], (0.5 + sgn / PI) @ v[0, 0], 1e-14)


def pin_zero_rows(lib):
    """A zero query or key has no direction: its cosine is taken as 0, similarity 1/2."""
    gh, gw, d = 2, 3, 4
    N = gh * gw
    q, k, v, _, _ = _problem(1, 1, gh, gw, d, 3, 61)
    wz, bz = _zero_filter(1, d, 3)
    q[0, 0, 2] = 0.0
    k[0, 0, 4] = 0.0
    out = oracle.forward(q, k, v, wz, bz, gh, gw, 3, lib=lib)
    assert np.all(np.isfinite(out))
    _close(out[0, 0, 2], 0.5 * v[0, 0].sum(axis=0), 1e-14)
    cos = np.zeros((N, N))
    qh, kh = q[0, 0].copy(), k[0, 0].copy()
    for t in range(N):
        for j in range(N):
            nq, nk = np.linalg.norm(qh[t]), np.linalg.norm(kh[j])
            cos[t, j] = 0.0 if nq == 0 or nk == 0 else qh[t] @ kh[j] / (nq * nk)
    _close(out[0, 0], (0.5 + cos / PI) @ v[0, 0], 1e-14)


# --------------------------------------------------------------------------
# the depthwise convolution branch (Eq. 9, M_DW V)
# --------------------------------------------------------------------------
def _attention_only(lib, q, k, v, gh, gw, ks):
    H, d = q.shape[1], q.shape[3]
    wz, bz = _zero_filter(H, d, ks)
    return oracle.forward(q, k, v, wz, bz, gh, gw, ks, lib=lib)


def pin_conv_known_filters(lib):
    B, H, gh, gw, d = 2, 2, 4, 5, 3
    for ks in (3, 5):
        r = (ks - 1) // 2
        q, k, v, _, b = _problem(B, H, gh, gw, d, ks, 70 + ks)
        att = _attention_only(lib, q, k, v, gh, gw, ks)
        vg = v.reshape(B, H, gh, gw, d)
        zeros_b = np.zeros(H * d)
        # delta filter: identity
        w = np.zeros((H * d, ks, ks)); w[:, r, r] = 1.0
        out = oracle.forward(q, k, v, w, zeros_b, gh, gw, ks, lib=lib)
        _close(out - att, v, 1e-13)
        # bias = None behaves as zero bias
        out_nb = oracle.forward(q, k, v, w, None, gh, gw, ks, lib=lib)
        _close(out_nb, out, 0.0)
        # zero filter: the bias alone, per head-channel h*d + j
        w0 = np.zeros((H * d, ks, ks))
        out = oracle.forward(q, k, v, w0, b, gh, gw, ks, lib=lib)
        _close(out - att, np.broadcast_to(b.reshape(1, H, 1, d), v.shape), 1e-13)
        # one-hot off-centre taps: shifted V with zero fill (cross-correlation orientation)
        for (ty, tx) in [(r, r + 1), (r - 1, r), (0, ks - 1), (ks - 1, 0)]:
            dy, dx = ty - r, tx - r
            w1 = np.zeros((H * d, ks, ks)); w1[:, ty, tx] = 1.0
            shifted = np.zeros_like(vg)
            for y in range(gh):
                for x in range(gw):
                    if 0 <= y + dy < gh and 0 <= x + dx < gw:
                        shifted[:, :, y, x] = vg[:, :, y + dy, x + dx]
            out = oracle.forward(q, k, v, w1, zeros_b, gh, gw, ks, lib=lib)
            _close(out - att, shifted.reshape(v.shape), 1e-13)
        # all-ones filter on all-ones V counts the in-grid neighbours (9 / 6 / 4 at 3x3)
        ones_v = np.ones_like(v)
        wb = np.ones((H * d, ks, ks))
        att1 = _attention_only(lib, q, k, ones_v, gh, gw, ks)
        out = oracle.forward(q, k, ones_v, wb, zeros_b, gh, gw, ks, lib=lib)
        cnt = _box_counts(gh, gw, ks).reshape(1, 1, gh * gw, 1)
        _close(out - att1, np.broadcast_to(cnt, v.shape), 1e-12)
    assert _box_counts(4, 5, 3)[0, 0] == 4 and _box_counts(4, 5, 3)[0, 2] == 6 and _box_counts(4, 5, 3)[1, 1] == 9


def pin_conv_head_channel_mapping(lib):
    """One filter per head-channel: a delta in head 1 channel 2 only touches that channel."""
    B, H, gh, gw, d, ks = 1, 3, 3, 3, 4, 3
    q, k, v, _, _ = _problem(B, H, gh, gw, d, ks, 81)
    att = _attention_only(lib, q, k, v, gh, gw, ks)
    w = np.zeros((H * d, ks, ks)); w[1 * d + 2, 1, 1] = 2.0
    out = oracle.forward(q, k, v, w, np.zeros(H * d), gh, gw, ks, lib=lib)
    expect = np.zeros_like(v); expect[:, 1, :, 2] = 2.0 * v[:, 1, :, 2]
    _close(out - att, expect, 1e-13)


def pin_conv_matrix_form(lib):
    """M_DW built explicitly (N x N per channel) on small grids: M_DW V equals the branch."""
    for (gh, gw, ks, seed) in [(4, 4, 3, 91), (5, 5, 5, 92), (4, 4, 5, 93), (2, 6, 7, 94)]:
        H, d, r, N = 2, 3, (ks - 1) // 2, gh * gw
        q, k, v, w, b = _problem(1, H, gh, gw, d, ks, seed)
        att = _attention_only(lib, q, k, v, gh, gw, ks)
        out = oracle.forward(q, k, v, w, b, gh, gw, ks, lib=lib)
        expect = np.zeros_like(v)
        for h in range(H):
            for j in range(d):
                M = np.zeros((N, N))
                for y in range(gh):
                    for x in range(gw):
                        for ty in range(ks):
                            for tx in range(ks):
                                yy, xx = y + ty - r, x + tx - r
                                if 0 <= yy < gh and 0 <= xx < gw:
                                    M[y * gw + x, yy * gw + xx] += w[h * d + j, ty, tx]
                expect[0, h, :, j] = M @ v[0, h, :, j] + b[h * d + j]
        _close(out - att, expect, 1e-13)


def pin_conv_library_routine(lib):
    """The branch is a grouped 2-D cross-correlation: compare with torch's conv2d (groups = channels)."""
    import torch
    import torch.nn.functional as F
    B, H, gh, gw, d, ks = 2, 3, 6, 5, 4, 3
    for ks in (3, 5):
        q, k, v, w, b = _problem(B, H, gh, gw, d, ks, 95 + ks)
        att = _attention_only(lib, q, k, v, gh, gw, ks)
        out = oracle.forward(q, k, v, w, b, gh, gw, ks, lib=lib)
        x = torch.from_numpy(v).reshape(B, H, gh, gw, d).permute(0, 1, 4, 2, 3).reshape(B, H * d, gh, gw)
        y = F.conv2d(x, torch.from_numpy(w).unsqueeze(1), torch.from_numpy(b), padding=(ks - 1) // 2, groups=H * d)
        y = y.reshape(B, H, d, gh, gw).permute(0, 1, 3, 4, 2).reshape(B, H, gh * gw, d).numpy()
        _close(out - att, y, 1e-13)


# --------------------------------------------------------------------------
# invariances
# --------------------------------------------------------------------------
def pin_scale_invariance(lib):
    """Positive per-token rescaling of q or k changes nothing (unit rows)."""
    B, H, gh, gw, d, ks = 1, 2, 3, 4, 5, 3
    q, k, v, w, b = _problem(B, H, gh, gw, d, ks, 101)
    ref = oracle.forward(q, k, v, w, b, gh, gw, ks, lib=lib)
    sq = np.exp(_rand((B, H, gh * gw, 1), 102))
    sk = np.exp(2 * _rand((B, H, gh * gw, 1), 103))
    _close(oracle.forward(q * sq, k * sk, v, w, b, gh, gw, ks, lib=lib), ref, 1e-12)


def pin_linearity_and_symmetry(lib):
    B, H, gh, gw, d, ks = 1, 2, 3, 3, 4, 3
    q, k, v, w, b = _problem(B, H, gh, gw, d, ks, 111)
    v2 = _rand(v.shape, 112)
    zb = np.zeros_like(b)
    f = lambda qq, kk, vv, ww, bb: oracle.forward(qq, kk, vv, ww, bb, gh, gw, ks, lib=lib)
    # linear in V (bias off)
    _close(f(q, k, 2.0 * v - 3.0 * v2, w, zb), 2.0 * f(q, k, v, w, zb) - 3.0 * f(q, k, v2, w, zb), 1e-12)
    # affine in (w, bias)
    w2, b2 = 0.3 * _rand(w.shape, 113), 0.3 * _rand(b.shape, 114)
    att = _attention_only(lib, q, k, v, gh, gw, ks)
    _close(f(q, k, v, w + w2, b + b2) - att, (f(q, k, v, w, b) - att) + (f(q, k, v, w2, b2) - att), 1e-12)
    # q -> -q flips only the linear term: the sum of the two outputs is sum_j v_j (+ 2 conv)
    wz, bz = _zero_filter(H, d, ks)
    s = f(q, k, v, wz, bz) + f(-q, k, v, wz, bz)
    _close(s, np.broadcast_to(v.sum(axis=2, keepdims=True), v.shape), 1e-12)
    # permuting the (k_j, v_j) pairs jointly leaves the attention part unchanged
    perm = np.random.default_rng(115).permutation(gh * gw)
    _close(f(q, k[:, :, perm], v[:, :, perm], wz, bz), f(q, k, v, wz, bz), 1e-12)
    # heads and batches are independent: evaluating one (b, h) alone gives the same slice
    q3, k3, v3, w3, b3 = _problem(2, 3, gh, gw, d, ks, 116)
    full = oracle.forward(q3, k3, v3, w3, b3, gh, gw, ks, lib=lib)
    one = oracle.forward(q3[1:2, 2:3], k3[1:2, 2:3], v3[1:2, 2:3], w3[2 * d:3 * d], b3[2 * d:3 * d], gh, gw, ks, lib=lib)
    _close(one[0, 0], full[1, 2], 1e-13)


def pin_threads_agree(lib):
    q, k, v, w, b = _problem(2, 3, 3, 3, 4, 3, 121)
    a = oracle.forward(q, k, v, w, b, 3, 3, 3, threads=1, lib=lib)
    c = oracle.forward(q, k, v, w, b, 3, 3, 3, threads=4, lib=lib)
    _close(a, c, 0.0)


def pin_prefix_tokens(lib):
    """Off-grid leading tokens (class tokens): attention terms over all tokens, convolution on the grid only.

    Pinned against the plain forward (itself pinned above) and a library convolution: with the filter bank
    zeroed the result is the plain forward of the same sequence on a 1 x T grid (the attention terms do not
    know about the grid); the difference the filters make is scipy's 2-D correlation of the grid tokens of V
    plus the bias, and exactly zero on the prefix rows."""
    from scipy.signal import correlate2d
    B, H, P, gh, gw, d, ks = 2, 2, 2, 3, 4, 5, 3
    T = P + gh * gw
    rng = np.random.default_rng(131)
    q, k, v = (rng.standard_normal((B, H, T, d)) for _ in range(3))
    w = 0.3 * rng.standard_normal((H * d, ks, ks)); b = 0.3 * rng.standard_normal((H * d,))
    wz, bz = _zero_filter(H, d, ks)
    att = oracle.forward(q, k, v, wz, bz, gh, gw, ks, lib=lib, prefix=P)
    _close(att, oracle.forward(q, k, v, wz, bz, 1, T, ks, lib=lib), 1e-12)
    full = oracle.forward(q, k, v, w, b, gh, gw, ks, lib=lib, prefix=P)
    diff = full - att
    assert float(np.max(np.abs(diff[:, :, :P]))) == 0.0, "the convolution touched a prefix row"
    for bb in range(B):
        for h in range(H):
            for j in range(d):
                img = v[bb, h, P:, j].reshape(gh, gw)
                want = correlate2d(img, w[h * d + j], mode="same", boundary="fill", fillvalue=0.0) + b[h * d + j]
                _close(diff[bb, h, P:, j].reshape(gh, gw), want, 1e-12)
    # prefix = 0 is the plain forward; threads agree
    q0, k0, v0, w0, b0 = _problem(1, 2, 3, 3, 4, 3, 132)
    _close(oracle.forward(q0, k0, v0, w0, b0, 3, 3, 3, lib=lib, prefix=0), oracle.forward(q0, k0, v0, w0, b0, 3, 3, 3, lib=lib), 0.0)
    _close(oracle.forward(q, k, v, w, b, gh, gw, ks, lib=lib, prefix=P, threads=3), full, 0.0)


def _worked_inputs():
    q = np.array([[3.0, 4.0], [0.0, 2.0]]).reshape(1, 1, 2, 2)
    k = np.array([[1.0, 0.0], [0.0, -5.0]]).reshape(1, 1, 2, 2)
    v = np.array([[1.0, 2.0], [3.0, 4.0]]).reshape(1, 1, 2, 2)
    w = np.array([[[9, 9, 9], [0.5, 1, 2], [9, 9, 9]], [[7, 7, 7], [-1, 0, 1], [7, 7, 7]]], dtype=np.float64)
    return q, k, v, w, np.array([0.25, -0.5])


def pin_variants_worked_example(lib):
    """The 1 x 2 instance under row normalisation (Eq. 3), the exact kernel (Eq. 5) and the masked softmax
    branch (Eq. 10): tests/golden/worked_example_1x2_variants.txt."""
    q, k, v, w, b = _worked_inputs()
    expect = {}
    for name, t, c, val in _rows("worked_example_1x2_variants.txt"):
        expect.setdefault(name, np.zeros((2, 2)))[int(t), int(c)] = float(val)
    _close(oracle.forward_rownorm(q, k, v, w, b, 1, 2, 3, lib=lib)[0, 0], expect["rownorm"], 1e-14)
    _close(oracle.forward_matrix(q, k, v, w, b, 1, 2, 3, rownorm=True, lib=lib)[0, 0], expect["rownorm"], 1e-14)
    _close(oracle.forward_matrix(q, k, v, w, b, 1, 2, 3, kernel=oracle.KERNEL_EXACT, lib=lib)[0, 0], expect["exact"], 1e-14)
    _close(oracle.forward_matrix(q, k, v, w, b, 1, 2, 3, sparse_eps=0.25, lib=lib)[0, 0], expect["sparse_0.25"], 1e-14)


def pin_rownorm(lib):
    """Eq. 3's denominator on the kept kernel: rows of the explicit weights sum to 1, so a constant V passes
    through the attention term exactly; the linear form equals the explicit one, with and without leading
    tokens; without the denominator the matrix form is the brute-force core."""
    q, k, v, w, b = _problem(2, 3, 5, 4, 6, 3, 201)
    wts = oracle.attention_weights(q[1, 2], k[1, 2], rownorm=True, lib=lib)
    _close(wts.sum(axis=1), np.ones(20), 1e-13)
    raw = oracle.attention_weights(q[1, 2], k[1, 2], lib=lib)
    _close(raw, 0.5 + (_unit(q[1, 2]) @ _unit(k[1, 2]).T) / PI, 1e-13)
    _close(wts, raw / raw.sum(axis=1, keepdims=True), 1e-13)
    _close(oracle.forward_rownorm(q, k, v, w, b, 5, 4, 3, lib=lib), oracle.forward_matrix(q, k, v, w, b, 5, 4, 3, rownorm=True, lib=lib), 1e-12)
    _close(oracle.forward_matrix(q, k, v, w, b, 5, 4, 3, lib=lib), oracle.forward_bruteforce(q, k, v, w, b, 5, 4, 3, lib=lib), 1e-13)
    # constant V: the attention term returns the constant, whatever q and k are
    c = np.array([1.5, -2.0, 0.25, 3.0, -0.5, 7.0])
    vc = np.broadcast_to(c, v.shape).copy()
    w0, b0 = _zero_filter(3, 6, 3)
    _close(oracle.forward_rownorm(q, k, vc, w0, b0, 5, 4, 3, lib=lib), vc, 1e-13)
    # explicit numpy evaluation of the whole variant, conv from the plain core with K = 0 (cosines 0, state 0)
    qh, kh = _unit(q), _unit(k)
    sim = 0.5 + np.einsum("bhtd,bhjd->bhtj", qh, kh) / PI
    att = np.einsum("bhtj,bhjd->bhtd", sim / sim.sum(axis=-1, keepdims=True), v)
    conv = oracle.forward(q, np.zeros_like(k), v, w, b, 5, 4, 3, lib=lib) - 0.5 * v.sum(axis=2, keepdims=True)
    _close(oracle.forward_rownorm(q, k, v, w, b, 5, 4, 3, lib=lib), att + conv, 1e-12)
    # leading tokens: they count in the row sums and the state, and get no convolution
    P = 2
    qp, kp, vp = (np.concatenate([_rand((2, 3, P, 6), 210 + i), t], axis=2) for i, t in enumerate((q, k, v)))
    simp = 0.5 + np.einsum("bhtd,bhjd->bhtj", _unit(qp), _unit(kp)) / PI
    attp = np.einsum("bhtj,bhjd->bhtd", simp / simp.sum(axis=-1, keepdims=True), vp)
    got = oracle.forward_rownorm(qp, kp, vp, w, b, 5, 4, 3, lib=lib, prefix=P)
    _close(got[:, :, :P], attp[:, :, :P], 1e-12)
    _close(got[:, :, P:], attp[:, :, P:] + conv, 1e-12)
    _close(oracle.forward_rownorm(q, k, v, w, b, 5, 4, 3, lib=lib, threads=3), oracle.forward_rownorm(q, k, v, w, b, 5, 4, 3, lib=lib), 0.0)


def pin_exact_kernel_attention(lib):
    """Eq. 4-5 as attention weights: 1 - arccos(cosine)/pi from numpy's arccos; aligned / orthogonal / opposite
    rows give 1, 1/2, 0; the difference to the kept kernel is the odd high-order part of Eq. 8's series."""
    q, k, v, w, b = _problem(1, 2, 4, 4, 5, 3, 221)
    cos = np.clip(_unit(q[0, 1]) @ _unit(k[0, 1]).T, -1.0, 1.0)
    ex = oracle.attention_weights(q[0, 1], k[0, 1], kernel=oracle.KERNEL_EXACT, lib=lib)
    _close(ex, 1.0 - np.arccos(cos) / PI, 1e-13)
    assert ex.min() >= 0.0 and ex.max() <= 1.0
    lin = oracle.attention_weights(q[0, 1], k[0, 1], lib=lib)
    resid = ex - lin
    series = sum(oracle.angular_series_coeff(kk) * cos ** (2 * kk + 1) for kk in range(1, 400)) / PI
    _close(resid, series, 1e-9)
    # special rows
    u = np.array([[2.0, 0.0, 0.0], [0.0, 3.0, 0.0], [-5.0, 0.0, 0.0]])
    sp = oracle.attention_weights(np.repeat(u[:1], 3, axis=0), u, kernel=oracle.KERNEL_EXACT, lib=lib)
    _close(sp[0], [1.0, 0.5, 0.0], 1e-15)
    # whole forward = explicit numpy evaluation + the convolution of the plain core
    full = oracle.forward_matrix(q, k, v, w, b, 4, 4, 3, kernel=oracle.KERNEL_EXACT, lib=lib)
    cosb = np.clip(np.einsum("bhtd,bhjd->bhtj", _unit(q), _unit(k)), -1.0, 1.0)
    conv = oracle.forward(q, np.zeros_like(k), v, w, b, 4, 4, 3, lib=lib) - 0.5 * v.sum(axis=2, keepdims=True)
    _close(full, np.einsum("bhtj,bhjd->bhtd", 1.0 - np.arccos(cosb) / PI, v) + conv, 1e-12)
    # d = 1: cosines are +-1, the weights 1 or 0: every query sums the values of the keys of its own sign
    q1, k1, v1 = _rand((1, 1, 6, 1), 222), _rand((1, 1, 6, 1), 223), _rand((1, 1, 6, 1), 224)
    w1, b1 = _zero_filter(1, 1, 3)
    got = oracle.forward_matrix(q1, k1, v1, w1, b1, 2, 3, 3, kernel=oracle.KERNEL_EXACT, lib=lib)[0, 0, :, 0]
    want = [sum(v1[0, 0, j, 0] for j in range(6) if np.sign(k1[0, 0, j, 0]) == np.sign(q1[0, 0, t, 0])) for t in range(6)]
    _close(got, want, 1e-14)


def pin_sparse_branch(lib):
    """Eq. 10: the masked softmax over the cosines, added to the kept kernel.  A threshold of 1 or more masks
    everything (the inference-time core, bit for bit); a negative threshold keeps everything (plain softmax
    attention on unit rows, rows summing to 1); in between exactly the probabilities above it survive, unscaled."""
    q, k, v, w, b = _problem(2, 2, 4, 5, 6, 3, 231)
    base = oracle.forward_matrix(q, k, v, w, b, 4, 5, 3, lib=lib)
    for thr in (1.0, 2.5):
        assert np.array_equal(oracle.forward_matrix(q, k, v, w, b, 4, 5, 3, sparse_eps=thr, lib=lib), base)
    cos = np.einsum("bhtd,bhjd->bhtj", _unit(q), _unit(k))
    p = np.exp(cos) / np.exp(cos).sum(axis=-1, keepdims=True)
    _close(oracle.softmax_probs(q[1, 0], k[1, 0], lib=lib), p[1, 0], 1e-14)
    _close(oracle.softmax_probs(q[1, 0], k[1, 0], lib=lib).sum(axis=1), np.ones(20), 1e-14)
    _close(oracle.forward_matrix(q, k, v, w, b, 4, 5, 3, sparse_eps=-1.0, lib=lib) - base, np.einsum("bhtj,bhjd->bhtd", p, v), 1e-12)
    thr = 0.05  # p is about 1/20: some entries on either side
    kept = p > thr
    assert 0.1 < kept.mean() < 0.9
    _close(oracle.forward_matrix(q, k, v, w, b, 4, 5, 3, sparse_eps=thr, lib=lib) - base,
           np.einsum("bhtj,bhjd->bhtd", np.where(kept, p, 0.0), v), 1e-12)
    # strictly greater: two identical keys have probability 1/2 each
    qq = np.array([[1.0, 2.0], [3.0, -1.0]]); kk = np.array([[0.5, 0.5], [2.0, 2.0]])
    wts_eq = oracle.attention_weights(qq, kk, sparse_eps=0.5, lib=lib) - oracle.attention_weights(qq, kk, lib=lib)
    _close(wts_eq, np.zeros((2, 2)), 0.0)
    wts_lt = oracle.attention_weights(qq, kk, sparse_eps=0.49, lib=lib) - oracle.attention_weights(qq, kk, lib=lib)
    _close(wts_lt, np.full((2, 2), 0.5), 1e-15)
    # the branch is added after the row normalisation, not inside it
    wn = oracle.attention_weights(q[0, 0], k[0, 0], rownorm=True, sparse_eps=thr, lib=lib)
    _close(wn, oracle.attention_weights(q[0, 0], k[0, 0], rownorm=True, lib=lib) + np.where(p[0, 0] > thr, p[0, 0], 0.0), 1e-13)


PINS = [pin_worked_example, pin_series_coefficients, pin_angular_values, pin_series_properties,
        pin_bruteforce_equals_linear, pin_similarity_matrix, pin_constant_v, pin_equal_keys,
        pin_d_equals_one, pin_zero_rows, pin_conv_known_filters, pin_conv_head_channel_mapping,
        pin_conv_matrix_form, pin_conv_library_routine, pin_scale_invariance,
        pin_linearity_and_symmetry, pin_threads_agree, pin_prefix_tokens, pin_variants_worked_example,
        pin_rownorm, pin_exact_kernel_attention, pin_sparse_branch]


@pytest.mark.parametrize("pin", PINS, ids=lambda f: f.__name__)
def test_pin(pin):
    pin(oracle.load())


# --------------------------------------------------------------------------
# planted mistakes: every one must trip some pin
# --------------------------------------------------------------------------
# (name, text in castling_oracle.c, replacement, how many times the text occurs)
MISTAKES = [
    ("half_term_dropped", "0.5 * vsum[j] + lin / M_PI", "lin / M_PI", 1),
    ("half_term_is_own_token", "0.5 * vsum[j] + lin", "0.5 * vh[(size_t)t * d + j] + lin", 1),
    ("pi_doubled", "lin / M_PI + conv", "lin / (2.0 * M_PI) + conv", 1),
    ("linear_sign", "0.5 * vsum[j] + lin / M_PI", "0.5 * vsum[j] - lin / M_PI", 1),
    ("state_transposed", "lin += xhat[i] * S[i * d + j];", "lin += xhat[i] * S[j * d + i];", 1),
    ("key_not_normalised", "unit_row(kh + (size_t)n * d, d, eps, xhat);",
     "memcpy(xhat, kh + (size_t)n * d, sizeof(double) * d);", 1),
    ("query_not_normalised", "unit_row(qh + (size_t)t * d, d, eps, xhat);",
     "memcpy(xhat, qh + (size_t)t * d, sizeof(double) * d);", 1),
    ("norm_without_sqrt", "return sqrt(ss);", "return ss;", 1),
    ("eps_floor_missing", "if (nrm < eps) nrm = eps;", "", 1),
    ("value_sum_of_keys", "vsum[j] += vh[(size_t)n * d + j];", "vsum[j] += xhat[j];", 1),
    ("state_keeps_last_token", "S[i * d + j] += xhat[i]", "S[i * d + j] = xhat[i]", 1),
    ("conv_flipped", "(dy + r)) * ksize + (dx + r)]", "(r - dy)) * ksize + (r - dx)]", 1),
    ("conv_taps_transposed", "(dy + r)) * ksize + (dx + r)]", "(dx + r)) * ksize + (dy + r)]", 1),
    ("conv_channel_ignores_head", "const int ch = h * d + j;", "const int ch = j;", 1),
    ("conv_bias_dropped", "double acc = bias ? bias[ch] : 0.0;", "double acc = 0.0;", 1),
    ("conv_last_row_lost", "yy >= gridH ||", "yy >= gridH - 1 ||", 1),
    ("conv_wraps_rows", "xx < 0 || xx >= gridW) continue;",
     "xx + yy * gridW < 0 || xx + yy * gridW >= gridH * gridW) continue;", 1),
    ("bruteforce_uses_exact_kernel", "sim[(size_t)t * N + j] = 0.5 + dot / M_PI;",
     "sim[(size_t)t * N + j] = 1.0 - acos(dot > 1 ? 1 : (dot < -1 ? -1 : dot)) / M_PI;", 2),
    ("bruteforce_cosine_transposed", "acc += sim[(size_t)t * N + j] * vh[(size_t)j * d + c];",
     "acc += sim[(size_t)j * N + t] * vh[(size_t)j * d + c];", 1),
    ("series_coefficient", "c *= (2.0 * i - 1.0) / (2.0 * i);", "c *= (2.0 * i - 1.0) / (2.0 * i + 1.0);", 1),
    ("series_constant", "double sum = 0.5 + x / M_PI;", "double sum = 0.5 + x / 3.0;", 1),
    ("exact_kernel_sign", "return 1.0 - acos(x) / M_PI;", "return acos(x) / M_PI;", 1),
    ("prefix_left_out_of_state", "for (int m = 0; m < T; ++m) {                      /* every token, prefix included */",
     "for (int m = prefix; m < T; ++m) {", 1),
    ("prefix_conv_reads_from_token_zero", "dwconv_head(vp + (size_t)prefix * d,", "dwconv_head(vp,", 1),
    ("prefix_rows_get_conv", "(m >= prefix) ? grid_conv[(size_t)(m - prefix) * d + c] : 0.0;",
     "grid_conv[(size_t)(m >= prefix ? m - prefix : m) * d + c];", 1),
    ("prefix_conv_row_offset", "grid_conv[(size_t)(m - prefix) * d + c] : 0.0;", "grid_conv[(size_t)(m - prefix + 1 < G ? m - prefix + 1 : 0) * d + c] : 0.0;", 1),
    ("prefix_half_term", "tok_sum[c] / 2.0 + dot / M_PI + on_grid;", "tok_sum[c] + dot / M_PI + on_grid;", 1),
    ("prefix_state_transposed", "dot += u[a] * state[a * d + c];", "dot += u[a] * state[c * d + a];", 1),
    ("rownorm_counts_grid_only", "double rowsum = 0.5 * T;", "double rowsum = 0.5 * G;", 1),
    ("rownorm_key_sum_not_normalised", "ktot[a] += u[a];", "ktot[a] += kp[(size_t)m * d + a];", 1),
    ("rownorm_pi_missing", "rowsum += u[a] * ktot[a] / M_PI;", "rowsum += u[a] * ktot[a];", 1),
    ("rownorm_divides_conv_too", "op[(size_t)m * d + c] = num / rowsum + on_grid;", "op[(size_t)m * d + c] = (num + on_grid) / rowsum;", 1),
    ("rownorm_half_term", "double num = 0.5 * vtot[c];", "double num = vtot[c];", 1),
    ("rownorm_state_transposed", "num += u[a] * kv[a * d + c] / M_PI;", "num += u[a] * kv[c * d + a] / M_PI;", 1),
    ("matrix_rownorm_by_column", "for (int j = 0; j < T; ++j) row[j] /= total;", "for (int j = 0; j < T; ++j) row[j] /= (total - row[j] + row[t]);", 1),
    ("matrix_exact_kernel_clamped_wrong", "const double xc = x > 1.0 ? 1.0 : (x < -1.0 ? -1.0 : x);", "const double xc = x > 0.5 ? 0.5 : (x < -1.0 ? -1.0 : x);", 1),
    ("sparse_softmax_over_queries", "for (int j = 0; j < T; ++j) z += exp(cosine[j]);", "for (int j = 0; j < T; ++j) z += exp(cosine[t < T ? t : j]);", 1),
    ("sparse_mask_not_strict", "if (p > sparse_eps) row[j] += p;", "if (p >= sparse_eps) row[j] += p;", 1),
    ("sparse_mask_binary", "if (p > sparse_eps) row[j] += p;", "if (p > sparse_eps) row[j] += 1.0;", 1),
    ("sparse_temperature", "const double p = exp(cosine[j]) / z;", "const double p = exp(2.0 * cosine[j]) / z;", 1),
    ("matrix_weights_transposed", "acc += wt[(size_t)t * T + j] * v[base + (size_t)j * d + c];", "acc += wt[(size_t)j * T + t] * v[base + (size_t)j * d + c];", 1),
    ("softmax_probs_unnormalised_keys", "for (int j = 0; j < T; ++j) unit_row(k + (size_t)j * d, d, eps, ku + (size_t)j * d);",
     "memcpy(ku, k, sizeof(double) * (size_t)T * d);", 1),
]


def _failed_pins(lib):
    failed = []
    for pin in PINS:
        try:
            pin(lib)
        except AssertionError:
            failed.append(pin.__name__)
    return failed


@pytest.mark.parametrize("mistake", MISTAKES, ids=lambda m: m[0])
def test_pins_catch_planted_mistakes(mistake, tmp_path):
    name, old, new, count = mistake
    src = open(os.path.join(os.path.dirname(oracle.__file__), "castling_oracle.c")).read()
    assert src.count(old) == count, f"mistake '{name}' no longer matches the oracle source"
    bad_c = tmp_path / f"oracle_{name}.c"
    bad_so = tmp_path / f"liboracle_{name}.so"
    bad_c.write_text(src.replace(old, new))
    subprocess.run(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-o", str(bad_so), str(bad_c), "-lm"], check=True)
    failed = _failed_pins(oracle.load(str(bad_so)))
    assert failed, f"no pin notices the planted mistake '{name}'"
