"""Sequence-sharded forward on one GPU: the bands of rows that different ranks would hold are processed one after
another on the same device, and the all-reduce of their states is a sum on that device (the exchange itself is
covered on CPU ranks in test_sharded_host_logic.py).  The result must be the unsharded forward of the oracle."""
from __future__ import annotations

import numpy as np
import pytest
import torch

import oracle
import workloads
from paper_2211_10526_b200 import sharded

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "bf16": 2e-2}

# B, H, gridH, gridW, d, ksize, dtype, world
CASES = [(2, 3, 12, 10, 32, 3, "f32", 2), (1, 2, 17, 9, 64, 5, "f32", 3), (2, 4, 64, 64, 32, 5, "bf16", 4),
         (2, 2, 33, 20, 64, 3, "bf16", 5), (1, 2, 8, 8, 48, 7, "f32", 2), (2, 8, 128, 128, 64, 3, "bf16", 8),
         (1, 3, 6, 5, 16, 1, "f32", 3), (2, 3, 50, 44, 64, 5, "bf16", 3), (1, 4, 96, 64, 64, 3, "bf16", 2)]


@pytest.mark.parametrize("case", CASES, ids=lambda c: "x".join(map(str, c)))
def test_bands_of_rows_reproduce_the_whole_forward(case):
    from paper_2211_10526_b200 import CastlingAttn
    B, H, gh, gw, d, ks, dtype, world = case
    c = workloads.custom_call(B, H, gh, gw, d, ks, dtype, seed=9000 + gh + world)
    dev = torch.device("cuda:0")
    q, k, v, w, b = (t.to(dev) for t in (c.q, c.k, c.v, c.dw_weight, c.dw_bias))
    r = (ks - 1) // 2
    with CastlingAttn(ksize=ks) as attn:
        bands = [sharded.band_rows(gh, world, rank) for rank in range(world)]
        rows = lambda t, y0, y1: t[:, :, y0 * gw:y1 * gw].contiguous()
        states = [attn.shard_state(rows(k, y0, y1), rows(v, y0, y1)) for y0, y1 in bands]
        total = torch.stack(states).sum(dim=0)            # what the all-reduce leaves on every rank
        outs = []
        for y0, y1 in bands:
            top, bottom = sharded.halo_rows(gh, y0, y1, ks)
            assert (top, bottom) == (min(r, y0), min(r, gh - y1)) or (y1 - y0) < r
            out = attn.shard_apply(rows(q, y0, y1), rows(v, y0 - top, y1 + bottom), w, b, total, y1 - y0, gw, top, bottom)
            outs.append(out)
        torch.cuda.synchronize()
        assert attn.device_status() == (0, 0)
        # bf16 bands of width-64 heads with at least 48 tokens run on the tensor-core kernels, the rest on CUDA cores
        want = 2 if (dtype == "bf16" and d == 64 and min(y1 - y0 for y0, y1 in bands) * gw >= 48) else 1
        assert attn.last_path()[0] == want
        got = torch.cat(outs, dim=2).double().cpu().numpy()
        # the states of the bands add up to the state of the whole sequence
        whole = attn.shard_state(k, v)
        torch.cuda.synchronize()
        assert float((whole - total).abs().max()) <= 1e-4 * float(whole.abs().max())
    ref = oracle.forward(c.q, c.k, c.v, c.dw_weight, c.dw_bias, gh, gw, ks, threads=8)
    err = float(np.max(np.abs(got - ref)) / np.max(np.abs(ref)))
    assert err <= TOL[dtype], f"{case}: max-rel error {err:.3e}"


def test_convolution_across_band_edges_alone():
    """K = 0, antisymmetric V: the output is the convolution alone, so a wrong or missing halo row is the whole
    error at the rows next to a band edge."""
    from paper_2211_10526_b200 import CastlingAttn
    gh, gw, ks, world = 20, 12, 5, 4
    c = workloads.custom_call(1, 2, gh, gw, 32, ks, "f32", seed=9100)
    c.k.zero_()
    n = gh * gw // 2
    c.v[:, :, n:] = -c.v[:, :, :n]
    c.dw_weight *= 20
    dev = torch.device("cuda:0")
    q, k, v, w, b = (t.to(dev) for t in (c.q, c.k, c.v, c.dw_weight, c.dw_bias))
    with CastlingAttn(ksize=ks) as attn:
        bands = [sharded.band_rows(gh, world, rank) for rank in range(world)]
        rows = lambda t, y0, y1: t[:, :, y0 * gw:y1 * gw].contiguous()
        total = torch.stack([attn.shard_state(rows(k, *bd), rows(v, *bd)) for bd in bands]).sum(dim=0)
        outs = []
        for y0, y1 in bands:
            top, bottom = sharded.halo_rows(gh, y0, y1, ks)
            outs.append(attn.shard_apply(rows(q, y0, y1), rows(v, y0 - top, y1 + bottom), w, b, total, y1 - y0, gw, top, bottom))
        torch.cuda.synchronize()
    got = torch.cat(outs, dim=2).double().cpu().numpy()
    ref = oracle.forward(c.q, c.k, c.v, c.dw_weight, c.dw_bias, gh, gw, ks)
    assert float(np.max(np.abs(got - ref)) / np.max(np.abs(ref))) <= 1e-5


def test_convolution_across_band_edges_alone_on_the_tensor_core_kernels():
    """The same isolation for bf16 bands of width-64 heads, which run on the tensor-core kernels: the neighbours' rows
    come through the taller V tensor, the zero padding only at the edge of the whole grid."""
    from paper_2211_10526_b200 import CastlingAttn
    for gh, gw, ks, world in ((40, 24, 5, 4), (36, 40, 3, 3)):
        c = workloads.custom_call(2, 2, gh, gw, 64, ks, "bf16", seed=9200 + gh)
        c.k.zero_()
        n = gh * gw // 2
        c.v[:, :, n:] = -c.v[:, :, :n]
        c.dw_weight = (c.dw_weight.float() * 20).to(c.dw_weight.dtype)
        dev = torch.device("cuda:0")
        q, k, v, w, b = (t.to(dev) for t in (c.q, c.k, c.v, c.dw_weight, c.dw_bias))
        with CastlingAttn(ksize=ks) as attn:
            bands = [sharded.band_rows(gh, world, rank) for rank in range(world)]
            rows = lambda t, y0, y1: t[:, :, y0 * gw:y1 * gw].contiguous()
            total = torch.stack([attn.shard_state(rows(k, *bd), rows(v, *bd)) for bd in bands]).sum(dim=0)
            outs = []
            for y0, y1 in bands:
                top, bottom = sharded.halo_rows(gh, y0, y1, ks)
                outs.append(attn.shard_apply(rows(q, y0, y1), rows(v, y0 - top, y1 + bottom), w, b, total, y1 - y0, gw, top, bottom))
                assert attn.last_path()[0] == 2
            torch.cuda.synchronize()
            assert attn.device_status() == (0, 0)
        got = torch.cat(outs, dim=2).double().cpu().numpy()
        ref = oracle.forward(c.q, c.k, c.v, c.dw_weight, c.dw_bias, gh, gw, ks)
        assert float(np.max(np.abs(got - ref)) / np.max(np.abs(ref))) <= 2e-2


def test_shard_entry_points_reject_what_they_do_not_take():
    from paper_2211_10526_b200 import CastlingAttn, binding as b
    dev = torch.device("cuda:0")
    t = torch.zeros(1, 1, 16, 32, device=dev)
    w, bias = torch.zeros(32, 3, 3, device=dev), torch.zeros(32, device=dev)
    with CastlingAttn(ksize=3, normalize_rows=True) as attn:
        with pytest.raises(b.CastlingError):
            attn.shard_state(t, t)
    with CastlingAttn(ksize=3) as attn:
        st = attn.shard_state(t, t)
        with pytest.raises(b.CastlingError):     # halo taller than the filter radius
            attn.shard_apply(t, torch.zeros(1, 1, 16 + 2 * 4, 32, device=dev), w, bias, st, 4, 4, 2, 0)
