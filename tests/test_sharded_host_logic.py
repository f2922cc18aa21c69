"""Host side of the sequence-sharded forward on CPU ranks (gloo, world size 2 and 3): band and halo arithmetic,
the exchange of neighbour rows, and the sum of the per-band states by all-reduce.  The per-band sums stand in
numpy here (unit key rows times values); the kernels themselves are covered on the GPU."""
from __future__ import annotations

import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2211_10526_b200 import sharded


def test_bands_cover_the_grid_once():
    for gh in (5, 8, 17, 64):
        for world in (1, 2, 3, 5):
            if gh < world:
                continue
            bands = [sharded.band_rows(gh, world, r) for r in range(world)]
            assert bands[0][0] == 0 and bands[-1][1] == gh
            assert all(a[1] == b[0] for a, b in zip(bands, bands[1:]))
            assert max(y1 - y0 for y0, y1 in bands) - min(y1 - y0 for y0, y1 in bands) <= 1
    assert sharded.halo_rows(10, 0, 5, 5) == (0, 2) and sharded.halo_rows(10, 5, 10, 5) == (2, 0)
    assert sharded.halo_rows(10, 3, 6, 3) == (1, 1) and sharded.halo_rows(10, 0, 10, 7) == (0, 0)
    with pytest.raises(ValueError):
        sharded.band_rows(3, 4, 0)


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, gh: int, gw: int, ks: int):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        g = torch.Generator().manual_seed(77)
        B, H, d = 2, 3, 8
        v = torch.randn(B, H, gh * gw, d, generator=g)
        k = torch.randn(B, H, gh * gw, d, generator=g)
        y0, y1 = sharded.band_rows(gh, world, rank)
        v_loc = v[:, :, y0 * gw:y1 * gw].contiguous()
        v_halo, top, bottom = sharded.exchange_halo(v_loc, gw, ks, rank, world)
        want_top, want_bottom = sharded.halo_rows(gh, y0, y1, ks)
        assert (top, bottom) == (want_top, want_bottom)
        assert torch.equal(v_halo, v[:, :, (y0 - top) * gw:(y1 + bottom) * gw])
        # the state of the whole sequence is the sum of the bands' states
        def state(kk, vv):
            ku = kk / kk.norm(dim=-1, keepdim=True)
            return torch.cat([torch.einsum("bhni,bhnj->bhij", ku, vv).flatten(2), vv.sum(dim=2)], dim=2)
        st = state(k[:, :, y0 * gw:y1 * gw].double(), v_loc.double())
        dist.all_reduce(st, op=dist.ReduceOp.SUM)
        assert torch.allclose(st, state(k.double(), v.double()), rtol=1e-12, atol=1e-12)
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,gh,ks", [(2, 7, 3), (3, 9, 5), (2, 4, 1)])
def test_halo_exchange_and_state_sum_on_cpu_ranks(world, gh, ks):
    mp.spawn(_rank_main, args=(world, _free_port(), gh, 5, ks), nprocs=world, join=True)
