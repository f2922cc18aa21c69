"""GPU tests of the C-ABI boundary: error codes, ownership, memory safety, determinism."""
from __future__ import annotations

import numpy as np
import pytest
import torch

import oracle
import workloads

pytestmark = pytest.mark.gpu


def _b():
    from paper_2211_10526_b200 import binding
    return binding


def _dev(call):
    dev = torch.device("cuda:0")
    return [t.to(dev) for t in (call.q, call.k, call.v, call.dw_weight, call.dw_bias)]


def _raw_forward(b, h, q, k, v, w, bias, out, s, dtype_code=None, stream=0):
    code = (b.CASTLING_F32 if q.dtype == torch.float32 else b.CASTLING_BF16) if dtype_code is None else dtype_code
    return b.castling_attn_forward(h, q.data_ptr(), k.data_ptr(), v.data_ptr(), w.data_ptr(),
                                   None if bias is None else bias.data_ptr(), out.data_ptr(),
                                   s.B, s.H, s.gridH, s.gridW, s.d, code, stream)


def test_error_codes():
    b = _b()
    c = workloads.custom_call(1, 2, 4, 4, 32, 3, "f32", seed=400)
    q, k, v, w, bias = _dev(c)
    out = torch.empty_like(q)
    s = c.shape
    h = b.castling_attn_create(3)
    try:
        assert _raw_forward(b, h, q, k, v, w, bias, out, s) == b.OK
        # NULL tensor
        assert b.castling_attn_forward(h, None, k.data_ptr(), v.data_ptr(), w.data_ptr(), None, out.data_ptr(),
                                       1, 2, 4, 4, 32, 0) == b.ERR_INVALID_ARG
        # non-positive dims
        for dims in ((0, 2, 4, 4, 32), (1, 0, 4, 4, 32), (1, 2, -4, 4, 32), (1, 2, 4, 0, 32), (1, 2, 4, 4, 0)):
            assert b.castling_attn_forward(h, q.data_ptr(), k.data_ptr(), v.data_ptr(), w.data_ptr(), None,
                                           out.data_ptr(), *dims, 0) == b.ERR_INVALID_ARG
        # unsupported head width / dtype
        for d in (8, 33, 144):
            assert b.castling_attn_forward(h, q.data_ptr(), k.data_ptr(), v.data_ptr(), w.data_ptr(), None,
                                           out.data_ptr(), 1, 2, 4, 4, d, 0) == b.ERR_UNSUPPORTED
        assert _raw_forward(b, h, q, k, v, w, bias, out, s, dtype_code=5) == b.ERR_UNSUPPORTED
        # misaligned tensor pointer (4 bytes off a 16-byte boundary)
        flat = torch.empty(q.numel() + 8, dtype=q.dtype, device=q.device)
        mis = flat[1:1 + q.numel()].view_as(q)
        assert mis.data_ptr() % 16 != 0
        assert _raw_forward(b, h, mis, k, v, w, bias, out, s) == b.ERR_ALIGNMENT
        assert _raw_forward(b, h, q, k, v, w, bias, mis, s) == b.ERR_ALIGNMENT
        # output overlapping an input
        assert _raw_forward(b, h, q, k, v, w, bias, v, s) == b.ERR_INVALID_ARG
        both = torch.empty(2 * q.numel() - 64, dtype=q.dtype, device=q.device)
        a_in = both[:q.numel()].view_as(q)
        a_out = both[q.numel() - 64:].view_as(q)
        assert _raw_forward(b, h, a_in, k, v, w, bias, a_out, s) == b.ERR_INVALID_ARG
        # workspace cap
        h2 = b.castling_attn_create(3, max_workspace=128)
        assert _raw_forward(b, h2, q, k, v, w, bias, out, s) == b.ERR_OOM
        b.castling_attn_destroy(h2)
        # the handle still works after every rejected call
        assert _raw_forward(b, h, q, k, v, w, bias, out, s) == b.OK
        torch.cuda.synchronize()
        path, launches = b.castling_attn_last_path(h)
        assert path in (b.PATH_SIMT, b.PATH_TENSOR) and launches >= 1
        assert b.castling_attn_device_status(h) == (b.OK, 0)
    finally:
        b.castling_attn_destroy(h)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", [(2, 3, 9, 7, 32, 3), (1, 2, 70, 75, 64, 5), (4, 12, 14, 14, 64, 3)],
                         ids=["small", "split", "deit"])
def test_guard_bands_and_inputs_untouched(shape, dtype):
    """Bytes before and after `out` keep their pattern; inputs are bit-identical afterwards."""
    b = _b()
    c = workloads.custom_call(*shape, dtype, seed=410)
    q, k, v, w, bias = _dev(c)
    s = c.shape
    n = q.numel()
    guard = 4096
    buf = torch.full((n + 2 * guard,), float("nan"), dtype=q.dtype, device=q.device)
    out = buf[guard:guard + n].view_as(q)
    assert out.data_ptr() % 16 == 0
    before = [t.clone() for t in (q, k, v, w, bias)]
    h = b.castling_attn_create(s.ksize)
    try:
        assert _raw_forward(b, h, q, k, v, w, bias, out, s) == b.OK
        torch.cuda.synchronize()
    finally:
        b.castling_attn_destroy(h)
    assert torch.isnan(buf[:guard]).all() and torch.isnan(buf[guard + n:]).all()
    assert torch.isfinite(out.float()).all(), "an output element was never written"
    for t, t0 in zip((q, k, v, w, bias), before):
        assert torch.equal(t.view(torch.uint8), t0.view(torch.uint8))


@pytest.mark.parametrize("name,idx", [("c1_fp32_tiny", 0), ("c4_detection_bf16", 0), ("c5_sweep_bf16", 1)])
def test_bitwise_reproducible(name, idx):
    """Reductions run in a fixed order: two runs give identical bits, also from a second handle."""
    b = _b()
    (c,) = list(workloads.iter_workload(name, only=[idx]))
    q, k, v, w, bias = _dev(c)
    s = c.shape
    outs = []
    for _ in range(2):
        h = b.castling_attn_create(s.ksize)
        for _ in range(2):
            out = torch.empty_like(q)
            assert _raw_forward(b, h, q, k, v, w, bias, out, s) == b.OK
            torch.cuda.synchronize()
            outs.append(out)
        b.castling_attn_destroy(h)
    for o in outs[1:]:
        assert torch.equal(o.view(torch.uint8), outs[0].view(torch.uint8))


@pytest.mark.parametrize("shape", [(2, 8, 64, 64, 64, 3), (2, 4, 96, 128, 64, 3), (4, 8, 64, 64, 32, 5)],
                         ids=lambda t: "x".join(map(str, t)))
def test_forwards_queued_back_to_back_do_not_disturb_each_other(shape):
    """On the tensor-core path the state kernel of a forward starts while the apply kernel of the previous one is
    still draining (programmatic dependent launch).  Forwards on alternating, different inputs are queued without
    any synchronisation, each into its own output; every output has to equal, bit for bit, the output of the same
    inputs run alone (the path is bitwise reproducible), so a state written too early, or read too late, shows."""
    b = _b()
    sets = []
    for seed in (431, 432, 433):
        c = workloads.custom_call(*shape, "bf16", seed=seed)
        sets.append((c, _dev(c)))
    s = sets[0][0].shape
    h = b.castling_attn_create(s.ksize)
    alone = []
    for c, (q, k, v, w, bias) in sets:
        out = torch.empty_like(q)
        assert _raw_forward(b, h, q, k, v, w, bias, out, s) == b.OK
        torch.cuda.synchronize()
        alone.append(out)
    assert not torch.equal(alone[0], alone[1])
    rounds = 12
    outs = [[torch.full_like(alone[0], float("nan")) for _ in sets] for _ in range(rounds)]
    for r in range(rounds):
        for i, (c, (q, k, v, w, bias)) in enumerate(sets):
            assert _raw_forward(b, h, q, k, v, w, bias, outs[r][i], s) == b.OK
    torch.cuda.synchronize()
    assert b.castling_attn_device_status(h)[0] == b.OK
    b.castling_attn_destroy(h)
    for r in range(rounds):
        for i in range(len(sets)):
            assert torch.equal(outs[r][i].view(torch.uint8), alone[i].view(torch.uint8)), (r, i)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_host_entry_point_matches_device_entry_point(dtype):
    from paper_2211_10526_b200 import CastlingAttn
    c = workloads.custom_call(2, 4, 14, 14, 32, 3, dtype, seed=420)
    s = c.shape
    with CastlingAttn(ksize=3) as attn:
        pinned = [t.pin_memory() for t in (c.q, c.k, c.v, c.dw_weight, c.dw_bias)]
        out_h = torch.empty_like(c.q).pin_memory()
        attn.forward_host(*pinned, s.gridH, s.gridW, out=out_h)
        out_d = attn.forward(*_dev(c), s.gridH, s.gridW)
        torch.cuda.synchronize()
        assert torch.equal(out_d.cpu().view(torch.uint8), out_h.view(torch.uint8))
        # pageable memory and no bias also work
        out_p = attn.forward_host(c.q, c.k, c.v, c.dw_weight, None, s.gridH, s.gridW)
    ref = oracle.forward(c.q, c.k, c.v, c.dw_weight, None, s.gridH, s.gridW, 3)
    err = np.max(np.abs(out_p.double().numpy() - ref)) / np.max(np.abs(ref))
    assert err <= (1e-5 if dtype == "f32" else 2e-2)


def test_two_handles_two_streams_and_shape_changes():
    """Distinct handles are independent; one handle may serve shapes of growing and shrinking size."""
    from paper_2211_10526_b200 import CastlingAttn
    calls = [workloads.custom_call(1, 2, 6, 6, 32, 3, "bf16", seed=430),
             workloads.custom_call(2, 4, 40, 40, 64, 3, "bf16", seed=431),
             workloads.custom_call(1, 1, 3, 5, 64, 3, "bf16", seed=432)]
    refs = [oracle.forward(c.q, c.k, c.v, c.dw_weight, c.dw_bias, c.shape.gridH, c.shape.gridW, 3, threads=8)
            for c in calls]
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    a1, a2 = CastlingAttn(3), CastlingAttn(3)
    outs = []
    dev_calls = [_dev(c) for c in calls]
    torch.cuda.synchronize()
    for i, (c, d) in enumerate(zip(calls, dev_calls)):
        with torch.cuda.stream(s1 if i % 2 == 0 else s2):
            attn = a1 if i % 2 == 0 else a2
            outs.append(attn.forward(*d, c.shape.gridH, c.shape.gridW))
    # and the same handle across all shapes on one stream
    with torch.cuda.stream(s1):
        outs2 = [a1.forward(*d, c.shape.gridH, c.shape.gridW) for c, d in zip(calls, dev_calls)]
    torch.cuda.synchronize()
    for o, o2, ref in zip(outs, outs2, refs):
        for t in (o, o2):
            err = np.max(np.abs(t.double().cpu().numpy() - ref)) / np.max(np.abs(ref))
            assert err <= 2e-2
    a1.close(); a2.close()


def test_create_destroy_cycles():
    b = _b()
    for _ in range(50):
        h = b.castling_attn_create(5)
        assert b.castling_attn_destroy(h) == b.OK


def test_host_entry_point_pipelines_batch_chunks():
    """Large host-side problems are uploaded, computed and downloaded in overlapping batch chunks."""
    from paper_2211_10526_b200 import CastlingAttn
    c = workloads.custom_call(4, 8, 128, 64, 64, 3, "bf16", seed=440)   # 33.5 MB per tensor -> four chunks
    s = c.shape
    pinned = [t.pin_memory() for t in (c.q, c.k, c.v, c.dw_weight, c.dw_bias)]
    out_h = torch.full_like(c.q, float("nan")).pin_memory()
    with CastlingAttn(ksize=3) as attn:
        for _ in range(2):
            attn.forward_host(*pinned, s.gridH, s.gridW, out=out_h)
        out_d = attn.forward(*_dev(c), s.gridH, s.gridW)
        torch.cuda.synchronize()
        assert attn.device_status() == (0, 0)
    assert torch.isfinite(out_h.float()).all()
    ref = oracle.forward(c.q, c.k, c.v, c.dw_weight, c.dw_bias, s.gridH, s.gridW, 3, threads=8)
    for got in (out_h, out_d.cpu()):
        err = np.max(np.abs(got.double().numpy() - ref)) / np.max(np.abs(ref))
        assert err <= 2e-2


# Pipelined chunks whose plane count differs from the head count: more planes than heads (a chunk spans
# several batches), fewer planes than heads (a chunk starts and ends inside one batch), and a head count
# that does not divide the chunk.  B, H, gridH, gridW, d, ksize, chunks expected, kernel family expected
CHUNK_CASES = [(16, 3, 54, 54, 64, 3, 2, 2), (2, 8, 128, 128, 64, 3, 4, 2), (5, 7, 96, 64, 64, 5, 3, 2),
               (7, 6, 96, 96, 32, 3, 2, 2)]


@pytest.mark.parametrize("case", CHUNK_CASES, ids=lambda c: "x".join(map(str, c[:6])))
def test_host_entry_point_chunks_that_do_not_align_with_heads(case):
    from paper_2211_10526_b200 import CastlingAttn, binding
    B, H, gh, gw, d, ks, chunks, family = case
    c = workloads.custom_call(B, H, gh, gw, d, ks, "bf16", seed=445 + sum(case[:6]))
    per_tensor = c.q.numel() * 2
    assert min(8, B * H, per_tensor // (8 << 20)) == chunks, "the case no longer makes the intended chunk count"
    pinned = [t.pin_memory() for t in (c.q, c.k, c.v, c.dw_weight, c.dw_bias)]
    out_h = torch.full_like(c.q, float("nan")).pin_memory()
    with CastlingAttn(ksize=ks) as attn:
        attn.forward_host(*pinned, gh, gw, out=out_h)
        assert attn.device_status() == (0, 0)
        assert attn.last_path()[0] == family, "a chunk fell back to the other kernel family"
    g = out_h.double().numpy()
    assert np.all(np.isfinite(g)), "part of the output was never written"
    ref = oracle.forward(c.q, c.k, c.v, c.dw_weight, c.dw_bias, gh, gw, ks, threads=16)
    err = np.max(np.abs(g - ref)) / np.max(np.abs(ref))
    assert err <= 2e-2
    # per plane as well: a plane computed from another plane's data would still be of the right size
    per_plane = np.max(np.abs(g - ref), axis=(2, 3)) / np.max(np.abs(ref), axis=(2, 3))
    assert per_plane.max() <= 2e-2, f"worst plane {np.unravel_index(per_plane.argmax(), per_plane.shape)}"


@pytest.mark.parametrize("shape", [(2, 4, 1, 14, 14, 32, 3, "f32"), (4, 8, 2, 128, 64, 64, 3, "bf16"), (3, 5, 1, 14, 14, 64, 3, "bf16")],
                         ids=lambda s: "x".join(map(str, s)))
def test_host_entry_point_with_leading_tokens(shape):
    """Host-buffer entry point (one piece and pipelined chunks) for sequences that start with off-grid tokens."""
    from paper_2211_10526_b200 import CastlingAttn
    B, H, P, gh, gw, d, ks, dtype = shape
    c = workloads.custom_call(B, H, 1, P + gh * gw, d, ks, dtype, seed=450 + sum(shape[:7]))
    pinned = [t.pin_memory() for t in (c.q, c.k, c.v, c.dw_weight, c.dw_bias)]
    out_h = torch.full_like(c.q, float("nan")).pin_memory()
    with CastlingAttn(ksize=ks, prefix_tokens=P) as attn:
        attn.forward_host(*pinned, gh, gw, out=out_h)
        assert attn.device_status() == (0, 0)
    ref = oracle.forward(c.q, c.k, c.v, c.dw_weight, c.dw_bias, gh, gw, ks, threads=8, prefix=P)
    g = out_h.double().numpy()
    assert np.all(np.isfinite(g))
    err = np.max(np.abs(g - ref)) / np.max(np.abs(ref))
    assert err <= (1e-5 if dtype == "f32" else 2e-2)


GRAPH_SHAPES = [  # B, H, prefix, gridH, gridW, d, ksize, dtype: one per kernel family
    (2, 4, 0, 14, 14, 32, 3, "f32"),     # CUDA-core state + apply
    (1, 2, 0, 48, 50, 32, 3, "f32"),     # CUDA-core with the token range split (reduce kernel)
    (64, 8, 0, 7, 7, 32, 3, "bf16"),     # CUDA-core single-launch kernel
    (4, 12, 1, 14, 14, 64, 3, "bf16"),   # single tensor-core kernel, one leading token
    (2, 8, 0, 64, 64, 64, 3, "bf16"),    # tensor-core state + apply (programmatic dependent launch), split state
    (8, 8, 0, 64, 64, 32, 5, "bf16"),    # width-32 token pairs, 5 x 5
    (2, 2, 2, 24, 20, 64, 3, "bf16"),    # tensor-core path + leading-rows kernel
]


@pytest.mark.parametrize("shape", GRAPH_SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_forward_inside_a_cuda_graph(shape):
    """A forward only enqueues kernels on the caller's stream once its workspace exists, so it can be
    captured into a CUDA graph and replayed on new data in the same buffers."""
    from paper_2211_10526_b200 import CastlingAttn
    B, H, P, gh, gw, d, ks, dtype = shape
    c1 = workloads.custom_call(B, H, 1, P + gh * gw, d, ks, dtype, seed=470 + sum(shape[:7]))
    c2 = workloads.custom_call(B, H, 1, P + gh * gw, d, ks, dtype, seed=471 + sum(shape[:7]))
    dev = torch.device("cuda:0")
    q, k, v, w, b = (t.to(dev) for t in (c1.q, c1.k, c1.v, c1.dw_weight, c1.dw_bias))
    out = torch.empty_like(q)
    side = torch.cuda.Stream()
    with CastlingAttn(ksize=ks, prefix_tokens=P) as attn:
        with torch.cuda.stream(side):
            attn.forward(q, k, v, w, b, gh, gw, out=out)   # first call: allocates the workspace (not capturable)
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            attn.forward(q, k, v, w, b, gh, gw, out=out)
        for t, src in ((q, c2.q), (k, c2.k), (v, c2.v), (w, c2.dw_weight), (b, c2.dw_bias)):
            t.copy_(src)
        out.fill_(float("nan"))
        graph.replay()
        graph.replay()
        torch.cuda.synchronize()
        assert attn.device_status() == (0, 0)
    ref = oracle.forward(c2.q, c2.k, c2.v, c2.dw_weight, c2.dw_bias, gh, gw, ks, threads=8, prefix=P)
    g = out.double().cpu().numpy()
    assert np.all(np.isfinite(g))
    err = float(np.max(np.abs(g - ref)) / np.max(np.abs(ref)))
    assert err <= (1e-5 if dtype == "f32" else 2e-2), err


def test_bounded_wait_gives_up_and_the_handle_stays_usable():
    """A wait that can never be satisfied (a barrier nothing completes) runs into its limit, the kernel returns,
    the status word reports it once as CASTLING_ERR_DEVICE, and a forward on the same handle is correct after."""
    import time
    import workloads
    from paper_2211_10526_b200 import CastlingAttn, binding as b
    dev = torch.device("cuda:0")
    c = workloads.custom_call(2, 2, 24, 20, 64, 3, "bf16", seed=910)
    s = c.shape
    ref = oracle.forward(c.q, c.k, c.v, c.dw_weight, c.dw_bias, s.gridH, s.gridW, s.ksize)
    args = tuple(t.to(dev) for t in (c.q, c.k, c.v, c.dw_weight, c.dw_bias))
    with CastlingAttn(ksize=3) as attn:
        out = attn.forward(*args, s.gridH, s.gridW)
        torch.cuda.synchronize()
        assert attn.device_status() == (0, 0)
        t0 = time.perf_counter()
        assert b.castling_attn_selftest_wait(attn.handle, 3000) == b.OK     # 3 ms limit
        waited = time.perf_counter() - t0
        assert 0.002 <= waited < 1.0, waited                                 # it did wait, and it did stop
        rc, raw = attn.device_status()
        assert rc == b.ERR_DEVICE and raw == 16
        assert attn.device_status() == (0, 0)                                # reported once, then cleared
        assert b.castling_attn_selftest_wait(attn.handle, 0) == b.ERR_INVALID_ARG
        out = attn.forward(*args, s.gridH, s.gridW)
        torch.cuda.synchronize()
        assert attn.device_status() == (0, 0)
    err = float(np.max(np.abs(out.double().cpu().numpy() - ref)) / np.max(np.abs(ref)))
    assert err <= 2e-2
