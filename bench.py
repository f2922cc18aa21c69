#!/usr/bin/env python
"""Benchmark of the linear-angular attention core.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME[:IDX]] [--impl ours|reference]

A step is one forward pass of the whole attention core (state build, reduction, apply +
depthwise convolution) over one synthetic batch.  The default workload is the largest
long-sequence sweep point (B=2, H=8, 256x256 tokens, d=64, bf16): its four tensors
(537 MB) exceed the 126 MB L2, so every step streams from HBM and no L2 flush is needed.
Smaller workloads (``--workload``) cycle through a ring of copies of their tensors three times
the size of L2 ("cold"); the time on one L2-resident set is reported beside it ("hot").
With N > 1 (under torchrun) every rank runs an independent replica of the workload on its
own GPU -- the (b,h) problems are independent, there is no collective on the data path --
and the reported value is the tokens all ranks processed divided by the slowest rank's time.

One JSON line is printed by rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch

import workloads

METRIC = "tokens/sec and achieved HBM GB/s (% of B200 peak) for linear-angular attn fwd"
UNIT = "tokens/s"
DEFAULT_WORKLOAD = "c5_sweep_bf16:3"
L2_BYTES = 126 * 1000 * 1000  # a workload under twice this is timed over a ring of buffer sets
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the dominant kernel from one ncu
# capture, with the summary file and the last commit that touched that kernel's source when it was taken.
# bench.py reports the figure only while `git log` still names that commit as the kernel's latest: after
# any later change to the kernel the counters are stale and `traffic` is null.
NCU_TRAFFIC = {
    ("c5_sweep_bf16:3", "tc_apply"): {"bytes": 281.8e6 + 122.1e6, "profile": "profiles/tc_kernels_c5_sweep.md",
                                      "source": "paper_2211_10526_b200/csrc/tc_apply.cu", "commit": "0c32e4c"},
    ("c3_deit_base_bf16", "tc_fused"): {"bytes": 57.9e6 + 2.0e6, "profile": "profiles/tc_fused_c3_deit_base.md",
                                        "source": "paper_2211_10526_b200/csrc/tc_fused.cu", "commit": "d209734"},
}
REPEATS = 5          # timed repeats; the median is reported
MIN_FORWARDS = 100   # forwards per repeat, at least


def ncu_traffic(workload: str, kernel: str):
    """(bytes per launch or None, where the figure comes from)."""
    ent = NCU_TRAFFIC.get((workload, kernel))
    if ent is None:
        return None, "no capture of this kernel on this workload"
    try:
        head = subprocess.run(["git", "-C", ROOT, "log", "-1", "--format=%h", "--", ent["source"]],
                              capture_output=True, text=True, timeout=10).stdout.strip()
    except Exception:
        head = ""
    if head and head[:7] != ent["commit"][:7]:
        return None, f"{ent['profile']} was captured at {ent['commit']}; {ent['source']} last changed at {head}"
    return ent["bytes"], f"{ent['profile']} (captured at {ent['commit']})"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, help="workload name[:call index]")
    ap.add_argument("--force-path", type=int, default=0, help="0 auto, 1 CUDA-core kernels, 2 tensor-core kernels")
    ap.add_argument("--layout", default="head_major", choices=["head_major", "token_major"],
                    help="memory layout of q, k, v, out: [B,H,N,d] contiguous, or [B,N,H,d] passed as strided views")
    ap.add_argument("--repeats", type=int, default=REPEATS, help="timed repeats (the median is reported)")
    ap.add_argument("--min-forwards", type=int, default=MIN_FORWARDS,
                    help="forwards per repeat, at least; a profiler run passes 1 here and to --repeats")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    return ap.parse_args()


def pick_call(spec: str, seed_offset: int = 0) -> workloads.CallInputs:
    name, _, idx = spec.partition(":")
    idx = int(idx) if idx else 0
    (call,) = list(workloads.iter_workload(name, only=[idx], seed_offset=seed_offset))
    return call


def measured_peak_hbm():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU with nvidia-smi while a region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for ln in self.proc.stdout:
            self.lines.append(ln.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def dist_setup(n_gpus: int):
    """(rank, world, local_rank); initialises torch.distributed when launched under torchrun."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        backend = "nccl" if torch.cuda.is_available() else "gloo"
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world, local


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(x: float, world: int, device) -> float:
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def cpu_oracle_rate(call: workloads.CallInputs, target_heads=None):
    """Time the oracle, as it stands, on a bounded sample of the workload: the first S (b,h)
    slices, one host thread each.  Returns (image tokens/s, threads used, sample text, seconds)."""
    import oracle
    s = call.shape
    cores = os.cpu_count() or 1
    BH = s.B * s.H
    S = min(BH, cores) if target_heads is None else min(BH, target_heads)
    b_cnt = (S + s.H - 1) // s.H
    # whole batches keep the [B,H,N,d] layout; trailing heads of the last batch are simply unused
    q, k, v = (t[:b_cnt] for t in (call.q, call.k, call.v))
    import numpy as np
    q64, k64, v64 = (t.double().numpy() for t in (q, k, v))
    w64, b64 = call.dw_weight.double().numpy(), call.dw_bias.double().numpy()
    lib = oracle.load()
    out = np.empty_like(q64)
    import ctypes
    from concurrent.futures import ThreadPoolExecutor
    dp = ctypes.POINTER(ctypes.c_double)
    ptr = lambda a: a.ctypes.data_as(dp)

    def run(i):
        return lib.castling_oracle_forward(ptr(q64), ptr(k64), ptr(v64), ptr(w64), ptr(b64), ptr(out), b_cnt, s.H,
                                           s.gridH, s.gridW, s.d, s.ksize, 1e-12, i, i + 1)
    threads = min(S, cores)
    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=threads) as pool:
        rcs = list(pool.map(run, range(S)))
    dt = time.perf_counter() - t0
    assert not any(rcs)
    tokens = S * s.N / s.H  # image tokens: B*N per forward covers H heads each
    return tokens / dt, threads, f"first {S} of {BH} (b,h) slices of {s.label()}, one thread each, float64", dt


def run_reference(args, rank, world):
    """The reference arm: the CPU oracle, as it stands, on host cores (rank 0 only)."""
    if rank != 0:
        return
    call = pick_call(args.workload)
    s = call.shape
    # one (b,h) slice on one thread, untimed, sizes the per-step sample: the whole run stays
    # near two minutes whatever K is
    _, _, _, t_one = cpu_oracle_rate(call, target_heads=1)
    cores = os.cpu_count() or 1
    steps = max(1, args.steps)
    budget = 120.0
    heads = max(1, min(s.B * s.H, cores, int(budget / (steps * max(t_one, 1e-4)) * cores)))
    if steps * t_one > budget and heads == 1:
        steps = max(1, int(budget / t_one))
    rates, secs = [], 0.0
    threads, sample = 1, ""
    for _ in range(steps):
        r, threads, sample, dt = cpu_oracle_rate(call, target_heads=heads)
        rates.append(r); secs += dt
    value = sum(rates) / len(rates)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": 1e3 * secs / steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{args.workload} {s.label()}", "note": "CPU oracle on a bounded sample per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def main():
    args = parse_args()
    rank, world, local = dist_setup(args.gpus)
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the attention core has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    from paper_2211_10526_b200 import CastlingAttn, binding

    call = pick_call(args.workload, seed_offset=rank)  # each rank: an independent replica
    s = call.shape
    host = [t.pin_memory() for t in (call.q, call.k, call.v, call.dw_weight, call.dw_bias)]
    q, k, v, w, b = (t.to(dev, non_blocking=True) for t in host)
    out = torch.empty_like(q)
    if args.layout == "token_major":  # same values, stored [B,N,H,d]; the library reads them through strides
        q, k, v, out = (t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3) for t in (q, k, v, out))
    attn = CastlingAttn(ksize=s.ksize, force_path=args.force_path)
    stream = torch.cuda.current_stream(dev)
    # A workload that fits in L2 is timed "cold" over a rotating ring of copies of its tensors whose
    # total is three times the L2 size, so that no step finds its inputs cached by the previous one.
    n_sets = 1 if s.algorithmic_bytes > 2 * L2_BYTES else min(512, -(-3 * L2_BYTES // s.algorithmic_bytes))
    ring = [(q, k, v, out)] + [(q.clone(), k.clone(), v.clone(), torch.empty_like(q)) for _ in range(n_sets - 1)]

    def step(i):
        q_, k_, v_, o_ = ring[i % n_sets]
        attn.forward(q_, k_, v_, w, b, s.gridH, s.gridW, out=o_)

    for i in range(max(args.warmup, 3)):
        step(i)
    torch.cuda.synchronize()
    path, launches_per_step = attn.last_path()
    hot_ms = graph_ms = None
    if n_sets > 1:  # the same number of steps on one set: every input served from L2
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0.record(stream)
        for _ in range(args.steps):
            step(0)
        h1.record(stream)
        torch.cuda.synchronize()
        hot_ms = h0.elapsed_time(h1) / args.steps
        # the same, replayed from a CUDA graph of 20 forwards: what is left when the host's launch cost is gone
        graph_ms = None
        try:
            side = torch.cuda.Stream(dev)
            side.wait_stream(stream)
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                for _ in range(20):
                    step(0)
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            graph.replay()
            g0.record(stream)
            for _ in range(max(1, args.steps // 20)):
                graph.replay()
            g1.record(stream)
            torch.cuda.synchronize()
            graph_ms = g0.elapsed_time(g1) / (20 * max(1, args.steps // 20))
        except Exception as exc:  # reported, never fatal: the headline does not depend on it
            graph_ms = f"unavailable: {exc}"
        for i in range(n_sets):  # push that set out of L2 again
            step(i)
        torch.cuda.synchronize()

    # ---- timed region: REPEATS repeats of max(K, MIN_FORWARDS) forwards each, device time between two events
    # on the launching stream, maximum over the ranks per repeat; the median repeat is the reported one.  The
    # clock sampler runs across all repeats.
    n_fwd = max(args.steps, args.min_forwards)
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.25)
    rep_ms = []
    for _ in range(max(1, args.repeats)):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier(world)
        torch.cuda.synchronize()
        e0.record(stream)
        for i in range(n_fwd):
            step(i)
        e1.record(stream)
        torch.cuda.synchronize()
        barrier(world)
        rep_ms.append(max_over_ranks(e0.elapsed_time(e1), world, dev) / n_fwd)
    clocks = sampler.stop()
    rep_sorted = sorted(rep_ms)
    ms_per_step = rep_sorted[len(rep_sorted) // 2]
    value = world * s.image_tokens / (ms_per_step * 1e-3)

    # ---- per-kernel durations: same loop with events between the kernels (not part of `value`) ----
    binding.castling_attn_set_profiling(attn.handle, True)
    acc = {}
    for i in range(min(args.steps, 50)):
        step(i)
        for name, ms in binding.castling_attn_kernel_times(attn.handle):
            acc.setdefault(name, []).append(ms)
    binding.castling_attn_set_profiling(attn.handle, False)
    kernels = {n: sum(v_) / len(v_) for n, v_ in acc.items()}
    peak, peak_src = measured_peak_hbm()
    tensor_bytes = s.B * s.H * s.N * s.d * s.elem_bytes
    # algorithmic bytes per launch: the state kernel must read K and V, the apply kernel must read Q
    # and write O (V's one compulsory read is booked to the state kernel); a single-kernel forward moves
    # all four tensors; the split reduction and the leading-token rows move no algorithmic bytes
    per_kernel = {"tc_state": 2, "tc_apply": 2, "simt_state": 2, "simt_apply": 2, "tc_fused": 4, "simt_fused": 4, "tc_pipe": 4}
    alg = {n: per_kernel.get(n, 0) * tensor_bytes for n in kernels}
    top = max(kernels, key=kernels.get) if kernels else None
    roofline = None
    if top is not None:
        achieved = alg[top] / (kernels[top] * 1e-3) / 1e9
        path_gbs = s.algorithmic_bytes / (ms_per_step * 1e-3) / 1e9
        traffic, traffic_src = ncu_traffic(args.workload, top)
        roofline = {"bound": "hbm", "kernel": top, "achieved": achieved, "peak": peak, "unit": "GB/s",
                    "frac": achieved / peak, "traffic": traffic, "traffic_source": traffic_src,
                    "traffic_unit": "bytes per launch, ncu", "peak_source": peak_src,
                    "kernel_ms": kernels, "path_achieved": path_gbs, "path_frac": path_gbs / peak,
                    "path_frac_of_8000": path_gbs / 8000.0}

    # ---- end to end through the host-buffer entry point (pinned memory, copies inside the timing) ----
    e2e = None
    if not args.no_e2e:
        out_h = torch.empty_like(call.q).pin_memory()
        n_e2e = max(3, min(args.steps, 20))
        for _ in range(2):
            attn.forward_host(*host, s.gridH, s.gridW, out=out_h, stream=stream.cuda_stream)
        barrier(world)
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            attn.forward_host(*host, s.gridH, s.gridW, out=out_h, stream=stream.cuda_stream)
        dt = max_over_ranks(time.perf_counter() - t0, world, dev)
        # the end-to-end result against the device-path result of the same inputs (the chunked pipeline splits
        # the token sums differently, so the two agree to rounding, not bit for bit)
        step(0)
        torch.cuda.synchronize()
        ref_o = ring[0][3].float().cpu()
        e2e_err = float((out_h.float() - ref_o).abs().max() / ref_o.abs().max().clamp_min(1e-30))
        if not e2e_err <= (2e-2 if s.dtype == "bf16" else 1e-5):
            raise SystemExit(f"end-to-end output differs from the device-path output: max-rel {e2e_err:.3e}")
        h2d = sum(t.numel() * t.element_size() for t in host)
        e2e = {"value": world * s.image_tokens * n_e2e / dt, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": out_h.numel() * out_h.element_size(), "steps": n_e2e,
               "ms_per_step": 1e3 * dt / n_e2e, "max_rel_diff_vs_device_path": e2e_err}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        r, threads, sample, _ = cpu_oracle_rate(call)
        cpu = {"value": r, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if s.dtype == "bf16" else "f32",
            "data": "synthetic",
            "config": {"workload": f"{args.workload} {s.label()}", "tokens_per_step": s.image_tokens,
                       "head_tokens_per_step": s.head_tokens, "algorithmic_bytes_per_step": s.algorithmic_bytes,
                       "l2": "inputs exceed L2, no flush" if n_sets == 1 else
                             f"cold: ring of {n_sets} copies of q, k, v, out ({n_sets * s.algorithmic_bytes / 1e6:.0f} MB) cycled",
                       "hot_ms_per_step": hot_ms, "hot_graph_replay_ms_per_step": graph_ms,
                       "layout": "[B,H,N,d]" if args.layout == "head_major" else "[B,N,H,d] (strided views)",
                       "parallelism": "independent replicas" if world > 1 else "single GPU",
                       "arithmetic": "bf16 tensor-core operands, fp32 accumulation" if s.dtype == "bf16" else "fp32",
                       "kernel_path": {1: "cuda-core", 2: "tensor-core"}.get(path, str(path))},
            "timing": {"repeats": len(rep_ms), "forwards_per_repeat": n_fwd, "ms_per_step_min": rep_sorted[0],
                       "ms_per_step_median": ms_per_step, "ms_per_step_max": rep_sorted[-1]},
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * n_fwd * len(rep_ms),
            "roofline": roofline, "cpu_baseline": cpu,
        }
        print(json.dumps(line), flush=True)
    attn.close()
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
