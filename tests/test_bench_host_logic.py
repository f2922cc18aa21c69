"""CPU tests of bench.py's host logic, including the multi-rank path on gloo (world size 2)."""
from __future__ import annotations

import json
import os
import socket
import subprocess
import sys
import textwrap

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _spawn_ranks(code: str, world: int = 2, extra_env=None):
    port = _free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), PYTHONPATH=ROOT, CUDA_VISIBLE_DEVICES="")
        env.update(extra_env or {})
        procs.append(subprocess.Popen([sys.executable, "-c", code], env=env, cwd=ROOT, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=240) for p in procs]
    for p, (so, se) in zip(procs, outs):
        assert p.returncode == 0, se[-2000:]
    return [so for so, _ in outs]


def test_max_over_ranks_and_barrier_on_gloo_world_size_2():
    code = textwrap.dedent("""
        import torch, bench
        rank, world, local = bench.dist_setup(2)
        assert world == 2 and rank == local
        bench.barrier(world)
        t = bench.max_over_ranks(10.0 + 5.0 * rank, world, torch.device("cpu"))
        assert t == 15.0, t
        # replicas: each rank draws its own copy of the workload (seed offset = rank), same shape
        call = bench.pick_call("c1_fp32_tiny", seed_offset=rank)
        s = torch.tensor([float(call.q.double().sum())], dtype=torch.float64)
        import torch.distributed as dist
        both = [torch.zeros_like(s) for _ in range(world)]
        dist.all_gather(both, s)
        assert both[0].item() != both[1].item()
        # whole-job value: tokens of all ranks over the slowest rank's time
        ms = bench.max_over_ranks(1.0 + rank, world, torch.device("cpu"))
        value = world * call.shape.image_tokens / (ms * 1e-3)
        assert abs(value - 2 * 392 / 2e-3) < 1e-6
        bench.barrier(world)
        dist.destroy_process_group()
        print("ok", rank)
    """)
    outs = _spawn_ranks(code)
    assert sorted(o.strip() for o in outs) == ["ok 0", "ok 1"]


def test_reference_arm_prints_on_rank_zero_only():
    code = "import sys; sys.argv=['bench.py','--impl','reference','--gpus','2','--steps','2','--warmup','1','--workload','c1_fp32_tiny']; import bench; bench.main()"
    outs = _spawn_ranks(code)
    lines = [o.strip() for o in outs if o.strip()]
    assert len(lines) == 1
    j = json.loads(lines[0])
    assert j["impl"] == "reference" and j["cpu_baseline"]["kind"] == "oracle" and j["value"] > 0
    assert j["e2e"]["h2d_bytes_per_step"] == 0 and j["unit"] == "tokens/s" and j["gpu_launches"] == 0


def test_clock_sampler_parsing():
    import bench
    cs = bench.ClockSampler(0)
    cs.proc = object()  # parsing only: pretend the sampler ran
    cs.lines = ["1965, 1965, 512.3, Not Active, Not Active, Not Active, Active",
                "1800, 1965, 950.1, Not Active, Not Active, Not Active, Not Active", "garbage"]

    class _P:
        def terminate(self): pass
        def wait(self, timeout=None): return 0
        def kill(self): pass
    cs.proc = _P()
    out = cs.stop()
    assert out["sm_max_mhz"] == 1965.0 and out["samples"] == 2 and out["reasons"] == ["sw_power_cap"]
    assert out["sm_mhz"] in (1800.0, 1965.0)


def test_pick_call_and_peak_lookup():
    import bench
    c = bench.pick_call("c5_sweep_bf16:1")
    assert tuple(c.q.shape) == (2, 8, 4096, 64) and c.q.dtype == torch.bfloat16
    peak, src = bench.measured_peak_hbm()
    assert peak > 1000 and src in ("measured", "fallback")


def test_bench_refuses_to_run_without_a_gpu():
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="", PYTHONPATH=ROOT)
    p = subprocess.run([sys.executable, "bench.py", "--steps", "1", "--warmup", "1", "--workload", "c1_fp32_tiny"],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=240)
    assert p.returncode != 0 and "no CPU path" in (p.stderr + p.stdout)
