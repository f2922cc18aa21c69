#!/usr/bin/env python
"""Benchmark of the linear-angular attention core.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME[:IDX]] [--impl ours|reference]

A step is one forward pass of the whole attention core (state build, reduction, apply +
depthwise convolution) over one synthetic batch.  The default workload is the largest
long-sequence sweep point (B=2, H=8, 256x256 tokens, d=64, bf16): its four tensors
(537 MB) exceed the 126 MB L2, so every step streams from HBM and no L2 flush is needed.
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
FALLBACK_HBM_GBS = 6650.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, help="workload name[:call index]")
    ap.add_argument("--force-path", type=int, default=0, help="0 auto, 1 CUDA-core kernels, 2 tensor-core kernels")
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
