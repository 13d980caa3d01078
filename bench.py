#!/usr/bin/env python
"""Benchmark of the ternary-weight hot path on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints ONE JSON line (rank 0).  A step is one pass of the workload's whole hot
path over one batch of seeded synthetic input.  Device timing uses CUDA events on
the launching stream; for N > 1 every rank runs an independent replica (the path
has no exchange step) and the slowest rank's time is used.

`--impl reference` times the CPU oracle (oracle/) on a bounded sample of the same
workload on the host cores; it is a deliberately slow baseline, not a target.
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
sys.path.insert(0, ROOT)


# ------------------------------------------------------------------ utilities
def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-i", str(self.index), "-lms", "100"], stdout=subprocess.PIPE, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.t.join(timeout=2)
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx = float(r[1])
            except (ValueError, IndexError):
                continue
            for nm, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(sm)}


def dist_env():
    return (int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)),
            int(os.environ.get("WORLD_SIZE", 1)))


# ------------------------------------------------------------------ workloads
class TernarizeWorkload:
    """Ternarize + 2-bit pack of one fp32 tensor of n weights drawn N(0,1):
    threshold reduction, Eq. 3 codes, Eq. 5 scale, packing.  8.25 algorithmic
    bytes per weight (two reads of 4 B: the threshold needs every weight before
    any code can be emitted; 0.25 B written)."""
    name = "ternarize_pack_n1e8_normal"
    metric = "ternarize+pack GB/s"
    unit = "GB/s"
    dtype = "f64"
    bytes_per_unit = 8.25
    launches_per_step = 2

    def __init__(self, n=100_000_000, seed=0):
        self.n, self.seed = n, seed

    def config(self):
        return {"workload": self.name, "n": self.n, "dist": "normal", "seed": self.seed,
                "delta_factor": 0.7, "l2": "input (400 MB) larger than L2 (126 MB)"}

    def host_inputs(self):
        from paper_1605_04711_b200 import datagen as dg
        return dg.draw(self.seed, "sweep-normal", self.n, "normal")

    def setup(self, torch, twn, host_W):
        self.torch, self.twn = torch, twn
        self.ld = twn.ld_for(self.n)
        self.W = torch.from_numpy(host_W).cuda()
        self.stats = twn.new_stats()
        self.packed = torch.empty(self.ld // 16, dtype=torch.int32, device="cuda")
        self.ws = torch.empty(twn.ternarize_workspace_bytes(), dtype=torch.uint8, device="cuda")
        self.host_W = torch.from_numpy(host_W).pin_memory()
        self.host_packed = torch.empty(self.ld // 16, dtype=torch.int32).pin_memory()
        self.host_stats = torch.empty(8, dtype=torch.int64).pin_memory()

    def step(self):
        self.twn.ternarize(self.W, 0.7, self.stats, self.packed, self.ld, None, self.ws,
                           rows=1, cols=self.n)

    def step_e2e(self):
        self.W.copy_(self.host_W, non_blocking=True)
        self.step()
        self.host_packed.copy_(self.packed, non_blocking=True)
        self.host_stats.copy_(self.stats, non_blocking=True)

    def e2e_bytes(self):
        return self.n * 4, self.ld // 4 + 64

    def units_per_step(self):
        return self.n * self.bytes_per_unit / 1e9  # GB of algorithmic traffic

    def roofline(self, ms_per_step, peaks):
        ach = self.n * self.bytes_per_unit / (ms_per_step * 1e-3) / 1e9
        return {"bound": "hbm", "kernel": "sum_abs_kernel + code_pack_kernel (one twn_ternarize call)",
                "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": ach / peaks["hbm_gbs"], "peak_source": peaks["source"],
                "frac_of_nominal_8TBs": ach / 8000.0, "traffic": None}

    def check(self):
        st = self.twn.stats_to_host(self.stats)
        assert st["status"] == 0 and st["n_neg"] + st["n_zero"] + st["n_pos"] == self.n, st

    # CPU oracle on the same tensor (full size: about a second per pass)
    def cpu_sample(self, host_W):
        import oracle
        t0 = time.perf_counter()
        st, codes = oracle.ternarize(host_W, 0.7)
        oracle.pack(codes, self.ld)
        dt = time.perf_counter() - t0
        return self.n * self.bytes_per_unit / dt / 1e9, f"full tensor, n={self.n}", 1


WORKLOADS = {"ternarize": TernarizeWorkload}
DEFAULT_WORKLOAD = "ternarize"


# ------------------------------------------------------------------ arms
def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    wl = WORKLOADS[args.workload]()
    host = wl.host_inputs()
    vals = []
    for i in range(args.warmup + args.steps):
        v, sample, cores = wl.cpu_sample(host)
        if i >= args.warmup:
            vals.append(v)
    value = sum(vals) / len(vals)
    line = {"impl": "reference", "metric": wl.metric, "value": value, "unit": wl.unit,
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": wl.units_per_step() / value * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": wl.config(), "gpu_launches": 0,
            "cpu_baseline": {"value": value, "unit": wl.unit, "cores": cores, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": wl.unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def run_ours(args):
    import torch
    from paper_1605_04711_b200 import twn
    twn.lib()  # fails loudly when the CUDA library is missing
    rank, local_rank, world = dist_env()
    torch.cuda.set_device(local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    wl = WORKLOADS[args.workload]()
    host = wl.host_inputs()
    wl.setup(torch, twn, host)
    peaks = measured_peaks()

    def timed(fn, steps, warmup):
        for _ in range(warmup):
            fn()
        barrier()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for _ in range(steps):
            fn()
        ev1.record()
        barrier()
        ms = ev0.elapsed_time(ev1)
        if world > 1:
            t = torch.tensor([ms], device="cuda", dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        return ms / steps

    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.start()
    ms = timed(wl.step, args.steps, max(args.warmup, 3))
    clocks = sampler.stop() if sampler else None
    wl.check()
    ms_e2e = timed(wl.step_e2e, max(2, min(args.steps, 5)), 1)
    wl.check()

    if rank == 0:
        h2d, d2h = wl.e2e_bytes()
        line = {"metric": wl.metric, "value": world * wl.units_per_step() / (ms * 1e-3),
                "unit": wl.unit, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
                "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": wl.dtype, "data": "synthetic", "config": wl.config(), "clocks": clocks,
                "e2e": {"value": world * wl.units_per_step() / (ms_e2e * 1e-3), "unit": wl.unit,
                        "ms_per_step": ms_e2e, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
                "gpu_launches": wl.launches_per_step * args.steps,
                "roofline": wl.roofline(ms, peaks)}
        if world == 1 and not args.no_cpu:
            v, sample, cores = wl.cpu_sample(host)
            line["cpu_baseline"] = {"value": v, "unit": wl.unit, "cores": cores, "kind": "oracle",
                                    "sample": sample}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
