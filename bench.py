#!/usr/bin/env python
"""Benchmark of the ternary-weight hot path on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints ONE JSON line (rank 0).  A step is one pass of the workload's whole hot path over one
batch of seeded synthetic input.  The default workload is the ResNet-18-shaped training step
(batch 64, 3x224x224): ternarize + pack every layer, forward through the ternary convolutions,
backward for data through the transposed codes, straight-through weight gradients.  Device
timing uses CUDA events on the launching stream; for N > 1 every rank runs an independent
replica (the path has no exchange step) and the slowest rank's time is used.

`--impl reference` times the CPU oracle (oracle/) on a bounded sample of the same workload on
the host cores; it is a deliberately slow baseline, not a target.
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
    """Samples the SM clock and the clock event reasons of one GPU while the timed region runs: through NVML
    from a thread every 2 ms (a timed region of a few tens of milliseconds still gets samples), else with an
    nvidia-smi loop.  Reads only; no setting of the GPU is touched."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int, uuid: str = ""):
        self.index, self.uuid, self.rows, self.proc, self.nvml = index, uuid, [], None, None
        self.first, self.halt, self.max_mhz = 0, threading.Event(), None

    def _nvml_handle(self):
        import pynvml
        pynvml.nvmlInit()
        if self.uuid:
            try:
                return pynvml, pynvml.nvmlDeviceGetHandleByUUID(self.uuid if self.uuid.startswith("GPU-") else "GPU-" + self.uuid)
            except pynvml.NVMLError:
                pass
        return pynvml, pynvml.nvmlDeviceGetHandleByIndex(self.index)

    def start(self):
        try:
            self.nvml, self.handle = self._nvml_handle()
            self.max_mhz = float(self.nvml.nvmlDeviceGetMaxClockInfo(self.handle, self.nvml.NVML_CLOCK_SM))
            self.source = "nvml, every 2 ms"
            self.t = threading.Thread(target=self._poll, daemon=True)
            self.t.start()
            time.sleep(0.05)
            self.first = len(self.rows)
            return
        except Exception:                     # no NVML binding or no permission: the nvidia-smi loop
            self.nvml = None
        try:
            self.source = "nvidia-smi -lms 50"
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-i", str(self.index), "-lms", "50"], stdout=subprocess.PIPE, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
            time.sleep(0.5)          # let the sampler come up before the timed region starts
            self.first = len(self.rows)
        except OSError:
            self.proc = None

    def _poll(self):
        n = self.nvml
        bits = [(n.nvmlClocksEventReasonHwSlowdown, "hw_slowdown"), (n.nvmlClocksEventReasonHwThermalSlowdown, "hw_thermal_slowdown"),
                (n.nvmlClocksEventReasonSwThermalSlowdown, "sw_thermal_slowdown"), (n.nvmlClocksEventReasonSwPowerCap, "sw_power_cap")]
        while not self.halt.is_set():
            try:
                mhz = n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM)
                r = n.nvmlDeviceGetCurrentClocksEventReasons(self.handle)
                self.rows.append([str(mhz), str(self.max_mhz)] + ["Active" if r & b else "Not Active" for b, _ in bits])
            except Exception:
                pass
            time.sleep(0.002)

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.nvml is not None:
            self.halt.set()
            self.t.join(timeout=2)
        elif self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
            self.t.join(timeout=2)
        else:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no NVML binding and no nvidia-smi"]}
        sm, mx, reasons = [], None, set()
        for r in self.rows[self.first:]:
            try:
                sm.append(float(r[0])); mx = float(r[1])
            except (ValueError, IndexError):
                continue
            for nm, v in zip(self.NAMES, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        lo = min(sm) if sm else None
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_min_mhz": lo, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(sm), "source": self.source}


def max_over_ranks(ms: float, world: int, dist=None, device=None) -> float:
    """Replicas are independent; the step time of the job is the slowest rank's."""
    if world <= 1:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def dist_env():
    return (int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)),
            int(os.environ.get("WORLD_SIZE", 1)))


# ------------------------------------------------------------------ workloads
class TernarizeWorkload:
    """Ternarize + 2-bit pack of one fp32 tensor of n weights drawn N(0,1): threshold
    reduction, Eq. 3 codes, Eq. 5 scale, packing.  8.25 algorithmic bytes per weight (two
    reads of 4 B: the threshold needs every weight before any code can be emitted; 0.25 B
    written)."""
    name = "ternarize_pack_n1e8_normal"
    metric = "ternarize+pack GB/s"
    unit = "GB/s"
    dtype = "f64"
    bytes_per_unit = 8.25
    default_steps = 2000

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

    def launches_per_step(self):
        return 2

    def units_per_step(self):
        return self.n * self.bytes_per_unit / 1e9  # GB of algorithmic traffic

    def roofline(self, ms_per_step, peaks):
        ach = self.n * self.bytes_per_unit / (ms_per_step * 1e-3) / 1e9
        return {"bound": "hbm", "kernel": "sum_abs_kernel + code_pack_kernel (one twn_ternarize call)",
                "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": ach / peaks["hbm_gbs"], "peak_source": peaks["source"],
                "frac_of_nominal_8TBs": ach / 8000.0,
                # dram__bytes_read.sum + dram__bytes_write.sum of the two kernels of one call (ncu capture of
                # this workload, summarised under profiles/); algorithmic: 8.25e8
                "traffic": 819.6e6 if self.n == 100_000_000 else None}

    def check(self):
        st = self.twn.stats_to_host(self.stats)
        assert st["status"] == 0 and st["n_neg"] + st["n_zero"] + st["n_pos"] == self.n, st

    def cpu_sample(self, host_W):
        import oracle
        t0 = time.perf_counter()
        st, codes = oracle.ternarize(host_W, 0.7)
        oracle.pack(codes, self.ld)
        dt = time.perf_counter() - t0
        return self.n * self.bytes_per_unit / dt / 1e9, f"full tensor, n={self.n}", 1


class TernarizeRowsWorkload(TernarizeWorkload):
    """Per-filter ternarize + pack (Algorithm 1 as printed: one threshold and one scale per filter)
    of a [rows, cols] fp32 matrix drawn N(0,1).  A filter stays on chip between the threshold
    reduction and the coding, so the algorithmic traffic is 4.25 bytes per weight (one read,
    0.25 B written)."""
    name = "ternarize_rows_pack_12288x8192_normal"
    bytes_per_unit = 4.25

    def __init__(self, rows=12288, cols=8192, seed=0):
        super().__init__(rows * cols, seed)
        self.rows, self.cols = rows, cols

    def config(self):
        return {"workload": self.name, "rows": self.rows, "cols": self.cols, "dist": "normal", "seed": self.seed,
                "delta_factor": 0.7, "l2": "input (403 MB) larger than L2 (126 MB)"}

    def setup(self, torch, twn, host_W):
        self.torch, self.twn = torch, twn
        self.ld = twn.ld_for(self.cols)
        self.W = torch.from_numpy(host_W).cuda().view(self.rows, self.cols)
        self.stats = twn.new_stats_rows(self.rows)
        self.packed = torch.empty((self.rows, self.ld // 16), dtype=torch.int32, device="cuda")
        self.host_W = torch.from_numpy(host_W).pin_memory().view(self.rows, self.cols)
        self.host_packed = torch.empty((self.rows, self.ld // 16), dtype=torch.int32).pin_memory()
        self.host_stats = torch.empty((self.rows, 8), dtype=torch.int64).pin_memory()

    def step(self):
        self.twn.ternarize_rows(self.W, 0.7, self.stats, self.packed, self.ld)

    def e2e_bytes(self):
        return self.n * 4, self.rows * (self.ld // 4 + 64)

    def launches_per_step(self):
        return 1

    def roofline(self, ms_per_step, peaks):
        r = super().roofline(ms_per_step, peaks)
        r["kernel"] = "ternarize_rows_kernel (one twn_ternarize_rows call)"
        # dram bytes of one launch from the ncu capture of this workload (profiles/); algorithmic: 4.28e8
        r["traffic"] = 427.7e6 if (self.rows, self.cols) == (12288, 8192) else None
        return r

    def check(self):
        st = self.twn.stats_rows_to_host(self.stats[:4])
        assert all(s["status"] == 0 and s["n_neg"] + s["n_zero"] + s["n_pos"] == self.cols for s in st), st

    def cpu_sample(self, host_W):
        import oracle
        rows = 1536          # a bounded sample of the filters (about 10 s of the oracle)
        W = host_W.reshape(self.rows, self.cols)[:rows]
        t0 = time.perf_counter()
        st, codes = oracle.ternarize_rows(W, 0.7)
        oracle.pack(codes, self.ld)
        dt = time.perf_counter() - t0
        return rows * self.cols * self.bytes_per_unit / dt / 1e9, f"oracle on {rows} of {self.rows} filters ({dt:.1f} s)", 1


class BinarizeWorkload(TernarizeWorkload):
    """Binary precision weights (the paper's BPWN baseline, Sec. 3): sign codes, alpha = mean |W|, 1-bit packing of
    one fp32 tensor of 1e8 weights drawn N(0,1).  No threshold is needed, so one sweep: 4 bytes read and 1/32 byte
    written per weight."""
    name = "binarize_pack_n1e8_normal"
    metric = "binarize+pack GB/s"
    bytes_per_unit = 4.03125

    def __init__(self, n=100_000_000 // 128 * 128, seed=0):
        super().__init__(n, seed)

    def config(self):
        c = super().config()
        c.pop("delta_factor", None)
        return c

    def setup(self, torch, twn, host_W):
        self.torch, self.twn = torch, twn
        self.ld = twn.ld_for_b1(self.n)
        self.W = torch.from_numpy(host_W).cuda()
        self.stats = twn.new_stats()
        self.packed = torch.empty(self.ld // 32, dtype=torch.int32, device="cuda")
        self.ws = torch.empty(twn.binarize_workspace_bytes(), dtype=torch.uint8, device="cuda")
        self.host_W = torch.from_numpy(host_W).pin_memory()
        self.host_packed = torch.empty(self.ld // 32, dtype=torch.int32).pin_memory()
        self.host_stats = torch.empty(8, dtype=torch.int64).pin_memory()

    def step(self):
        self.twn.binarize(self.W, self.stats, self.packed, self.ld, self.ws, rows=1, cols=self.n)

    def e2e_bytes(self):
        return self.n * 4, self.ld // 8 + 64

    def launches_per_step(self):
        return 1

    def roofline(self, ms_per_step, peaks):
        r = super().roofline(ms_per_step, peaks)
        r["kernel"] = "binarize_kernel (one twn_binarize call)"
        r["traffic"] = None
        return r

    def cpu_sample(self, host_W):
        import oracle
        t0 = time.perf_counter()
        st, codes = oracle.binarize(host_W)
        oracle.pack1(codes, self.ld)
        dt = time.perf_counter() - t0
        return self.n * self.bytes_per_unit / dt / 1e9, f"full tensor, n={self.n}", 1


class SgdTernarizeWorkload(TernarizeWorkload):
    """End of one iteration and start of the next (Algorithm 1): SGD-with-momentum update of 1e8 fp32
    master weights fused with the threshold reduction of the updated weights, then the coding sweep
    (codes, 2-bit packing, scale).  Algorithmic bytes per weight: update 12 read (W, dW, V) + 8 written
    (W, V), coding 4 read + 0.25 written = 24.25; the unfused sequence reads the weights once more."""
    name = "sgd_update_ternarize_n1e8_normal"
    metric = "sgd update + ternarize+pack GB/s"
    bytes_per_unit = 24.25

    def config(self):
        c = super().config()
        c.update({"workload": self.name, "lr": 0.01, "momentum": 0.9, "weight_decay": 1e-4,
                  "l2": "W, dW, V (1.2 GB) larger than L2 (126 MB)"})
        return c

    def setup(self, torch, twn, host_W):
        from paper_1605_04711_b200 import datagen as dg
        super().setup(torch, twn, host_W)
        self.dW = torch.from_numpy(dg.draw(self.seed, "sweep-grad", self.n, "normal", 0.0, 0.01)).cuda()
        self.V = torch.zeros(self.n, dtype=torch.float32, device="cuda")

    def step(self):
        self.twn.sgd_update(self.W, self.dW, self.V, 0.01, 0.9, 1e-4, 0.7, self.stats, self.ws)
        self.twn.ternarize_codes(self.W, 1, self.n, self.stats, self.packed, self.ld, None, self.ws)

    def step_e2e(self):
        self.dW.copy_(self.host_W, non_blocking=True)       # a gradient-sized tensor arrives from the host
        self.step()
        self.host_packed.copy_(self.packed, non_blocking=True)
        self.host_stats.copy_(self.stats, non_blocking=True)

    def roofline(self, ms_per_step, peaks):
        r = super().roofline(ms_per_step, peaks)
        r["kernel"] = "sgd_update_kernel + code_pack_kernel (twn_sgd_update, twn_ternarize_codes)"
        r["traffic"] = None
        return r

    def cpu_sample(self, host_W):
        import oracle
        import numpy as np
        n = self.n
        W = host_W[:n]
        g = np.full(n, 0.01, np.float32)
        t0 = time.perf_counter()
        w1, v1 = oracle.sgd_update(W, g, np.zeros(n, np.float32), 0.01, 0.9, 1e-4)
        st, codes = oracle.ternarize(w1, 0.7)
        oracle.pack(codes, oracle.ld_for(n))
        dt = time.perf_counter() - t0
        return n * self.bytes_per_unit / dt / 1e9, f"oracle on all {n} weights ({dt:.1f} s)", 1


class GemmWorkload:
    """One ternary-weight GEMM (Algorithm 1, forward of a fully connected layer): Y = alpha * X T^T with
    bf16 X [M, K], 2-bit T [N, K] ternarized from N(0,1) weights, bf16 Y.  2MNK flops per step."""
    metric = "ternary GEMM TFLOP/s"
    unit = "TFLOP/s"
    dtype = "bf16"
    default_steps = 200

    def __init__(self, M, N=4096, K=4096, seed=0):
        self.M, self.N, self.K, self.seed = M, N, K, seed
        self.name = f"ternary_gemm_m{M}_n{N}_k{K}"

    def config(self):
        mb = (2 * self.M * self.K + 2 * self.M * self.N) / 1e6
        return {"workload": self.name, "seed": self.seed, "delta_factor": 0.7,
                "l2": f"X and Y of a step: {mb:.0f} MB" + (" (larger than L2)" if mb > 126 else " (fits L2: weights and X stay resident, as in a served layer)")}

    def host_inputs(self):
        from paper_1605_04711_b200 import datagen as dg
        return (dg.draw(self.seed, "gemm.w", self.N * self.K, "normal").reshape(self.N, self.K),
                dg.draw_bf16(self.seed, "gemm.x", self.M * self.K, "normal").reshape(self.M, self.K))

    def setup(self, torch, twn, host):
        import numpy as np
        self.torch, self.twn = torch, twn
        Wm, X = host
        self.ld = twn.ld_for(self.K)
        self.stats = twn.new_stats()
        self.packed = torch.empty((self.N, self.ld // 16), dtype=torch.int32, device="cuda")
        ws = torch.empty(twn.ternarize_workspace_bytes(), dtype=torch.uint8, device="cuda")
        twn.ternarize(torch.from_numpy(Wm).cuda(), 0.7, self.stats, self.packed, self.ld, None, ws,
                      rows=self.N, cols=self.K)
        self.host_x = torch.from_numpy(X.view(np.int16)).pin_memory()
        self.X = self.host_x.cuda().view(torch.bfloat16)
        self.Y = torch.empty((self.M, self.N), dtype=torch.bfloat16, device="cuda")
        self.host_y = torch.empty((self.M, self.N), dtype=torch.int16).pin_memory()
        self.epi = twn.epilogue(out_dtype=twn.BF16)
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def step(self):
        self.twn.gemm(self.X, self.K, self.packed, self.ld, self.stats, self.M, self.N, self.K, self.epi,
                      self.Y, self.N, self.status)

    def step_e2e(self):
        self.X.view(self.torch.int16).copy_(self.host_x, non_blocking=True)
        self.step()
        self.host_y.copy_(self.Y.view(self.torch.int16), non_blocking=True)

    def e2e_bytes(self):
        return self.M * self.K * 2, self.M * self.N * 2

    def launches_per_step(self):
        return 1

    def units_per_step(self):
        return 2.0 * self.M * self.N * self.K / 1e12

    def roofline(self, ms_per_step, peaks):
        ach = self.units_per_step() / (ms_per_step * 1e-3)
        return {"bound": "tensor", "kernel": "tconv_kernel (one twn_gemm call)", "achieved": ach,
                "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": ach / peaks["bf16_tflops"],
                "peak_source": peaks["source"] + " (bf16 burst: the kernel is timed alone)",
                # DRAM bytes of one launch from the ncu capture of the M = 4096 case (profiles/)
                "traffic": 40.6e6 if (self.M, self.N, self.K) == (4096, 4096, 4096) else None}

    def check(self):
        assert self.twn.read_status(self.status) == 0
        assert bool(self.torch.isfinite(self.Y[:64].float()).all())

    def cpu_sample(self, host, seconds=10.0):
        import oracle
        Wm, X = host
        st, codes = oracle.ternarize(Wm, 0.7)
        rows = 8
        while True:
            t0 = time.perf_counter()
            oracle.gemm(X[:rows], codes, st.alpha)
            dt = time.perf_counter() - t0
            if dt >= seconds * 0.5 or rows >= self.M:
                break
            rows = int(min(self.M, max(rows * 2, rows * seconds / max(dt, 1e-3))))
        return 2.0 * rows * self.N * self.K / dt / 1e12, f"oracle gemm on {rows} of {self.M} rows ({dt:.1f} s)", oracle.num_threads()


def flush_l2(torch, _cache={}):
    """Writes a buffer larger than L2 (126 MB) so that the next launch starts cold."""
    if "buf" not in _cache:
        _cache["buf"] = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    _cache["buf"].fill_(1)


def time_cold(torch, fn, reps=20, warm=3):
    """Median and minimum (microseconds) of `reps` single launches, each after an L2 flush."""
    for _ in range(warm):
        fn()
    us = []
    for _ in range(reps):
        flush_l2(torch)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); fn(); e1.record()
        e1.synchronize()
        us.append(e0.elapsed_time(e1) * 1e3)
    us.sort()
    return us[len(us) // 2], us[0]


def bound_of(flops, nbytes, peaks):
    """Roofline of one launch timed alone: the slower of its flops at the measured bf16 burst peak and
    its algorithmic bytes at the measured copy bandwidth.  Returns (kind, microseconds)."""
    t_tensor = flops / (peaks["bf16_tflops"] * 1e12) * 1e6
    t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9) * 1e6
    return ("tensor", t_tensor) if t_tensor >= t_hbm else ("hbm", t_hbm)


SWEEP_KN = [(512, 512), (1152, 128), (2304, 256), (4608, 512), (4096, 4096)]
SWEEP_M = [128, 1024, 4096, 16384]
# the shapes the 60 % target is stated for
SWEEP_GATED = [(4096, 4608, 512), (16384, 4608, 512), (4096, 4096, 4096), (16384, 4096, 4096), (16384, 2304, 256)]


class GemmSweepWorkload:
    """The ternary-weight GEMM sweep Y = alpha * X T^T (Eq. 2, inner-product form): bf16 X [M, K] drawn N(0,1),
    T [N, K] ternarized from He-normal weights and 2-bit packed, fp32 Y, for M in {128, 1024, 4096, 16384} and
    (K, N) in {(512,512), (1152,128), (2304,256), (4608,512), (4096,4096)}.  A step is one pass over the 20
    shapes.  Algorithmic bytes of a shape: 2MK (X) + KN/4 (codes) + 4MN (Y); flops 2MKN."""
    name = "ternary_gemm_sweep_fp32_out"
    metric = "ternary GEMM TFLOP/s"
    unit = "TFLOP/s"
    dtype = "bf16"
    default_steps = 20

    def config(self):
        return {"workload": self.name, "seed": 0, "delta_factor": 0.7, "shapes": 20, "out_dtype": "f32",
                "l2": "per-shape times: L2 flushed (256 MB written) before every timed launch; "
                      "the sweep's step time: 20 shapes back to back, 2.4 GB of operands per pass"}

    def host_inputs(self):
        from paper_1605_04711_b200 import datagen as dg
        w = {(K, N): dg.he_normal(0, f"sweep{N}x{K}", N, K) for K, N in SWEEP_KN}
        x = {(M, K): dg.draw_bf16(1, f"sweepx{M}x{K}", M * K, "normal").reshape(M, K)
             for M in SWEEP_M for K in sorted({k for k, _ in SWEEP_KN})}
        return w, x

    def setup(self, torch, twn, host):
        import numpy as np
        self.torch, self.twn = torch, twn
        w, x = host
        ws = torch.empty(twn.ternarize_workspace_bytes(), dtype=torch.uint8, device="cuda")
        self.layers, self.X, self.cases = {}, {}, []
        for (K, N), Wm in w.items():
            ld = twn.ld_for(K)
            stats = twn.new_stats()
            packed = torch.empty((N, ld // 16), dtype=torch.int32, device="cuda")
            twn.ternarize(torch.from_numpy(Wm).cuda(), 0.7, stats, packed, ld, None, ws, rows=N, cols=K)
            self.layers[(K, N)] = (packed, ld, stats)
        for (M, K), xb in x.items():
            self.X[(M, K)] = torch.from_numpy(xb.view(np.int16)).cuda().view(torch.bfloat16)
        self.Y = torch.empty(16384 * 4096, dtype=torch.float32, device="cuda")
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")
        for K, N in SWEEP_KN:
            for M in SWEEP_M:
                self.cases.append((M, K, N))
        self.host_x = torch.empty(16384 * 4608, dtype=torch.int16).pin_memory()
        self.host_y = torch.empty(16384 * 4096, dtype=torch.float32).pin_memory()

    def _run(self, M, K, N):
        packed, ld, stats = self.layers[(K, N)]
        self.twn.gemm(self.X[(M, K)], K, packed, ld, stats, M, N, K, None, self.Y[:M * N].view(M, N), N, self.status)

    def step(self):
        for c in self.cases:
            self._run(*c)

    def step_e2e(self):
        t = self.torch
        for M, K, N in self.cases:
            self.X[(M, K)].view(t.int16).view(-1).copy_(self.host_x[:M * K], non_blocking=True)
            self._run(M, K, N)
            self.host_y[:M * N].copy_(self.Y[:M * N], non_blocking=True)

    def e2e_bytes(self):
        return sum(2 * M * K for M, K, N in self.cases), sum(4 * M * N for M, K, N in self.cases)

    def launches_per_step(self):
        return len(self.cases)

    def units_per_step(self):
        return sum(2.0 * M * K * N for M, K, N in self.cases) / 1e12

    def roofline(self, ms_per_step, peaks):
        shapes, worst = [], None
        for M, K, N in self.cases:
            med, mn = time_cold(self.torch, lambda: self._run(M, K, N))
            flops, nbytes = 2.0 * M * K * N, 2.0 * M * K + K * N / 4.0 + 4.0 * M * N
            kind, t_us = bound_of(flops, nbytes, peaks)
            row = {"M": M, "K": K, "N": N, "us_median": round(med, 2), "us_min": round(mn, 2), "bound": kind,
                   "bound_us": round(t_us, 2), "frac": round(t_us / med, 3), "tflops": round(flops / med / 1e6, 1),
                   "gbs": round(nbytes / med / 1e3, 1), "gated": (M, K, N) in SWEEP_GATED}
            shapes.append(row)
            if row["gated"] and (worst is None or row["frac"] < worst["frac"]):
                worst = row
        unit = "TFLOP/s" if worst["bound"] == "tensor" else "GB/s"
        ach = worst["tflops"] if worst["bound"] == "tensor" else worst["gbs"]
        peak = peaks["bf16_tflops"] if worst["bound"] == "tensor" else peaks["hbm_gbs"]
        return {"bound": worst["bound"], "kernel": "tconv_kernel / tconv_res_kernel (one twn_gemm call per shape); headline = "
                f"the worst of the five gated shapes: M={worst['M']} K={worst['K']} N={worst['N']}",
                "achieved": ach, "peak": peak, "unit": unit, "frac": worst["frac"],
                "peak_source": peaks["source"] + " (bf16 burst / copy bandwidth: every shape is timed alone, cold L2)",
                "traffic": None, "shapes": shapes}

    def check(self):
        assert self.twn.read_status(self.status) == 0

    def cpu_sample(self, host, seconds=10.0):
        import oracle
        w, x = host
        K, N, M = 4096, 4096, 16384
        st, codes = oracle.ternarize(w[(K, N)], 0.7)
        rows = 8
        while True:
            t0 = time.perf_counter()
            oracle.gemm(x[(M, K)][:rows], codes, st.alpha)
            dt = time.perf_counter() - t0
            if dt >= seconds * 0.5 or rows >= M:
                break
            rows = int(min(M, max(rows * 2, rows * seconds / max(dt, 1e-3))))
        return 2.0 * rows * N * K / dt / 1e12, f"oracle gemm on {rows} of {M} rows of the K=N=4096 shape ({dt:.1f} s)", oracle.num_threads()


LAYER_SHAPES = {   # name: (H = W, Cin, Cout, kernel, stride, pad): the 3x3 layers of the four ResNet-18 stages
    "l1": (56, 64, 64, 3, 1, 1), "l2": (28, 128, 128, 3, 1, 1), "l3": (14, 256, 256, 3, 1, 1), "l4": (7, 512, 512, 3, 1, 1)}


class LayerWorkload:
    """One ternary convolution forward (Eq. 2) of a ResNet-18 stage shape with folded batch-norm affine and ReLU,
    bf16 in and out.  Used for per-layer numbers and for profiler captures at a reduced batch (--batch)."""
    metric = "ternary conv TFLOP/s"
    unit = "TFLOP/s"
    dtype = "bf16"
    default_steps = 200

    def __init__(self, which, batch=64):
        self.which, self.B = which, batch
        self.H, self.Cin, self.Cout, self.k, self.s, self.p = LAYER_SHAPES[which]
        self.name = f"conv_fwd_{which}_{self.H}x{self.H}x{self.Cin}_to_{self.Cout}_b{batch}"

    def config(self):
        mb = self.B * self.H * self.H * (self.Cin + self.Cout) * 2 / 1e6
        return {"workload": self.name, "seed": 0, "delta_factor": 0.7,
                "l2": f"activations in and out: {mb:.0f} MB per step; L2 flushed between the timed launches of the roofline figure"}

    def host_inputs(self):
        from paper_1605_04711_b200 import datagen as dg
        K = self.k * self.k * self.Cin
        return (dg.he_normal(0, f"layer.{self.which}.w", self.Cout, K),
                dg.draw_bf16(0, f"layer.{self.which}.x", self.B * self.H * self.H * self.Cin, "normal"))

    def setup(self, torch, twn, host):
        import numpy as np
        self.torch, self.twn = torch, twn
        Wm, x = host
        K = self.k * self.k * self.Cin
        self.ld = twn.ld_for(K)
        self.stats = twn.new_stats()
        self.packed = torch.empty((self.Cout, self.ld // 16), dtype=torch.int32, device="cuda")
        ws = torch.empty(twn.ternarize_workspace_bytes(), dtype=torch.uint8, device="cuda")
        twn.ternarize(torch.from_numpy(Wm).cuda(), 0.7, self.stats, self.packed, self.ld, None, ws, rows=self.Cout, cols=K)
        self.d = twn.conv_desc(self.B, self.H, self.H, self.Cin, self.Cout, self.k, self.s, self.p)
        self.host_x = torch.from_numpy(x.view(np.int16)).pin_memory()
        self.X = self.host_x.cuda().view(torch.bfloat16).view(self.B, self.H, self.H, self.Cin)
        self.Y = torch.empty((self.B, self.d.Ho, self.d.Wo, self.Cout), dtype=torch.bfloat16, device="cuda")
        self.host_y = torch.empty(self.Y.numel(), dtype=torch.int16).pin_memory()
        self.scale = torch.ones(self.Cout, device="cuda")
        self.shift = torch.zeros(self.Cout, device="cuda")
        self.epi = twn.epilogue(self.scale, self.shift, None, relu=True, out_dtype=twn.BF16)
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def step(self):
        self.twn.conv2d_fwd(self.d, self.X, self.packed, self.ld, self.stats, self.epi, self.Y, self.status)

    def step_e2e(self):
        t = self.torch
        self.X.view(t.int16).view(-1).copy_(self.host_x, non_blocking=True)
        self.step()
        self.host_y.copy_(self.Y.view(t.int16).view(-1), non_blocking=True)

    def e2e_bytes(self):
        return self.X.numel() * 2, self.Y.numel() * 2

    def launches_per_step(self):
        return 1

    def flops(self):
        return 2.0 * self.B * self.d.Ho * self.d.Wo * self.k * self.k * self.Cin * self.Cout

    def nbytes(self):
        return self.X.numel() * 2 + self.k * self.k * self.Cin * self.Cout / 4.0 + self.Y.numel() * 2

    def units_per_step(self):
        return self.flops() / 1e12

    def roofline(self, ms_per_step, peaks):
        med, mn = time_cold(self.torch, self.step)
        kind, t_us = bound_of(self.flops(), self.nbytes(), peaks)
        return {"bound": kind, "kernel": "one twn_conv2d_fwd call, timed alone after an L2 flush",
                "achieved": self.flops() / med / 1e6 if kind == "tensor" else self.nbytes() / med / 1e3,
                "peak": peaks["bf16_tflops"] if kind == "tensor" else peaks["hbm_gbs"],
                "unit": "TFLOP/s" if kind == "tensor" else "GB/s", "frac": t_us / med, "us_median": med, "us_min": mn,
                "bound_us": t_us, "algorithmic_bytes": self.nbytes(), "flops": self.flops(),
                "peak_source": peaks["source"] + " (burst: timed alone)", "traffic": None}

    def check(self):
        assert self.twn.read_status(self.status) == 0

    def cpu_sample(self, host, seconds=10.0):
        import numpy as np
        import oracle
        Wm, x = host
        st, codes = oracle.ternarize(Wm, 0.7)
        d = oracle.conv_desc(self.B, self.H, self.H, self.Cin, self.Cout, self.k, self.s, self.p)
        X = x.reshape(self.B, self.H, self.H, self.Cin)
        total = self.B * d.Ho * d.Wo
        npix = 64
        while True:
            pix = np.arange(npix) % total
            t0 = time.perf_counter()
            oracle.conv2d_fwd(d, X, codes.reshape(self.Cout, self.k, self.k, self.Cin), st.alpha, pixels=pix)
            dt = time.perf_counter() - t0
            if dt >= seconds * 0.5 or npix >= total:
                break
            npix = int(min(total, max(npix * 2, npix * seconds / max(dt, 1e-3))))
        return 2.0 * npix * self.k * self.k * self.Cin * self.Cout / dt / 1e12, \
            f"oracle conv2d_fwd on {npix} of {total} output pixels ({dt:.1f} s)", oracle.num_threads()


class NetWorkload:
    """A chained network workload: images/s of a forward pass or of a whole training step,
    replayed from a CUDA graph (the step is a fixed sequence of ~200 launches)."""
    metric = "images/s"
    unit = "images/s"
    dtype = "bf16"
    default_steps = 200

    def __init__(self, kind):
        self.kind = kind
        self.name = {"resnet18_train": "resnet18_train_step_b64_224", "vgg7_fwd": "vgg7_forward_b128",
                     "lenet5_fwd": "lenet5_forward_b100", "resnet18b_train": "resnet18b_train_step_b64_224",
                     "resnet18_train_sgd": "resnet18_train_step_with_update_b64_224"}[kind]

    def train_kind(self):
        return self.kind in ("resnet18_train", "resnet18b_train", "resnet18_train_sgd")

    def make(self, nets):
        if self.kind == "resnet18_train":
            return nets.resnet18(64, train=True)
        if self.kind == "resnet18b_train":
            return nets.resnet18b(64, train=True)
        if self.kind == "resnet18_train_sgd":
            # a learning rate small enough that hundreds of steps on the same synthetic batch stay finite
            return nets.resnet18(64, train=True, optimizer=dict(lr=1e-12, momentum=0.9, weight_decay=1e-4))
        if self.kind == "vgg7_fwd":
            return nets.vgg7(128)
        return nets.lenet5(100)

    def config(self):
        c = {"workload": self.name, "seed": 0, "delta_factor": 0.7,
             "l2": "activations of a step (> 1 GB for ResNet-18) exceed L2 (126 MB)",
             "launch": "one CUDA graph replay per step",
             "e2e": "pipelined: the pinned-host copy of batch i+1 runs on a copy stream while step i computes; "
                    "the result read back every step is the logits (the weight gradients stay on the device)"}
        if self.train_kind():
            c["step"] = ("ternarize+pack 21 tensors, transpose codes, forward, backward for data, "
                         "straight-through dW; synthetic dY N(0,1e-2) at the logits")
            if self.kind == "resnet18_train_sgd":
                c["step"] += ("; SGD-momentum update of the master weights (lr 1e-12 so that repeated steps on one "
                              "synthetic batch stay finite), whose threshold reduction replaces the first ternarization sweep")
        else:
            c["step"] = "forward through ternary conv/FC with packed weights (ternarization done once, untimed)"
            c["l2"] = "L2 flushed between timed steps is not needed: one step per replay, working set noted"
        return c

    def host_inputs(self):
        from paper_1605_04711_b200 import datagen as dg
        shape = {"resnet18_train": (64, 224, 224, 3), "resnet18b_train": (64, 224, 224, 3),
                 "resnet18_train_sgd": (64, 224, 224, 3), "vgg7_fwd": (128, 32, 32, 3),
                 "lenet5_fwd": (100, 28, 28, 1)}[self.kind]
        n = 1
        for s in shape:
            n *= s
        dist = "uniform01" if self.kind == "lenet5_fwd" else "normal"
        x = dg.draw_bf16(0, f"{self.name}.input", n, dist)
        dy = dg.draw_bf16(0, f"{self.name}.dlogits", 64 * 1000, "normal", 0.0, 0.1) if self.train_kind() else None
        return x, dy

    def setup(self, torch, twn, host):
        from paper_1605_04711_b200 import nets
        import numpy as np
        self.torch, self.twn = torch, twn
        x, dy = host
        self.net = net = self.make(nets)
        self.train = self.train_kind()
        self.host_x = torch.from_numpy(x.view(np.int16)).pin_memory()
        net.act["input"].view(torch.int16).view(-1).copy_(self.host_x)
        last = net.ops[-1][1]
        self.logits = net.act[last.name]
        self.host_logits = torch.empty(self.logits.shape, dtype=self.logits.dtype).pin_memory()
        if self.train:
            self.host_dy = torch.from_numpy(dy.view(np.int16)).pin_memory()
            self.dY = torch.zeros((64, 1000), dtype=torch.bfloat16, device="cuda")
            self.dY.view(torch.int16).view(-1).copy_(self.host_dy)
        else:
            net.ternarize_all()
        # eager warm-up (first-call set-up, lazy buffers), then capture the step
        for _ in range(2):
            self._eager()
        torch.cuda.synchronize()
        net.check_status()
        self.graph = torch.cuda.CUDAGraph()
        # The step is captured on a high-priority stream: the forward / backward-for-data chain is the
        # critical path, while the weight gradients and the code re-layouts (streams of default
        # priority forked from it) fill the SMs it leaves free.
        with torch.cuda.graph(self.graph, stream=torch.cuda.Stream(priority=-1)):
            self._eager()
        # per-kernel device times from one eager pass; a spin keeps the GPU behind the host so
        # that the events bracket kernels only
        net.timed = []
        torch.cuda._sleep(int(40e6))
        self._eager()
        torch.cuda.synchronize()
        agg = {}
        for kind, name, flops, e0, e1 in net.timed:
            a = agg.setdefault(kind, [0, 0.0, 0.0])
            a[0] += 1; a[1] += e0.elapsed_time(e1); a[2] += flops
        self.kernel_times = agg
        net.timed = None
        self.per_layer = self._per_layer_pass()

    def _eager(self):
        if self.train:
            self.net.train_step(self.dY)
        else:
            self.net.forward()

    def _per_layer_pass(self, reps=20):
        """Isolated device time of every tensor-core call of a step: the step is run eagerly with the weight-gradient
        and code-layout streams joined to the main stream, so that every kernel has the GPU to itself (the inputs are
        as the preceding kernels of the step left them: the activations of a layer exceed L2 for the large layers
        only).  Returns {(kind, name): (flops, [microseconds per repetition])}."""
        t, net = self.torch, self.net
        main = t.cuda.current_stream()
        saved = net.dw_stream, net.side_streams
        net.dw_stream, net.side_streams = main, [main]
        rows = {}
        try:
            for _ in range(reps + 2):
                net.timed = []
                t.cuda._sleep(int(10e6))       # the host runs ahead of the device: events bracket kernels only
                self._eager()
                t.cuda.synchronize()
                for kind, name, flops, e0, e1 in net.timed:
                    rows.setdefault((kind, name), (flops, []))[1].append(e0.elapsed_time(e1) * 1e3)
        finally:
            net.timed = None
            net.dw_stream, net.side_streams = saved
        return {k: (f, v[2:]) for k, (f, v) in rows.items()}

    def _op_bytes(self, L, op):
        """Algorithmic bytes of one call: operands once in, result once out, packed codes at 2 bits."""
        e = L.extra
        in_b = (e["xf"].numel() if L.fold else e["xcol"].numel() if L.small_cin else L.B * L.H * L.W * L.Cin) * 2
        out_px = L.B * L.Ho * L.Wo
        codes = L.K * L.Cout / 4.0
        if op == "fwd":
            return in_b + codes + out_px * L.Cout * (4 if L.out_f32 else 2) + (out_px * L.Cout * 2 if L.residual else 0)
        if op == "dX":
            return out_px * L.Cout * 2 + codes + L.B * L.H * L.W * L.Cin * 2
        return in_b + out_px * L.Cout * 2 + L.K * L.Cout * 4.0

    def step(self):
        self.graph.replay()

    def _prefetch(self):
        """Enqueues, on the copy stream, the host-to-device copy of the next step's inputs into the
        staging buffers (once the previous contents have been consumed)."""
        t = self.torch
        with t.cuda.stream(self.copy_stream):
            self.copy_stream.wait_event(self.ev_free)
            self.stage_x.view(t.int16).view(-1).copy_(self.host_x, non_blocking=True)
            if self.train:
                self.stage_dy.view(t.int16).view(-1).copy_(self.host_dy, non_blocking=True)
            self.ev_h2d.record(self.copy_stream)

    def step_e2e(self):
        """One step as an input pipeline runs it: every step copies one batch from pinned host memory
        (on a copy stream, so the batch of step i+1 travels while step i computes), moves it into the
        network's input buffer, replays the step and reads the logits back."""
        t = self.torch
        main = t.cuda.current_stream()
        if not hasattr(self, "copy_stream"):
            self.copy_stream = t.cuda.Stream()
            self.stage_x = t.empty_like(self.net.act["input"])
            self.stage_dy = t.empty_like(self.dY) if self.train else None
            self.ev_h2d, self.ev_free = t.cuda.Event(), t.cuda.Event()
            self.ev_free.record(main)
            self._prefetch()
        main.wait_event(self.ev_h2d)
        self.net.act["input"].copy_(self.stage_x, non_blocking=True)
        if self.train:
            self.dY.copy_(self.stage_dy, non_blocking=True)
        self.ev_free.record(main)
        self._prefetch()
        self.graph.replay()
        self.host_logits.copy_(self.logits, non_blocking=True)

    def e2e_bytes(self):
        h2d = self.host_x.numel() * 2 + (self.host_dy.numel() * 2 if self.train else 0)
        return h2d, self.host_logits.numel() * self.host_logits.element_size()

    def launches_per_step(self):
        n = 0
        net = self.net
        for op in net.ops:
            if op[0] == "layer":
                L = op[1]
                n += 1 + (1 if L.small_cin else 0)                       # forward (+ im2col or input fold)
                if self.train:
                    n += 1 if L.fold else 0                              # folded codes
                    n += 1 + 1 + (1 if L.fold else 0)                    # act_bwd, dW (+ unfold)
                    # the reduction of the pixel splits of dW runs only when there is more than one split
                    if L.fold:
                        n += 1
                    else:
                        d = L.extra["dw_desc"]
                        splits = self.twn.conv2d_bwd_weight_workspace_bytes(d) // (d.Cout * d.kh * d.kw * d.Cin * 4)
                        n += 1 if splits > 1 else 0
                    if L.src != "input":
                        # backward for data: one launch per residue class of the stride that a tap reaches
                        # (a 1x1 projection shortcut adds into the dense gradient in place: one class)
                        shortcut = L.k == 1 and L.stride > 1 and not L.relu and not L.residual
                        n += 1 if shortcut else L.stride * L.stride
            elif op[0] in ("maxpool", "avgpool"):
                n += 2 if self.train else 1
        if self.train:
            n += 3 * ((len(net.layers) + 31) // 32)     # batched ternarization (two sweeps) and code transposes
            # with the update: coding sweep + update instead of the two sweeps, the same count
        return n

    def units_per_step(self):
        return self.net.B

    def roofline(self, ms_per_step, peaks):
        """Headline: the ternary contractions of a step (every forward and backward-for-data call), each timed alone
        (median of 20), against the measured bf16 burst peak.  `per_layer` lists every tensor-core call with its own
        bound (the slower of flops at the burst peak and algorithmic bytes at the copy bandwidth) and fraction;
        `contended` keeps the per-kind times of one eager pass with the weight gradients on their own stream."""
        k = self.kernel_times
        per_layer, sums = [], {}
        for (kind, name), (flops, us) in self.per_layer.items():
            if kind == "ternarize":
                continue
            us = sorted(us)
            med, mn = us[len(us) // 2], us[0]
            lname, op = name.rsplit(".", 1)
            nbytes = self._op_bytes(self.net.layers[lname], op)
            bkind, t_us = bound_of(flops, nbytes, peaks)
            per_layer.append({"call": name, "us_median": round(med, 2), "us_min": round(mn, 2), "gflop": round(flops / 1e9, 2),
                              "mbytes": round(nbytes / 1e6, 2), "bound": bkind, "bound_us": round(t_us, 2),
                              "frac": round(t_us / med, 3)})
            a = sums.setdefault(kind, [0.0, 0.0, 0.0, 0])
            a[0] += med; a[1] += flops; a[2] += t_us; a[3] += 1
        t = sums.get("tconv", [0.0, 0.0, 0.0, 0])
        ach = t[1] / t[0] / 1e6 if t[0] > 0 else 0.0
        peak = peaks["bf16_tflops"]
        tern = self.per_layer_ternarize_us()
        step_flops = 2.0 * self.net.total_macs()
        out = {"bound": "tensor", "kernel": "tconv_kernel + tconv_res_kernel (every forward and backward-for-data call of a step, each timed alone)",
               "achieved": ach, "peak": peak, "unit": "TFLOP/s", "frac": ach / peak,
               "peak_source": peaks["source"] + " (bf16 burst: isolated kernels)", "traffic": self.measured_traffic(),
               "launches": t[3], "us_in_kernel_isolated": round(t[0], 1), "us_at_bound": round(t[2], 1),
               "frac_of_own_bounds": (t[2] / t[0]) if t[0] > 0 else None,
               "isolated_sums_us": {kk: round(v[0], 1) for kk, v in sums.items()},
               "isolated_tflops": {kk: round(v[1] / v[0] / 1e6, 1) for kk, v in sums.items() if v[0] > 0},
               "ternarize_us_isolated": tern,
               "contended": {"note": "one eager pass, weight gradients on their own stream beside the backward-for-data chain",
                             "ms": {kk: round(v[1], 4) for kk, v in k.items()}},
               "step_flops": step_flops,
               "step_frac_of_burst_peak": step_flops / (ms_per_step * 1e-3) / 1e12 / peak,
               "step_frac_of_sustained_peak": step_flops / (ms_per_step * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
               "per_layer": per_layer}
        return out

    def per_layer_ternarize_us(self):
        us = [v for (kind, _), (_, vals) in self.per_layer.items() if kind == "ternarize" for v in [sorted(vals)[len(vals) // 2]]]
        return round(sum(us), 1) if us else None

    def measured_traffic(self):
        """DRAM bytes per step of the ternary contractions of the ResNet-18 step: sum over the launches of
        dram__bytes_read.sum + dram__bytes_write.sum over the 50 forward and backward-for-data launches of one step,
        from one ncu capture of this workload at its full size (profiles/tconv_resnet18_step_dram.md); None for the
        other workloads."""
        return TRAFFIC_RESNET18_STEP if self.kind in ("resnet18_train", "resnet18_train_sgd") else None

    def check(self):
        self.net.check_status()
        assert bool(self.torch.isfinite(self.logits.float()).all())

    def _ops(self):
        from paper_1605_04711_b200 import nets
        if self.kind in ("resnet18_train", "resnet18_train_sgd"):
            return nets.resnet18_ops(), 64
        if self.kind == "resnet18b_train":
            return nets.resnet18_ops(widths=(96, 192, 384, 768)), 64
        if self.kind == "vgg7_fwd":
            return nets.vgg7_ops(), 128
        return nets.lenet5_ops(), 100

    def cpu_sample(self, host, seconds=24.0, full=False):
        """The oracle (fp64, OpenMP) on every layer of the workload: forward, and for a training step backward for
        data and the weight gradient.  A layer whose full size fits its share of the time budget is run in full;
        otherwise the oracle runs on sampled output pixels (weight-gradient entries) at batch 2 and the time is
        scaled to the layer's full size.  The step time is the sum over layers, plus (training step only) the ternarization
        of all weights.  full=True runs every layer at its full size whatever it takes."""
        import numpy as np
        import oracle
        from paper_1605_04711_b200 import datagen as dg
        ops, B = self._ops()
        layers = [op[1] for op in ops if op[0] == "layer"]
        train = self.train_kind()
        budget = 1e9 if full else seconds / (len(layers) * (3 if train else 1))
        Bs = 2

        def run(fn, n_total, scale):
            """fn(indices) on a growing sample of range(n_total); returns seconds extrapolated to scale * n_total items."""
            n, full = min(16, n_total), False
            while True:
                idx = np.arange(n, dtype=np.int64) * max(1, n_total // n) % n_total
                t0 = time.perf_counter()
                fn(idx)
                dt = time.perf_counter() - t0
                if n >= n_total:
                    full = True
                    break
                if dt >= budget * 0.5:
                    break
                n = int(min(n_total, max(n * 2, n * budget / max(dt, 1e-4))))
            return dt / n * n_total * scale, full and scale == 1.0

        t_cpu0 = time.perf_counter()
        total_s, n_full, n_ops, n_weights = 0.0, 0, 0, 0
        for L in layers:
            K = L.k * L.k * L.Cin
            # layers small enough are taken at their full batch, the others at batch 2
            b = B if (full or B * L.Ho * L.Wo * K * L.Cout <= 3e9) else Bs
            d = oracle.conv_desc(b, L.H, L.W, L.Cin, L.Cout, L.k, L.stride, L.pad)
            X = dg.draw_bf16(0, f"cpu.{L.name}.x", b * L.H * L.W * L.Cin, "normal").reshape(b, L.H, L.W, L.Cin)
            Wm = dg.he_normal(0, f"cpu.{L.name}.w", L.Cout, K)
            t0 = time.perf_counter()
            st, codes = oracle.ternarize(Wm, 0.7)
            oracle.pack(codes.reshape(L.Cout, K), oracle.ld_for(K))
            if train:
                total_s += time.perf_counter() - t0
            n_weights += Wm.size
            codes4 = codes.reshape(L.Cout, L.k, L.k, L.Cin)
            sec, full = run(lambda pix: oracle.conv2d_fwd(d, X, codes4, st.alpha, pixels=pix), b * L.Ho * L.Wo, B / b)
            total_s += sec; n_full += full; n_ops += 1
            if train:
                dZ = dg.draw_bf16(0, f"cpu.{L.name}.dz", b * L.Ho * L.Wo * L.Cout, "normal", 0.0, 0.1).reshape(b, L.Ho, L.Wo, L.Cout)
                if L.src != "input":
                    sec, full = run(lambda pix: oracle.conv2d_bwd_data(d, dZ, codes4, st.alpha, pixels=pix), b * L.H * L.W, B / b)
                    total_s += sec; n_full += full; n_ops += 1
                sec, full = run(lambda ent: oracle.conv2d_bwd_weight(d, X, dZ, entries=ent), L.Cout * K, B / b)
                total_s += sec; n_full += full; n_ops += 1
        spent = time.perf_counter() - t_cpu0
        what = "forward, backward for data and weight gradient" if train else "forward"
        return B / total_s, (f"oracle {what} of all {len(layers)} layers, one by one on seeded inputs, plus ternarize+pack of their "
                             f"{n_weights} weights; {n_full} of {n_ops} calls at full size, the others on sampled outputs at batch {Bs} "
                             f"scaled to batch {B} ({spent:.1f} s of CPU; oracle step time {total_s:.1f} s)"), oracle.num_threads()

# From the ncu capture summarised in profiles/tconv_resnet18_step_dram.md (see NetWorkload.measured_traffic).
TRAFFIC_RESNET18_STEP = 873.2e6

WORKLOADS = {"ternarize": lambda: TernarizeWorkload(), "binarize": lambda: BinarizeWorkload(), "sgd_ternarize": lambda: SgdTernarizeWorkload(), "ternarize_rows": lambda: TernarizeRowsWorkload(), "resnet18_train": lambda: NetWorkload("resnet18_train"),
             "gemm_16384": lambda: GemmWorkload(16384), "gemm_4096": lambda: GemmWorkload(4096),
             "vgg7_fwd": lambda: NetWorkload("vgg7_fwd"), "lenet5_fwd": lambda: NetWorkload("lenet5_fwd"),
             "resnet18b_train": lambda: NetWorkload("resnet18b_train"),
             "resnet18_train_sgd": lambda: NetWorkload("resnet18_train_sgd"),
             "gemm_sweep": lambda: GemmSweepWorkload(),
             "layer_l1": lambda: LayerWorkload("l1"), "layer_l2": lambda: LayerWorkload("l2"),
             "layer_l3": lambda: LayerWorkload("l3"), "layer_l4": lambda: LayerWorkload("l4")}
DEFAULT_WORKLOAD = "resnet18_train"


# ------------------------------------------------------------------ arms
def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    wl = WORKLOADS[args.workload]()
    host = wl.host_inputs() if isinstance(wl, (TernarizeWorkload, GemmWorkload, GemmSweepWorkload, LayerWorkload)) else None
    vals = []
    steps = args.steps if args.steps else 3
    for i in range(args.warmup + steps):
        v, sample, cores = wl.cpu_sample(host, full=True) if (args.full_oracle and isinstance(wl, NetWorkload)) else wl.cpu_sample(host)
        if i >= args.warmup:
            vals.append(v)
    value = sum(vals) / len(vals)
    if isinstance(wl, GemmSweepWorkload):
        wl.cases = [(M, K, N) for K, N in SWEEP_KN for M in SWEEP_M]
    if isinstance(wl, LayerWorkload):
        import oracle as _o
        wl.d = _o.conv_desc(wl.B, wl.H, wl.H, wl.Cin, wl.Cout, wl.k, wl.s, wl.p)
    upstep = wl.units_per_step() if isinstance(wl, (TernarizeWorkload, GemmWorkload, GemmSweepWorkload, LayerWorkload)) else wl._ops()[1]
    line = {"impl": "reference", "metric": wl.metric, "value": value, "unit": wl.unit,
            "n_gpus": args.gpus, "steps": steps, "warmup": args.warmup,
            "ms_per_step": upstep / value * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": wl.config(), "gpu_launches": 0,
            "cpu_baseline": {"value": value, "unit": wl.unit, "cores": cores, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": wl.unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def ternarize_leg(torch, twn, peaks, steps=300):
    """GB/s of twn_ternarize (per layer) and twn_ternarize_rows (per filter) on 1e8 seeded N(0,1)
    weights, timed with CUDA events after warm-up; the 400 MB input exceeds L2."""
    wl = TernarizeWorkload()
    W = wl.host_inputs()
    wl.setup(torch, twn, W)
    out = {}
    rows_wl = TernarizeRowsWorkload(rows=wl.n // 8192)      # the same weights as 12207 filters of 8192
    legs = [("per_layer", wl, wl.step)]
    if wl.n >= rows_wl.n:
        rows_wl.torch, rows_wl.twn = torch, twn
        rows_wl.ld = twn.ld_for(rows_wl.cols)
        rows_wl.W = wl.W[:rows_wl.n].view(rows_wl.rows, rows_wl.cols)
        rows_wl.stats = twn.new_stats_rows(rows_wl.rows)
        rows_wl.packed = torch.empty((rows_wl.rows, rows_wl.ld // 16), dtype=torch.int32, device="cuda")
        legs.append(("per_filter", rows_wl, rows_wl.step))
    for name, w, fn in legs:
        for _ in range(5):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        w.check()
        ms = e0.elapsed_time(e1) / steps
        gbs = w.n * w.bytes_per_unit / (ms * 1e-3) / 1e9
        out[name] = {"value": gbs, "unit": "GB/s", "n": w.n, "bytes_per_weight": w.bytes_per_unit, "ms": ms,
                     "frac_of_hbm_peak": gbs / peaks["hbm_gbs"], "frac_of_nominal_8TBs": gbs / 8000.0,
                     "peak_source": peaks["source"]}
    return out


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
    if args.batch and isinstance(wl, LayerWorkload):
        wl = LayerWorkload(wl.which, args.batch)
    steps = args.steps if args.steps else wl.default_steps
    warmup = max(args.warmup, 3)
    host = wl.host_inputs()
    wl.setup(torch, twn, host)
    peaks = measured_peaks()

    def timed(fn, n_steps, n_warm):
        """Mean step time over exactly n_steps back-to-back steps (the reported value), and the
        median and minimum of the single steps, from one event per step boundary."""
        for _ in range(n_warm):
            fn()
        barrier()
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(n_steps + 1)]
        evs[0].record()
        for i in range(n_steps):
            fn()
            evs[i + 1].record()
        barrier()
        ms = max_over_ranks(evs[0].elapsed_time(evs[-1]), world, dist if world > 1 else None, "cuda")
        each = sorted(evs[i].elapsed_time(evs[i + 1]) for i in range(n_steps))
        return ms / n_steps, {"median_ms": each[len(each) // 2], "min_ms": each[0], "steps": n_steps}

    sampler = ClockSampler(local_rank, str(getattr(torch.cuda.get_device_properties(local_rank), 'uuid', ''))) if rank == 0 else None
    if sampler:
        sampler.start()
    ms, spread = timed(wl.step, steps, warmup)
    clocks = sampler.stop() if sampler else None
    wl.check()
    ms_e2e, _ = timed(wl.step_e2e, max(2, min(steps, 20)), 1)
    wl.check()

    if rank == 0:
        h2d, d2h = wl.e2e_bytes()
        line = {"metric": wl.metric, "value": world * wl.units_per_step() / (ms * 1e-3),
                "unit": wl.unit, "n_gpus": world, "steps": steps, "warmup": warmup,
                "ms_per_step": ms, "ms_per_step_median": spread["median_ms"], "ms_per_step_min": spread["min_ms"],
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": wl.dtype, "data": "synthetic", "config": wl.config(), "clocks": clocks,
                "e2e": {"value": world * wl.units_per_step() / (ms_e2e * 1e-3), "unit": wl.unit,
                        "ms_per_step": ms_e2e, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
                "gpu_launches": wl.launches_per_step() * steps,
                "roofline": wl.roofline(ms, peaks)}
        if args.workload == DEFAULT_WORKLOAD and world == 1 and not args.no_ternarize_leg:
            # the second half of the headline metric, measured in the same run: ternarize + pack of
            # one 1e8-weight tensor (larger than L2), in GB/s of algorithmic traffic
            line["ternarize_pack"] = ternarize_leg(torch, twn, peaks)
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
    ap.add_argument("--steps", type=int, default=0, help="timed steps (0: the workload's default)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--batch", type=int, default=0, help="layer_* workloads: batch size (default 64)")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--full-oracle", action="store_true",
                    help="--impl reference, network workloads: run the oracle on every layer at its full size (no sampling)")
    ap.add_argument("--no-ternarize-leg", action="store_true",
                    help="default workload only: skip the ternarize+pack GB/s measurement added to the line")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
