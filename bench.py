#!/usr/bin/env python
"""Benchmark of the MVUE prune+pack (and consuming products) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

Prints ONE JSON line.  A step is one pass of the hot path over one synthetic batch of
the `conv_im2col` workload (gradient g bf16 [200704 x 256], ReLU-sparse lognormal; MVUE
2:4 along the token axis).  `value` is the throughput with inputs resident in HBM;
`e2e` repeats the measurement through the same C-ABI call with pinned host buffers and the
host<->device copies inside the timed region.  `--impl reference` times the CPU oracle on a
bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

METRIC = "prune+pack GB/s (% HBM peak); MVUE-sparse GEMM TFLOP/s vs dense bf16"
L2_BYTES = 126 * 1024 * 1024


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def prune_bytes(rows: int, cols: int, elem_bytes: int) -> int:
    """Algorithmic bytes of one prune+pack: g read once, K/2 bf16 survivors and 4 bits of
    metadata per group of four written once."""
    n = rows * cols
    return n * elem_bytes + n + n // 8


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while a region runs."""

    def __init__(self, index: int, period_s: float = 0.05):
        self.index, self.period = index, period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# --------------------------------------------------------------------------- CPU oracle arm
def oracle_sample(cfg, n, m, sample_rows: int):
    """Time the oracle's prune+pack, as it stands, on the first `sample_rows` token rows."""
    import oracle
    from paper_2203_10991_b200 import workloads
    g = workloads.gradient((sample_rows, cfg["out"]), cfg["g_dist"], cfg["seed"], dtype=cfg["g_dtype"])
    threads = oracle.host_threads()
    t0 = time.perf_counter()
    oracle.prune(g, n, m, axis=0, seed=0, k_total=cfg["T"], k_offset=0, threads=threads)
    dt = time.perf_counter() - t0
    nbytes = prune_bytes(sample_rows, cfg["out"], 2 if cfg["g_dtype"] == "bf16" else 4)
    return nbytes / dt / 1e9, threads, dt


def run_reference(args, cfg, n, m):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    # size the per-step sample so that K + W steps of the oracle take about a minute in all
    _, _, dt_probe = oracle_sample(cfg, n, m, 8192)
    rows_per_s = 8192 / dt_probe
    budget_s = 60.0
    sample_rows = int(rows_per_s * budget_s / max(1, args.steps + args.warmup))
    sample_rows = max(1024, min(cfg["T"], sample_rows // 16 * 16))
    vals = []
    for _ in range(args.warmup):
        oracle_sample(cfg, n, m, sample_rows)
    t_all = 0.0
    for _ in range(args.steps):
        gbs, threads, dt = oracle_sample(cfg, n, m, sample_rows)
        vals.append(gbs)
        t_all += dt
    value = float(np.mean(vals))
    sample = f"first {sample_rows} of {cfg['T']} token rows x {cfg['out']} channels, MVUE {n}:{m}, axis 0"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_all / max(1, args.steps),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": args.workload, "prune": f"{n}:{m}", "axis": 0, "sample_rows": sample_rows},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# --------------------------------------------------------------------------- GPU arm
def run_ours(args, cfg, n, m):
    import torch
    import torch.distributed as dist
    from paper_2203_10991_b200 import binding, workloads

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    binding.lib()                                       # fail loudly if the CUDA library is absent

    T, out = cfg["T"], cfg["out"]
    elem = 2 if cfg["g_dtype"] == "bf16" else 4
    # every rank draws its own batch (weak scaling: independent batches, no data-path collective)
    g_host = workloads.gradient((T, out), cfg["g_dist"], cfg["seed"] + 1000 * rank, dtype=cfg["g_dtype"])
    g_t = torch.from_numpy(g_host.view(np.int16) if elem == 2 else g_host)
    step_bytes = prune_bytes(T, out, elem)
    # rotate over enough distinct input/output buffers that no step finds its data in L2
    n_buf = max(2, int(np.ceil(2.5 * L2_BYTES / step_bytes)) + 1)
    gs = []
    for i in range(n_buf):
        x = g_t.to(dev)
        gs.append(x.view(torch.bfloat16) if elem == 2 else x)
    outs = [(torch.empty((out, T // 2), dtype=torch.bfloat16, device=dev),
             torch.empty((out, T // 8), dtype=torch.uint8, device=dev)) for _ in range(n_buf)]

    def step(i):
        b = i % n_buf
        binding.mvue_prune(gs[b], n, m, 0, i, values=outs[b][0], meta=outs[b][1])

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(3, args.warmup)):
        step(i)
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clocks:
        barrier()
        ev0.record()
        for i in range(args.steps):
            step(i)
        ev1.record()
        barrier()
    ms = ev0.elapsed_time(ev1)
    if world > 1:
        t = torch.tensor([ms], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    ms_per_step = ms / args.steps
    value = world * step_bytes / (ms_per_step * 1e-3) / 1e9

    # end to end: pinned host input -> device -> prune -> packed result back to pinned host
    g_pin = g_t.pin_memory()
    v_pin = torch.empty((out, T // 2), dtype=torch.bfloat16).pin_memory()
    m_pin = torch.empty((out, T // 8), dtype=torch.uint8).pin_memory()
    g_dev = gs[0]
    e2e_steps = max(3, min(args.steps, 20))

    def e2e_step(i):
        g_dev.view(torch.int16 if elem == 2 else torch.float32).copy_(g_pin, non_blocking=True)
        binding.mvue_prune(g_dev, n, m, 0, i, values=outs[0][0], meta=outs[0][1])
        v_pin.copy_(outs[0][0], non_blocking=True)
        m_pin.copy_(outs[0][1], non_blocking=True)

    for i in range(3):
        e2e_step(i)
    barrier()
    ev0.record()
    for i in range(e2e_steps):
        e2e_step(i)
    ev1.record()
    barrier()
    e2e_ms = ev0.elapsed_time(ev1)
    if world > 1:
        t = torch.tensor([e2e_ms], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms = float(t.item())
    e2e_value = world * step_bytes / (e2e_ms / e2e_steps * 1e-3) / 1e9

    if rank == 0:
        peaks = measured_peaks()
        achieved = step_bytes / (ms_per_step * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": args.workload, "g": [T, out], "g_dtype": cfg["g_dtype"],
                       "prune": f"{n}:{m}", "axis": 0, "l2": f"rotating {n_buf} buffer sets (> 2.5x L2)"},
            "clocks": clocks.summary(),
            "e2e": {"value": e2e_value, "unit": "GB/s", "h2d_bytes_per_step": T * out * elem,
                    "d2h_bytes_per_step": T * out + T * out // 8},
            "gpu_launches": args.steps,
            "roofline": {"bound": "hbm", "kernel": "prune_axis0_kernel", "achieved": achieved,
                         "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                         "peak_source": peaks["source"], "traffic": None},
        }
        if world == 1 and not args.no_cpu_baseline:
            sample_rows = min(T, 1 << 19)
            gbs, threads, dt = oracle_sample(cfg, n, m, sample_rows)
            line["cpu_baseline"] = {"value": gbs, "unit": "GB/s", "cores": threads, "kind": "oracle",
                                    "sample": f"first {sample_rows} of {T} token rows x {out} channels, "
                                              f"MVUE {n}:{m}, axis 0, {dt:.2f} s"}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="conv_im2col")
    ap.add_argument("--prune", default="2:4")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    from paper_2203_10991_b200 import workloads
    cfg = workloads.CONFIGS[args.workload]
    n, m = (int(x) for x in args.prune.split(":"))
    if args.impl == "reference":
        args.steps = 5 if args.steps is None else args.steps
        run_reference(args, cfg, n, m)
    else:
        args.steps = 2000 if args.steps is None else args.steps
        run_ours(args, cfg, n, m)


if __name__ == "__main__":
    main()
