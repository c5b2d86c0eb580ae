#!/usr/bin/env python
"""Benchmark of the MVUE hot path on B200: prune+pack of the neural gradient followed by the
2:4-sparse update product that consumes it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME] [--prune n:m]

Prints ONE JSON line.  A step is one pass of the whole path over one synthetic batch of the
`conv_im2col` workload: g bf16 [200704 x 256] (ReLU-sparse lognormal), h bf16 [200704 x 2304]:
    values, meta = mvue_prune(g, 2:4, along the token axis)      # Sec. 4.2 / App. A.2
    dW[256 x 2304] = theta(g)^T h                                  # Sec. 1, update equation
`value` is the step's algorithmic bytes per second with every input resident in HBM (the step is
HBM-bound on this workload: h alone is 925 MB, far beyond L2, so no step finds its inputs cached);
the per-kernel figures (prune GB/s, GEMM effective TFLOP/s, dense cuBLAS for the same shape) ride
along.  `e2e` repeats the step through the same C-ABI calls from pinned host buffers with the
copies inside the timed region.  `--impl reference` times the CPU oracle on a bounded sample.
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


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def prune_bytes(rows: int, cols: int, elem_bytes: int) -> int:
    """Algorithmic bytes of one prune+pack: g read once; K/2 bf16 survivors and 4 bits of metadata per
    group of four written once (3.125 B per bf16 element, 5.125 B per fp32 element)."""
    n = rows * cols
    return n * elem_bytes + n + n // 8


def gemm_bytes(M: int, N: int, K: int, c_bytes: int = 4) -> int:
    """Minimum traffic of C[MxN] = A_packed[MxK] . B[KxN]: survivors, metadata, B and C once each."""
    return M * K + M * K // 8 + K * N * 2 + M * N * c_bytes


# dram__bytes_read.sum + dram__bytes_write.sum per launch on the conv_im2col workload, from one ncu capture of
# each kernel (summaries under profiles/).  Each figure is tied to a digest of the sources the kernel is built
# from: once those change the counters no longer describe the kernel and `traffic` is reported as null.
NCU_TRAFFIC = {
    "sparse_gemm_pair_kernel": (983140864 + 5710080, ("mvue_gemm.cu", "mvue_tma.h", "mvue_internal.h"),
                                "af3ecf5baf4a736b"),
    "prune_axis0_bf16_kernel/table": (103502080 + 26827520,
                                      ("mvue_prune.cu", "mvue_device.cuh", "mvue_tma.h", "mvue_internal.h"),
                                      "383e6715b6c6e3ef"),
    "prune_axis0_bf16_kernel/systematic": (103674368 + 26032128,
                                           ("mvue_prune.cu", "mvue_device.cuh", "mvue_tma.h", "mvue_internal.h"),
                                           "383e6715b6c6e3ef"),
}


def ncu_traffic(kernel: str, workload: str):
    import hashlib
    if workload != "conv_im2col" or kernel not in NCU_TRAFFIC:
        return None
    nbytes, sources, digest = NCU_TRAFFIC[kernel]
    h = hashlib.sha256()
    for name in sources:
        h.update((ROOT / "paper_2203_10991_b200" / "csrc" / name).read_bytes())
    return nbytes if h.hexdigest()[:16] == digest else None


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while a region runs."""

    def __init__(self, index: int, period_s: float = 0.02):
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
def oracle_sample(cfg, n, m, sample_rows: int, joint: int = 0):
    """One pass of the oracle, as it stands, over the first `sample_rows` token rows: prune+pack,
    unpack, and the fp64 plain-loop update product.  Returns (GB/s of algorithmic bytes, threads, s)."""
    import oracle
    from paper_2203_10991_b200 import workloads
    g = workloads.gradient((sample_rows, cfg["out"]), cfg["g_dist"], cfg["seed"], dtype=cfg["g_dtype"])
    h = workloads.normal_bf16((sample_rows, cfg["inp"]), cfg["seed"] + 100)
    threads = oracle.host_threads()
    t0 = time.perf_counter()
    values, meta = oracle.prune(g, n, m, axis=0, seed=0, k_total=cfg["T"], k_offset=0, threads=threads, joint=joint)
    oracle.gemm(oracle.unpack(values, meta), h, threads=threads)
    dt = time.perf_counter() - t0
    nbytes = (prune_bytes(sample_rows, cfg["out"], 2 if cfg["g_dtype"] == "bf16" else 4)
              + gemm_bytes(cfg["out"], cfg["inp"], sample_rows))
    return nbytes / dt / 1e9, threads, dt


def run_reference(args, cfg, n, m):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    joint = {"table": 0, "systematic": 1, "approx": 2}[args.joint]
    # size the per-step sample so that K + W steps of the oracle take about a minute in all: its cost
    # grows faster than linearly with the rows (the plain loops leave the cache), so probe by doubling
    per_step_s = 60.0 / max(1, args.steps + args.warmup)
    sample_rows = 512
    while sample_rows * 2 <= cfg["T"]:
        _, _, dt_probe = oracle_sample(cfg, n, m, sample_rows, joint)
        if dt_probe > per_step_s / 3:
            break
        sample_rows *= 2
    for _ in range(args.warmup):
        oracle_sample(cfg, n, m, sample_rows, joint)
    vals, t_all, threads = [], 0.0, 1
    for _ in range(args.steps):
        gbs, threads, dt = oracle_sample(cfg, n, m, sample_rows, joint)
        vals.append(gbs)
        t_all += dt
    value = float(np.mean(vals))
    sample = (f"first {sample_rows} of {cfg['T']} token rows: MVUE {n}:{m} prune+pack of g[{sample_rows}x{cfg['out']}] "
              f"and the fp64 update product with h[{sample_rows}x{cfg['inp']}]")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_all / max(1, args.steps),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "prune": f"{n}:{m}", "joint": args.joint, "axis": 0,
                   "sample_rows": sample_rows},
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
    TC = binding.MVUE_LAYOUT_TC

    T, out, inp = cfg["T"], cfg["out"], cfg["inp"]
    elem = 2 if cfg["g_dtype"] == "bf16" else 4
    # every rank draws its own token shard (data parallel over tokens, weak scaling)
    g_host = workloads.gradient((T, out), cfg["g_dist"], cfg["seed"] + 1000 * rank, dtype=cfg["g_dtype"])
    h_host = workloads.normal_bf16((T, inp), cfg["seed"] + 100 + 1000 * rank)
    g_t = torch.from_numpy(g_host.view(np.int16) if elem == 2 else g_host)
    h_t = torch.from_numpy(h_host.view(np.int16))
    g_dev = g_t.to(dev)
    g_dev = g_dev.view(torch.bfloat16) if elem == 2 else g_dev
    h_dev = h_t.to(dev).view(torch.bfloat16)
    _, meta_bytes = binding.mvue_packed_sizes(T, out, n, m, 0, TC)
    values = torch.empty((out, T // 2), dtype=torch.bfloat16, device=dev)
    meta = torch.empty(meta_bytes, dtype=torch.uint8, device=dev)
    dW = torch.empty((out, inp), dtype=torch.float32, device=dev)
    ws_bytes = binding.mvue_gemm_workspace_bytes(0, out, inp, T)
    ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    launches_per_step = 2 + (1 if ws_bytes > 0 else 0)      # prune, sparse GEMM, split-K reduction

    p_bytes = prune_bytes(T, out, elem)
    m_bytes = gemm_bytes(out, inp, T)
    step_bytes = p_bytes + m_bytes
    gemm_flops = 2.0 * out * inp * T

    joints = {"table": binding.MVUE_JOINT_TABLE, "systematic": binding.MVUE_JOINT_SYSTEMATIC,
              "approx": binding.MVUE_JOINT_APPROX}
    joint = [joints[args.joint]]                        # cells, so that the other estimators can be timed with the same step
    nm = [(n, m)]

    def step(i, ev=None):
        if ev:
            ev[0].record()
        binding.mvue_prune(g_dev, nm[0][0], nm[0][1], 0, i, values=values, meta=meta, layout=TC, joint=joint[0])
        if ev:
            ev[1].record()
        binding.mvue_sparse_update_gemm(values, meta, h_dev, out=dW, workspace=ws, dev_status=status)
        if ev:
            ev[2].record()
        if world > 1:
            dist.all_reduce(dW)                              # the data-parallel exchange of the update

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    warm = max(3, args.warmup)
    for i in range(warm):
        step(i)
    barrier()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clocks:
        barrier()
        ev0.record()
        for i in range(args.steps):
            step(i, evs[i])
        ev1.record()
        barrier()
    assert int(status.item()) == 0, "a bounded device-side wait expired"
    ms = ev0.elapsed_time(ev1)
    prune_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in evs]))
    gemm_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in evs]))
    if world > 1:
        t = torch.tensor([ms], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    ms_per_step = ms / args.steps
    value = world * step_bytes / (ms_per_step * 1e-3) / 1e9

    # the same step with the other 2:4 estimators, for the per-kernel prune time only (the product that
    # follows keeps L2 cold for the next prune exactly as in the timed region above)
    others = []
    if rank == 0 and world == 1 and m == 4 and not args.no_extra:
        for other_name in [k for k in joints if k != args.joint]:
            joint[0] = joints[other_name]
            k2 = max(3, min(args.steps, 200))
            for i in range(3):
                step(i)
            evs2 = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(k2)]
            torch.cuda.synchronize()
            for i in range(k2):
                step(i, evs2[i])
            torch.cuda.synchronize()
            others.append((other_name, float(np.mean([e[0].elapsed_time(e[1]) for e in evs2])), k2))
        joint[0] = joints[args.joint]
        # and MVUE 1:2 (emitted as a valid 2:4 pattern, so the same product consumes it)
        nm[0] = (1, 2)
        for i in range(3):
            step(i)
        evs2 = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(k2)]
        torch.cuda.synchronize()
        for i in range(k2):
            step(i, evs2[i])
        torch.cuda.synchronize()
        others.append(("1:2", float(np.mean([e[0].elapsed_time(e[1]) for e in evs2])), k2))
        # and MVUE 1:4 (one survivor beside a zero in the 2:4 container)
        nm[0] = (1, 4)
        for i in range(3):
            step(i)
        evs2 = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(k2)]
        torch.cuda.synchronize()
        for i in range(k2):
            step(i, evs2[i])
        torch.cuda.synchronize()
        others.append(("1:4", float(np.mean([e[0].elapsed_time(e[1]) for e in evs2])), k2))
        nm[0] = (n, m)

    # the step's prune timed alone (no product in between), L2-cold: inputs rotated over copies of g that together
    # exceed 2.5 x L2
    alone_ms = None
    if rank == 0 and world == 1 and not args.no_extra:
        copies = max(2, int(2.5 * 126e6 / (T * out * elem)) + 1)
        gs = [g_dev.clone() for _ in range(copies)]
        for i in range(3):
            binding.mvue_prune(gs[i % copies], n, m, 0, i, values=values, meta=meta, layout=TC, joint=joint[0])
        torch.cuda.synchronize()
        ka = max(3, min(args.steps, 100))
        ev0.record()
        for i in range(ka):
            binding.mvue_prune(gs[i % copies], n, m, 0, i, values=values, meta=meta, layout=TC, joint=joint[0])
        ev1.record()
        torch.cuda.synchronize()
        alone_ms = ev0.elapsed_time(ev1) / ka
        del gs

    # dense cuBLAS bf16 for the same shape (context for the sparse product)
    dense_ms = None
    if rank == 0 and elem == 2:
        gT = g_dev.t()
        for _ in range(3):
            torch.matmul(gT, h_dev)
        torch.cuda.synchronize()
        ev0.record()
        for _ in range(10):
            torch.matmul(gT, h_dev)
        ev1.record()
        torch.cuda.synchronize()
        dense_ms = ev0.elapsed_time(ev1) / 10

    # end to end: pinned host g and h -> device -> prune -> GEMM -> dW back to pinned host
    g_pin, h_pin = g_t.pin_memory(), h_t.pin_memory()
    dW_pin = torch.empty((out, inp), dtype=torch.float32).pin_memory()
    e2e_steps = max(2, min(args.steps, 5))

    def e2e_step(i):
        g_dev.view(torch.int16 if elem == 2 else torch.float32).copy_(g_pin, non_blocking=True)
        h_dev.view(torch.int16).copy_(h_pin, non_blocking=True)
        step(i)
        dW_pin.copy_(dW, non_blocking=True)

    e2e_step(0)
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
        prune_gbs = p_bytes / (prune_ms * 1e-3) / 1e9
        gemm_gbs = m_bytes / (gemm_ms * 1e-3) / 1e9
        gemm_tf = gemm_flops / (gemm_ms * 1e-3) / 1e12
        sparse_peak = 2.0 * peaks["bf16_tflops"]
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": warm, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": args.workload, "g": [T, out], "h": [T, inp], "g_dtype": cfg["g_dtype"],
                       "prune": f"{n}:{m}", "joint": args.joint, "axis": 0, "dW_dtype": "f32",
                       "l2": "inputs larger than L2 (h is 925 MB, read once per step)"},
            "clocks": clocks.summary(),
            "e2e": {"value": e2e_value, "unit": "GB/s", "h2d_bytes_per_step": T * out * elem + T * inp * 2,
                    "d2h_bytes_per_step": out * inp * 4},
            "gpu_launches": args.steps * launches_per_step,
            "prune": {"joint": args.joint, "ms": prune_ms, "gbs": prune_gbs,
                      "frac_of_hbm_peak": prune_gbs / peaks["hbm_gbs"]},
            "gemm": {"ms": gemm_ms, "tflops_effective": gemm_tf, "frac_of_sparse_peak": gemm_tf / sparse_peak,
                     "sparse_peak_tflops": sparse_peak, "gbs": gemm_gbs,
                     "dense_cublas_ms": dense_ms,
                     "dense_cublas_tflops": None if dense_ms is None else gemm_flops / (dense_ms * 1e-3) / 1e12},
            # the dominant kernel of the step is the sparse product; on this shape (256 x 2304 outputs over
            # 200704 rows, ~240 flop/B) it is bound by streaming h from HBM, not by the tensor cores
            "roofline": {"bound": "hbm", "kernel": "sparse_gemm_pair_kernel", "achieved": gemm_gbs,
                         "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gemm_gbs / peaks["hbm_gbs"],
                         "peak_source": peaks["source"],
                         "traffic": ncu_traffic("sparse_gemm_pair_kernel", args.workload) if (n, m) == (2, 4) else None},
            "roofline_prune": {"bound": "hbm", "kernel": "prune_axis0_bf16_kernel", "achieved": prune_gbs,
                               "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": prune_gbs / peaks["hbm_gbs"],
                               "peak_source": peaks["source"],
                               "traffic": ncu_traffic("prune_axis0_bf16_kernel/" + args.joint, args.workload)
                               if (n, m) == (2, 4) else None},
        }
        if alone_ms is not None:
            agbs = p_bytes / (alone_ms * 1e-3) / 1e9
            line["prune_alone"] = {"joint": args.joint, "ms": alone_ms, "gbs": agbs,
                                   "frac_of_hbm_peak": agbs / peaks["hbm_gbs"],
                                   "note": "the step's prune launched back to back, L2-cold, without the product"}
        for other in others:
            ogbs = p_bytes / (other[1] * 1e-3) / 1e9
            key = {"table": "prune_other_joint", "systematic": "prune_other_joint", "1:2": "prune_1of2", "1:4": "prune_1of4"}.get(
                other[0], "prune_" + other[0])
            line[key] = {"joint": other[0], "ms": other[1], "gbs": ogbs,
                         "frac_of_hbm_peak": ogbs / peaks["hbm_gbs"], "steps": other[2]}
        if world == 1 and not args.no_extra:
            line["ffn_large"] = tensor_bound_case(n, m, peaks, joint[0])
            line["mlp_stack"] = chain_case(n, m)
        if world == 1 and args.sweep:
            line["prune_sweep"] = prune_sweep(peaks)
        if world == 1 and not args.no_cpu_baseline:
            sample_rows = min(T, 65536)
            gbs, threads, dt = oracle_sample(cfg, n, m, sample_rows, joint[0])
            line["cpu_baseline"] = {"value": gbs, "unit": "GB/s", "cores": threads, "kind": "oracle",
                                    "sample": f"first {sample_rows} of {T} token rows: MVUE {n}:{m} prune+pack and "
                                              f"fp64 update product [{out}x{inp}], {dt:.1f} s"}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def tensor_bound_case(n, m, peaks, joint):
    """The large FFN layer (tokens 16384, 4096 -> 14336): the shape on which the sparse product is bound by
    the tensor cores, timed kernel by kernel next to dense cuBLAS.  Rides along in the JSON line."""
    import torch
    from paper_2203_10991_b200 import binding, workloads
    cfg = workloads.CONFIGS["ffn_large"]
    T, out, inp = cfg["T"], cfg["out"], cfg["inp"]
    TC = binding.MVUE_LAYOUT_TC
    g = torch.from_numpy(workloads.gradient((T, out), cfg["g_dist"], cfg["seed"], dtype="bf16").view(np.int16))
    g = g.cuda().view(torch.bfloat16)
    h = torch.from_numpy(workloads.normal_bf16((T, inp), cfg["seed"] + 100).view(np.int16)).cuda().view(torch.bfloat16)
    values, meta = binding.mvue_prune(g, n, m, 0, 0, layout=TC)
    dW = torch.empty((out, inp), dtype=torch.float32, device="cuda")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(fn, iters):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters

    prune_ms = timed(lambda: binding.mvue_prune(g, n, m, 0, 1, values=values, meta=meta, layout=TC, joint=joint), 20)
    sys_ms = timed(lambda: binding.mvue_prune(g, n, m, 0, 1, values=values, meta=meta, layout=TC,
                                              joint=binding.MVUE_JOINT_SYSTEMATIC), 20)
    table_ms = timed(lambda: binding.mvue_prune(g, n, m, 0, 1, values=values, meta=meta, layout=TC,
                                                joint=binding.MVUE_JOINT_TABLE), 20)
    binding.mvue_prune(g, n, m, 0, 1, values=values, meta=meta, layout=TC, joint=joint)
    gemm_ms = timed(lambda: binding.mvue_sparse_update_gemm(values, meta, h, out=dW), 30)
    fused_ms = timed(lambda: binding.mvue_fused_update_gemm(g, h, n, m, 1, out=dW), 3)
    gT = g.t()
    dense_ms = timed(lambda: torch.matmul(gT, h), 30)
    # what the sparse tensor cores retire when nothing is loaded (zeros in shared memory, so no power throttling
    # either): the ceiling of any tiling, above what real operands can reach under the power cap
    probe_status = torch.zeros(1, dtype=torch.int32, device="cuda")
    probe_iters = 4096
    _, probe_flops = binding.mvue_probe_sparse_mma(probe_iters, probe_status)
    probe_ms = min(timed(lambda: binding.mvue_probe_sparse_mma(probe_iters, probe_status), 1) for _ in range(5))
    assert int(probe_status.item()) == 0
    issue_ceiling = probe_flops / (probe_ms * 1e-3) / 1e12
    flops = 2.0 * out * inp * T
    tf = flops / (gemm_ms * 1e-3) / 1e12
    pgbs = prune_bytes(T, out, 2) / (prune_ms * 1e-3) / 1e9
    return {"g": [T, out], "h": [T, inp], "prune": f"{n}:{m}",
            "prune_ms": prune_ms, "prune_gbs": pgbs, "prune_frac_of_hbm_peak": pgbs / peaks["hbm_gbs"],
            "prune_systematic_ms": sys_ms,
            "prune_systematic_frac_of_hbm_peak": prune_bytes(T, out, 2) / (sys_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "prune_table_ms": table_ms,
            "prune_table_frac_of_hbm_peak": prune_bytes(T, out, 2) / (table_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "gemm_ms": gemm_ms, "gemm_tflops_effective": tf,
            "gemm_frac_of_sparse_peak_burst": tf / (2 * peaks["bf16_tflops"]),
            "gemm_frac_of_sparse_peak_sustained": tf / (2 * peaks["bf16_tflops_sustained"]),
            "sparse_mma_issue_ceiling_tflops": issue_ceiling,
            "gemm_frac_of_issue_ceiling": tf / issue_ceiling,
            "dense_cublas_ms": dense_ms, "dense_cublas_tflops": flops / (dense_ms * 1e-3) / 1e12,
            # three-way comparison: separate prune + sparse product vs the fused kernel vs dense cuBLAS
            "separate_ms": prune_ms + gemm_ms, "fused_ms": fused_ms,
            "fused_tflops_effective": flops / (fused_ms * 1e-3) / 1e12,
            "roofline": {"bound": "tensor", "kernel": "sparse_gemm_pair_kernel", "achieved": tf,
                         "peak": 2 * peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": tf / (2 * peaks["bf16_tflops"]),
                         "peak_source": peaks["source"] + " dense bf16 burst x 2 (2:4 sparse)", "traffic": None}}


def prune_sweep(peaks, max_log2: int = 32):
    """Standalone prune+pack bandwidth over bf16 tensors of 2^20 .. 2^max_log2 bytes ([bytes / 8192 x 4096],
    Student-t values), both pruned axes, 2:4 (pair table, systematic sampling), 1:2 and 1:4.  Every point is a CUDA graph of
    `reps` launches over rotating input copies that together exceed 2.5 x L2, replayed and timed with events, so the
    small sizes are neither launch-bound on the host nor L2-warm."""
    import torch
    from paper_2203_10991_b200 import binding, workloads
    dev = torch.device("cuda")
    TC = binding.MVUE_LAYOUT_TC
    l2 = 126e6
    cols = 4096
    # 256 MB of seeded values drawn on the host, tiled on the device up to the largest tensor
    seed_rows = 1 << 15
    base = workloads.gradient((seed_rows, cols), "student_t", 5, dtype="bf16")
    base_dev = torch.from_numpy(base.view(np.int16)).to(dev).view(torch.bfloat16)
    total_rows = 1 << (max_log2 - 13)
    if total_rows > seed_rows:
        base_dev = base_dev.repeat(total_rows // seed_rows, 1)
    out_v = torch.empty(base_dev.numel() // 2, dtype=torch.bfloat16, device=dev)
    out_m = torch.empty(base_dev.numel() // 8 + (1 << 16), dtype=torch.uint8, device=dev)
    modes = [("2:4 table", 2, 4, binding.MVUE_JOINT_TABLE), ("2:4 systematic", 2, 4, binding.MVUE_JOINT_SYSTEMATIC),
             ("1:2", 1, 2, binding.MVUE_JOINT_TABLE), ("1:4", 1, 4, binding.MVUE_JOINT_TABLE)]
    points = []
    side = torch.cuda.Stream()
    for lg in range(20, max_log2 + 1):
        nbytes = 1 << lg
        rows = nbytes // (2 * cols)
        copies = max(1, min(int(2.5 * l2 / nbytes) + 1, (base_dev.numel() * 2) // nbytes))
        reps = max(4, min(64, copies))
        views = [base_dev[i * rows:(i + 1) * rows] for i in range(copies)]
        point = {"bytes": nbytes, "shape": [rows, cols], "copies": copies}
        for axis in (0, 1):
            mrows, k = (rows, cols) if axis == 1 else (cols, rows)
            values = out_v[:mrows * k // 2].view(mrows, k // 2)
            for name, n, m, joint in modes:
                def burst():
                    for i in range(reps):
                        binding.mvue_prune(views[i % copies], n, m, axis, i, values=values, meta=out_m, layout=TC,
                                           joint=joint)
                side.wait_stream(torch.cuda.current_stream())
                with torch.cuda.stream(side):
                    burst()
                torch.cuda.current_stream().wait_stream(side)
                torch.cuda.synchronize()
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph):
                    burst()
                graph.replay()
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                graph.replay()
                e1.record()
                torch.cuda.synchronize()
                us = e0.elapsed_time(e1) * 1e3 / reps
                gbs = prune_bytes(rows, cols, 2) / us / 1e3
                point[f"axis{axis} {name}"] = {"us": round(us, 2), "gbs": round(gbs, 1),
                                               "frac_of_hbm_peak": round(gbs / peaks["hbm_gbs"], 4)}
                del graph
        points.append(point)
    return {"dtype": "bf16", "cols": cols, "dist": "student_t", "layout": "tensor-core metadata order",
            "timing": "CUDA graph replay, inputs rotated over > 2.5 x L2 where the tensor is smaller than that",
            "points": points}


def chain_case(n, m):
    """The MLP-stack workload: backward + update chain of 12 blocks x (1024 -> 4096, activation, 4096 -> 1024) over
    T = 32768 tokens, every neural gradient MVUE-pruned (prune along tokens -> sparse update product; independent
    prune along the features -> sparse backward product with the f'(z) epilogue), timed as a whole next to the same
    chain with dense bf16 matmuls.  Activations and f'(z) are seeded random tensors of the right shapes (the forward
    pass is not part of the path)."""
    import torch
    from paper_2203_10991_b200 import binding, chain, workloads
    cfg = workloads.CONFIGS["mlp_stack"]
    T, d_ff, d = cfg["T"], cfg["out"], cfg["inp"]
    dev = torch.device("cuda")
    gen = torch.Generator(device=dev).manual_seed(cfg["seed"])
    layers = []
    for i in range(2 * cfg["layers"]):                      # top layer first: [d <- d_ff], [d_ff <- d], ...
        out_f, in_f = (d, d_ff) if i % 2 == 0 else (d_ff, d)
        layers.append({
            "W": (torch.randn((out_f, in_f), generator=gen, device=dev) * in_f ** -0.5).to(torch.bfloat16),
            "h": torch.randn((T, in_f), generator=gen, device=dev).to(torch.bfloat16),
            "act_grad": None if i == 2 * cfg["layers"] - 1 else
                        torch.rand((T, in_f), generator=gen, device=dev).to(torch.bfloat16)})
    g_host = workloads.gradient((T, d), cfg["g_dist"], cfg["seed"], dtype="bf16")
    g_top = torch.from_numpy(g_host.view(np.int16)).to(dev).view(torch.bfloat16)

    def dense_chain():
        g = g_top
        for L in layers:
            torch.matmul(g.t(), L["h"])
            if L["act_grad"] is not None:
                g = torch.matmul(g, L["W"]) * L["act_grad"]

    def timed(fn, iters):
        fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters

    def graphed(fn):
        """The chain is ~94 short launches: replayed from a CUDA graph so that the device, not the Python caller, is
        what is timed (the eager figure rides along)."""
        fn()
        torch.cuda.synchronize()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            fn()                                            # warm the allocator on the capture stream
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            fn()
        return graph.replay

    def run_table():
        chain.backward_update(g_top, layers, n, m, base_seed=1)

    def run_sys():
        chain.backward_update(g_top, layers, n, m, base_seed=1, joint=binding.MVUE_JOINT_SYSTEMATIC)

    def run_sys_overlap():
        chain.backward_update(g_top, layers, n, m, base_seed=1, joint=binding.MVUE_JOINT_SYSTEMATIC, overlap=True)

    eager_ms = timed(run_table, 5)
    table_ms = timed(graphed(run_table), 10)
    sys_ms = timed(graphed(run_sys), 10) if m == 4 else None
    overlap_ms = timed(graphed(run_sys_overlap), 10) if m == 4 else None
    dense_ms = timed(graphed(dense_chain), 10)
    n_layers = len(layers)
    flops = 2.0 * T * d * d_ff * (2 * n_layers - 1)         # update product per layer, backward for all but the bottom
    return {"layers": n_layers, "T": T, "d": d, "d_ff": d_ff, "prune": f"{n}:{m}",
            "launches_per_chain": 4 * n_layers - 2,
            "timing": "CUDA graph replay", "eager_ms": eager_ms,
            "ms": table_ms, "tflops_effective": flops / (table_ms * 1e-3) / 1e12,
            "systematic_ms": sys_ms,
            "systematic_tflops_effective": None if sys_ms is None else flops / (sys_ms * 1e-3) / 1e12,
            # the same chain with each update product on a second stream beside the next axis-1 prune
            "systematic_two_stream_ms": overlap_ms,
            "systematic_two_stream_tflops_effective": None if overlap_ms is None else flops / (overlap_ms * 1e-3) / 1e12,
            "dense_torch_ms": dense_ms, "dense_torch_tflops": flops / (dense_ms * 1e-3) / 1e12}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="conv_im2col")
    ap.add_argument("--prune", default="2:4")
    ap.add_argument("--joint", default="systematic", choices=["table", "systematic", "approx"],
                    help="2:4 estimator used by the step: systematic sampling (the faster of the two exact MVUE laws), "
                         "the App. A.2 pair table, or approx-MVUE (Sec. 4.4); the others are timed beside it")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep", action="store_true",
                    help="add the standalone prune+pack bandwidth sweep over bf16 tensors of 1 MB .. 4 GB")
    ap.add_argument("--no-extra", action="store_true",
                    help="skip the riders: the other 2:4 law, the tensor-bound ffn_large case and the MLP-stack chain")
    args = ap.parse_args()
    from paper_2203_10991_b200 import workloads
    cfg = workloads.CONFIGS[args.workload]
    n, m = (int(x) for x in args.prune.split(":"))
    if args.impl == "reference":
        args.steps = 3 if args.steps is None else args.steps
        run_reference(args, cfg, n, m)
    else:
        args.steps = 1000 if args.steps is None else args.steps
        run_ours(args, cfg, n, m)


if __name__ == "__main__":
    main()
