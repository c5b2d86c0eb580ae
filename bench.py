#!/usr/bin/env python
"""Benchmark of the MVUE hot path on B200: prune+pack of the neural gradient followed by the
2:4-sparse products that consume it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME] [--prune n:m]

Prints ONE JSON line.  A step is one pass of the whole path over one synthetic batch of the
`conv_im2col` workload: g bf16 [200704 x 256] (ReLU-sparse lognormal), h bf16 [200704 x 2304]:
    values, meta = mvue_prune(g, 2:4, along the token axis)      # Sec. 4.2 / App. A.2
    dW[256 x 2304] = theta(g)^T h                                  # Sec. 1, update equation
`value` is the metric's first half: the prune+pack kernel's algorithmic GB/s inside that step, inputs resident in
HBM (every step reads 925 MB of h in between, so the prune never finds g in L2).  The whole step's bytes per
second, the product's GB/s (this shape is HBM-bound) and effective TFLOP/s, dense cuBLAS for the same shape and the
other workloads (small linear layer, transformer FFN, large FFN, MLP-stack chain, three sizes of the prune sweep)
ride along in the same line.  `e2e` repeats the step through the same C-ABI calls from pinned host buffers with the
copies inside the timed region.  `--impl reference` times the CPU oracle on a bounded sample.
With --gpus N (> 1) and no torchrun environment the script starts its own N ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

METRIC = "prune+pack GB/s (% HBM peak); MVUE-sparse GEMM TFLOP/s vs dense bf16"
L2_BYTES = 126e6
NOMINAL_SPARSE_BF16_TFLOPS = 4500.0      # dense 2250 x 2 (2:4)


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


def gemm_bytes(M: int, N: int, K: int, c_bytes: int = 4, scale: bool = False) -> int:
    """Minimum traffic of C[MxN] = A_packed[MxK] . B[KxN] (* E[MxN]): survivors, metadata, B, C (and E) once each."""
    return M * K + M * K // 8 + K * N * 2 + M * N * c_bytes + (M * N * 2 if scale else 0)


# dram__bytes_read.sum + dram__bytes_write.sum per launch on the conv_im2col workload, from one ncu capture of
# each kernel (summaries under profiles/).  Each figure is tied to a digest of the sources the kernel is built
# from: once those change the counters no longer describe the kernel and `traffic` is reported as null.
NCU_TRAFFIC = {
    "sparse_gemm_pair_kernel": (982859520 + 4034048, ("mvue_gemm.cu", "mvue_tma.h", "mvue_internal.h"),
                                "14864604f8e1a0f7"),
    "prune_axis0_bf16_whole_tiles_kernel/table/16": (102822144 + 27183872,
                                                     ("mvue_prune.cu", "mvue_device.cuh", "mvue_tma.h", "mvue_internal.h"),
                                                     "65483dfb9e3e781a"),
    "prune_axis0_bf16_whole_tiles_kernel/systematic/16": (102779136 + 20355328,
                                                          ("mvue_prune.cu", "mvue_device.cuh", "mvue_tma.h",
                                                           "mvue_internal.h"),
                                                          "65483dfb9e3e781a"),
}


def source_digest(sources) -> str:
    import hashlib
    h = hashlib.sha256()
    for name in sources:
        h.update((ROOT / "paper_2203_10991_b200" / "csrc" / name).read_bytes())
    return h.hexdigest()[:16]


def ncu_traffic(kernel: str, workload: str):
    if workload != "conv_im2col" or kernel not in NCU_TRAFFIC:
        return None
    nbytes, sources, digest = NCU_TRAFFIC[kernel]
    return nbytes if source_digest(sources) == digest else None


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

    def _sample(self):
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
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

    def _loop(self):
        while not self._stop.is_set():
            self._sample()
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
        if self.nv is not None and not self.samples:
            self._sample()

    def summary(self):
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# --------------------------------------------------------------------------- CPU oracle arm
def oracle_sample(cfg, n, m, sample_rows: int, joint: int = 0, prune_repeats: int = 1, eps16: bool = False):
    """One pass of the oracle, as it stands, over the first `sample_rows` token rows: prune+pack (repeated
    `prune_repeats` times so that the timed work is seconds, not milliseconds), unpack, and the fp64 plain-loop update
    product.  Returns (GB/s of the prune+pack's algorithmic bytes, GB/s of one whole pass, threads, seconds of one
    pass, seconds of all the prune+pack repeats)."""
    import oracle
    from paper_2203_10991_b200 import workloads
    g = workloads.gradient((sample_rows, cfg["out"]), cfg["g_dist"], cfg["seed"], dtype=cfg["g_dtype"])
    h = workloads.normal_bf16((sample_rows, cfg["inp"]), cfg["seed"] + 100)
    threads = oracle.host_threads()
    t0 = time.perf_counter()
    for rep in range(prune_repeats):
        values, meta = oracle.prune(g, n, m, axis=0, seed=rep, k_total=cfg["T"], k_offset=0, threads=threads, joint=joint,
                                    eps16=eps16)
    t1 = time.perf_counter()
    oracle.gemm(oracle.unpack(values, meta), h, threads=threads)
    t2 = time.perf_counter()
    p_bytes = prune_bytes(sample_rows, cfg["out"], 2 if cfg["g_dtype"] == "bf16" else 4)
    nbytes = p_bytes + gemm_bytes(cfg["out"], cfg["inp"], sample_rows)
    dt = (t1 - t0) / prune_repeats + (t2 - t1)
    return prune_repeats * p_bytes / (t1 - t0) / 1e9, nbytes / dt / 1e9, threads, dt, t1 - t0


def run_reference(args, cfg, n, m):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    joint = JOINT_IDS[args.joint]
    # size the per-step sample so that K + W steps of the oracle take about a minute in all: its cost
    # grows faster than linearly with the rows (the plain loops leave the cache), so probe by doubling
    per_step_s = 60.0 / max(1, args.steps + args.warmup)
    sample_rows = 512
    while sample_rows * 2 <= cfg["T"]:
        dt_probe = oracle_sample(cfg, n, m, sample_rows, joint, eps16=args.eps16)[3]
        if dt_probe > per_step_s / 3:
            break
        sample_rows *= 2
    for _ in range(args.warmup):
        oracle_sample(cfg, n, m, sample_rows, joint, eps16=args.eps16)
    vals, steps_gbs, t_all, threads = [], [], 0.0, 1
    for _ in range(args.steps):
        p_gbs, s_gbs, threads, dt, _ = oracle_sample(cfg, n, m, sample_rows, joint, prune_repeats=20, eps16=args.eps16)
        vals.append(p_gbs)
        steps_gbs.append(s_gbs)
        t_all += dt
    value = float(np.mean(vals))
    sample = (f"first {sample_rows} of {cfg['T']} token rows: MVUE {n}:{m} prune+pack of g[{sample_rows}x{cfg['out']}] "
              f"(20 passes timed: the value) and the fp64 update product with h[{sample_rows}x{cfg['inp']}] (ms_per_step: one whole pass)")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_all / max(1, args.steps),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "prune": f"{n}:{m}", "joint": args.joint,
                   "random_bits_per_block": 16 if args.eps16 else 32, "axis": 0, "sample_rows": sample_rows},
        "step_gbs": float(np.mean(steps_gbs)),
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


JOINT_IDS = {"table": 0, "systematic": 1, "approx": 2}


# --------------------------------------------------------------------------- timing helpers
class Timer:
    """CUDA-event timing on the current stream.  Every timed iteration is preceded by an L2 flush (a write over
    a buffer larger than L2) unless the caller rotates or streams inputs larger than L2 itself."""

    def __init__(self, dev):
        import torch
        self.torch = torch
        self.flush_buf = torch.empty(int(2.2 * L2_BYTES), dtype=torch.uint8, device=dev)

    def flush(self):
        self.flush_buf.fill_(1)

    def each(self, fn, iters: int, flush: bool = True, warm: int = 3):
        """Times every call of fn on its own pair of events; returns (mean_ms, best_ms)."""
        torch = self.torch
        for _ in range(warm):
            fn()
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
        torch.cuda.synchronize()
        for a, b in evs:
            if flush:
                self.flush()
            a.record()
            fn()
            b.record()
        torch.cuda.synchronize()
        t = [a.elapsed_time(b) for a, b in evs]
        return float(np.mean(t)), float(np.min(t))

    def loop(self, fn, iters: int, warm: int = 3):
        """fn back to back, one pair of events around the loop; returns ms per call."""
        torch = self.torch
        for _ in range(warm):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters


def bf16_dev(a: np.ndarray, dev):
    import torch
    return torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)


def hbm_roofline(kernel, nbytes, ms, peaks, traffic=None):
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"bound": "hbm", "kernel": kernel, "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": gbs / peaks["hbm_gbs"], "peak_source": peaks["source"] + " copy bandwidth", "traffic": traffic}


def tensor_roofline(kernel, flops, ms, peaks, issue_cold_tflops):
    """Dense-equivalent TFLOP/s of a sparse product against the rate at which this GPU retires the very instruction
    of the kernel with nothing to load (measured cold at the start of the run; the nominal sparse bf16 rate if the
    probe did not run).  The fraction of twice the measured dense cuBLAS rate rides along under its own name."""
    tf = flops / (ms * 1e-3) / 1e12
    peak = issue_cold_tflops if issue_cold_tflops else NOMINAL_SPARSE_BF16_TFLOPS
    return {"bound": "tensor", "kernel": kernel, "achieved": tf, "peak": peak, "unit": "TFLOP/s", "frac": tf / peak,
            "peak_source": ("sparse tcgen05.mma issue-rate probe of this run, cold" if issue_cold_tflops
                            else "nominal sparse bf16"),
            "frac_of_nominal_sparse_bf16": tf / NOMINAL_SPARSE_BF16_TFLOPS,
            "frac_of_2x_dense_cublas_burst": tf / (2 * peaks["bf16_tflops"]),
            "frac_of_2x_dense_cublas_sustained": tf / (2 * peaks["bf16_tflops_sustained"]),
            "traffic": None}


def issue_probe(binding, tm: Timer):
    """Dense-equivalent TFLOP/s of the sparse MMA issue-rate probe (best of 5 launches)."""
    import torch
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    iters = 4096
    _, flops = binding.mvue_probe_sparse_mma(iters, st)
    ms = min(tm.loop(lambda: binding.mvue_probe_sparse_mma(iters, st), 1, warm=1) for _ in range(5))
    assert int(st.item()) == 0
    return flops / (ms * 1e-3) / 1e12


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
    tm = Timer(dev)
    solo = world == 1 and rank == 0
    extras = solo and not args.no_extra
    issue_cold = issue_probe(binding, tm) if extras else None      # before anything has warmed the GPU up

    T, out, inp = cfg["T"], cfg["out"], cfg["inp"]
    elem = 2 if cfg["g_dtype"] == "bf16" else 4
    # data parallel over tokens (weak scaling): every rank holds its own token shard of a batch of world x T tokens and
    # prunes it under the global block numbering (k_total = world T, k_offset = rank T), so the masks are those of the
    # unsharded batch; the partial dW are summed by one all-reduce
    k_total, k_offset = world * T, rank * T
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
    base_opt = binding.MVUE_OPT_EPS16 if args.eps16 else binding.MVUE_OPT_NONE
    opts = [base_opt]

    def step(i, ev=None):
        if ev:
            ev[0].record()
        binding.mvue_prune(g_dev, nm[0][0], nm[0][1], 0, i, k_total=k_total, k_offset=k_offset, values=values,
                           meta=meta, layout=TC, joint=joint[0], options=opts[0])
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

    def step_kernel_times(k):
        """k steps, each kernel bracketed by events: per-step (prune_ms, gemm_ms) lists."""
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(k)]
        torch.cuda.synchronize()
        for i in range(k):
            step(i, evs[i])
        torch.cuda.synchronize()
        return [e[0].elapsed_time(e[1]) for e in evs], [e[1].elapsed_time(e[2]) for e in evs]

    warm = max(3, args.warmup)
    for i in range(warm):
        step(i)
    barrier()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local, period_s=0.002) as clocks:
        barrier()
        ev0.record()
        for i in range(args.steps):
            step(i, evs[i])
        ev1.record()
        barrier()
    assert int(status.item()) == 0, "a bounded device-side wait expired"
    ms = ev0.elapsed_time(ev1)
    prune_times = [e[0].elapsed_time(e[1]) for e in evs]
    gemm_times = [e[1].elapsed_time(e[2]) for e in evs]
    prune_ms, gemm_ms = float(np.mean(prune_times)), float(np.mean(gemm_times))
    if world > 1:
        t = torch.tensor([ms, prune_ms], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms, prune_ms = float(t[0].item()), float(t[1].item())
    ms_per_step = ms / args.steps
    step_gbs = world * step_bytes / (ms_per_step * 1e-3) / 1e9
    value = world * p_bytes / (prune_ms * 1e-3) / 1e9           # the metric: prune+pack GB/s, all ranks

    # the step back to back for at least a second with the clock sampler running: what the path sustains
    sustained = None
    if extras:
        k_s = max(50, int(1.2e3 / ms_per_step))
        with ClockSampler(local, period_s=0.01) as clocks_s:
            pt, gt = step_kernel_times(k_s)
        sustained = {"steps": k_s, "seconds": 1e-3 * (sum(pt) + sum(gt)),
                     "prune_ms_mean": float(np.mean(pt)), "prune_ms_best": float(np.min(pt)),
                     "prune_gbs": p_bytes / (float(np.mean(pt)) * 1e-3) / 1e9,
                     "prune_frac_of_hbm_peak": p_bytes / (float(np.mean(pt)) * 1e-3) / 1e9 / measured_peaks()["hbm_gbs"],
                     "gemm_ms_mean": float(np.mean(gt)), "gemm_ms_best": float(np.min(gt)),
                     "clocks": clocks_s.summary()}

    # the same step with the other estimators, for the per-kernel prune time only (the product that
    # follows keeps L2 cold for the next prune exactly as in the timed region above)
    others = []
    if extras and m == 4:
        k2 = max(20, min(args.steps, 200))
        variants = [(name, (2, 4), jid, base_opt) for name, jid in joints.items() if name != args.joint]
        variants += [("1:2", (1, 2), joints[args.joint], base_opt), ("1:4", (1, 4), joints[args.joint], base_opt),
                     # the step's law with the survivors rounded to bf16 stochastically (unbiased storage)
                     ("stochastic_rounding", (2, 4), joints[args.joint], base_opt | binding.MVUE_OPT_STOCHASTIC_ROUNDING),
                     # and with the other width of the random stream (32 bits per block if the step draws 16, and back)
                     ("eps32" if args.eps16 else "eps16", (2, 4), joints[args.joint], base_opt ^ binding.MVUE_OPT_EPS16)]
        for name, nm_v, jid, opt in variants:
            joint[0], nm[0], opts[0] = jid, nm_v, opt
            for i in range(3):
                step(i)
            pt, _ = step_kernel_times(k2)
            others.append((name, float(np.mean(pt)), float(np.min(pt)), k2))
        joint[0], nm[0], opts[0] = joints[args.joint], (n, m), base_opt

    # the step's prune timed alone (no product in between), L2-cold: inputs rotated over copies of g that together
    # exceed 2.5 x L2
    alone = None
    if extras:
        copies = max(2, int(2.5 * L2_BYTES / (T * out * elem)) + 1)
        gs = [g_dev.clone() for _ in range(copies)]
        it = [0]

        def prune_rot():
            binding.mvue_prune(gs[it[0] % copies], n, m, 0, it[0], values=values, meta=meta, layout=TC, joint=joint[0],
                               options=base_opt)
            it[0] += 1
        alone_loop = tm.loop(prune_rot, max(20, min(args.steps, 100)))
        alone_mean, alone_best = tm.each(prune_rot, 20, flush=False)
        alone = (alone_loop, alone_mean, alone_best)
        del gs

    # dense cuBLAS bf16 for the same shape (context for the sparse product)
    dense_ms = None
    if rank == 0 and elem == 2:
        gT = g_dev.t()
        dense_ms = tm.loop(lambda: torch.matmul(gT, h_dev), 10)

    # end to end: pinned host g and h -> device -> prune -> GEMM -> dW back to pinned host
    g_pin, h_pin = g_t.pin_memory(), h_t.pin_memory()
    dW_pin = torch.empty((out, inp), dtype=torch.float32).pin_memory()
    e2e_steps = max(2, min(args.steps, 5))
    e2e_evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(e2e_steps)]

    def e2e_step(i, ev=None):
        g_dev.view(torch.int16 if elem == 2 else torch.float32).copy_(g_pin, non_blocking=True)
        h_dev.view(torch.int16).copy_(h_pin, non_blocking=True)
        step(i, ev)
        dW_pin.copy_(dW, non_blocking=True)

    e2e_step(0)
    barrier()
    ev0.record()
    for i in range(e2e_steps):
        e2e_step(i, e2e_evs[i])
    ev1.record()
    barrier()
    e2e_ms = ev0.elapsed_time(ev1)
    if world > 1:
        t = torch.tensor([e2e_ms], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms = float(t.item())
    # the same metric (prune+pack bytes per second), with everything a caller pays per step in the denominator:
    # the host -> device copies, the prune, the product that consumes it and the device -> host read of dW
    e2e_value = world * p_bytes / (e2e_ms / e2e_steps * 1e-3) / 1e9
    e2e_step_gbs = world * step_bytes / (e2e_ms / e2e_steps * 1e-3) / 1e9

    if rank == 0:
        peaks = measured_peaks()
        prune_gbs = p_bytes / (prune_ms * 1e-3) / 1e9
        gemm_gbs = m_bytes / (gemm_ms * 1e-3) / 1e9
        gemm_tf = gemm_flops / (gemm_ms * 1e-3) / 1e12
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": warm, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": args.workload, "g": [T, out], "h": [T, inp], "g_dtype": cfg["g_dtype"],
                       "prune": f"{n}:{m}", "joint": args.joint, "random_bits_per_block": 16 if args.eps16 else 32,
                       "axis": 0, "dW_dtype": "f32",
                       "value_is": "prune+pack kernel GB/s (algorithmic bytes: g read, survivors + metadata written) "
                                   "measured inside the step, mean over the timed steps",
                       "k_total": k_total, "k_offset_of_rank0": 0,
                       "l2": "inputs larger than L2 (h is 925 MB, read once per step between two prunes)"},
            "value_frac_of_hbm_peak": value / world / peaks["hbm_gbs"],
            "step": {"gbs": step_gbs, "bytes": step_bytes,
                     "note": "prune + product algorithmic bytes over the whole step's time"},
            "clocks": clocks.summary(),
            "e2e": {"value": e2e_value, "unit": "GB/s", "h2d_bytes_per_step": T * out * elem + T * inp * 2,
                    "d2h_bytes_per_step": out * inp * 4, "step_gbs": e2e_step_gbs,
                    "note": "prune+pack bytes over the time of the whole step from pinned host buffers "
                            "(copies in, prune, product, dW out)"},
            "gpu_launches": args.steps * launches_per_step,
            "prune": {"joint": args.joint, "ms": prune_ms, "ms_best": float(np.min(prune_times)), "gbs": prune_gbs,
                      "frac_of_hbm_peak": prune_gbs / peaks["hbm_gbs"]},
            "gemm": {"ms": gemm_ms, "ms_best": float(np.min(gemm_times)), "tflops_effective": gemm_tf, "gbs": gemm_gbs,
                     "frac_of_hbm_peak": gemm_gbs / peaks["hbm_gbs"],
                     "dense_cublas_ms": dense_ms,
                     "dense_cublas_tflops": None if dense_ms is None else gemm_flops / (dense_ms * 1e-3) / 1e12},
            # the dominant kernel of the step is the sparse product; on this shape (256 x 2304 outputs over
            # 200704 rows, ~240 flop/B) it is bound by streaming h from HBM, not by the tensor cores
            "roofline": hbm_roofline("sparse_gemm_pair_kernel", m_bytes, gemm_ms, peaks,
                                     ncu_traffic("sparse_gemm_pair_kernel", args.workload) if (n, m) == (2, 4) else None),
            "roofline_prune": hbm_roofline("prune_axis0_bf16_whole_tiles_kernel", p_bytes, prune_ms, peaks,
                                           ncu_traffic(f"prune_axis0_bf16_whole_tiles_kernel/{args.joint}/{16 if args.eps16 else 32}", args.workload)
                                           if (n, m) == (2, 4) else None),
        }
        if sustained is not None:
            line["sustained"] = sustained
        if alone is not None:
            agbs = p_bytes / (alone[0] * 1e-3) / 1e9
            line["prune_alone"] = {"joint": args.joint, "ms": alone[0], "ms_each_mean": alone[1], "ms_each_best": alone[2],
                                   "gbs": agbs, "frac_of_hbm_peak": agbs / peaks["hbm_gbs"],
                                   "note": "the step's prune launched back to back, L2-cold (inputs rotated), no product"}
        for name, mean_ms, best_ms, k2 in others:
            ogbs = p_bytes / (mean_ms * 1e-3) / 1e9
            key = {"1:2": "prune_1of2", "1:4": "prune_1of4"}.get(name, "prune_" + name)
            line[key] = {"estimator": name, "ms": mean_ms, "ms_best": best_ms, "gbs": ogbs,
                         "frac_of_hbm_peak": ogbs / peaks["hbm_gbs"], "steps": k2}
        if extras:
            line["sparse_issue_rate_cold_tflops"] = issue_cold
            line["linear_small"] = linear_small_case(tm, peaks)
            line["ffn_768"] = ffn_768_case(tm, peaks, issue_cold, joint[0])
            line["ffn_large"] = tensor_bound_case(tm, n, m, peaks, joint[0], issue_cold, base_opt)
            line["mlp_stack"] = chain_case(n, m)
            line["prune_sweep"] = prune_sweep(peaks, sizes_log2=(26, 29, 32) if not args.sweep else range(20, 33),
                                              step_joint=joint[0], options=base_opt)
        if solo and args.gemm_shapes:
            line["gemm_shapes"] = gemm_shapes_case(tm, peaks, issue_cold)
        if solo and not args.no_cpu_baseline:
            sample_rows = min(T, 65536)
            reps = 200
            p_gbs, s_gbs, threads, dt, dt_prune = oracle_sample(cfg, n, m, sample_rows, joint[0], prune_repeats=reps, eps16=args.eps16)
            line["cpu_baseline"] = {"value": p_gbs, "unit": "GB/s", "cores": threads, "kind": "oracle",
                                    "step_gbs": s_gbs,
                                    "sample": f"first {sample_rows} of {T} token rows: MVUE {n}:{m} prune+pack, {reps} passes "
                                              f"({dt_prune:.1f} s, the value), and one fp64 update product "
                                              f"[{out}x{inp}] over those rows (one whole pass: {dt:.1f} s, step_gbs)"}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def linear_small_case(tm: Timer, peaks):
    """The single small linear layer: g binary32 [512 x 256] (ReLU-sparse normal), MVUE 1:2 along the tokens, then
    dW[256 x 256] = theta(g)^T h.  Launch-bound: times are per call with L2 flushed before each."""
    import torch
    from paper_2203_10991_b200 import binding, workloads
    cfg = workloads.CONFIGS["linear_small"]
    T, out, inp = cfg["T"], cfg["out"], cfg["inp"]
    TC = binding.MVUE_LAYOUT_TC
    g = torch.from_numpy(workloads.gradient((T, out), cfg["g_dist"], cfg["seed"], dtype="f32")).cuda()
    h = bf16_dev(workloads.normal_bf16((T, inp), cfg["seed"] + 100), "cuda")
    values, meta = binding.mvue_prune(g, 1, 2, 0, 0, layout=TC)
    dW = torch.empty((out, inp), dtype=torch.float32, device="cuda")
    ws = torch.empty(max(16, binding.mvue_gemm_workspace_bytes(0, out, inp, T)), dtype=torch.uint8, device="cuda")
    p_mean, p_best = tm.each(lambda: binding.mvue_prune(g, 1, 2, 0, 0, values=values, meta=meta, layout=TC), 20)
    g_mean, g_best = tm.each(lambda: binding.mvue_sparse_update_gemm(values, meta, h, out=dW, workspace=ws), 20)
    gT = g.t().to(torch.bfloat16).contiguous()
    d_mean, d_best = tm.each(lambda: torch.matmul(gT, h), 20)
    flops = 2.0 * out * inp * T
    return {"g": [T, out], "g_dtype": "f32", "prune": "1:2", "timing": "per call, L2 flushed before each; mean / best of 20",
            "prune_us": 1e3 * p_mean, "prune_us_best": 1e3 * p_best,
            "roofline_prune": hbm_roofline("prune_axis0_kernel", prune_bytes(T, out, 4), p_best, peaks),
            "gemm_us": 1e3 * g_mean, "gemm_us_best": 1e3 * g_best, "gemm_tflops_effective": flops / (g_best * 1e-3) / 1e12,
            "roofline_gemm": hbm_roofline("sparse_gemm_pair_kernel", gemm_bytes(out, inp, T), g_best, peaks),
            "dense_cublas_us": 1e3 * d_mean, "dense_cublas_us_best": 1e3 * d_best,
            "note": "0.7 MB of traffic and 67 MFLOP: both kernels are launch-latency-bound, the rooflines are for the record"}


def ffn_768_case(tm: Timer, peaks, issue_cold, joint):
    """The transformer FFN layer (8192 tokens, 768 <-> 3072): the gradients of both linears pruned 2:4 along each
    consuming product's own reduction axis; both update products, both backward products (with and without the f'(z)
    factors), dense cuBLAS beside each."""
    import torch
    from paper_2203_10991_b200 import binding, workloads
    T, d, dff = 8192, 768, 3072
    TC = binding.MVUE_LAYOUT_TC
    seed = workloads.CONFIGS["ffn_768"]["seed"]
    res = {"T": T, "d_model": d, "d_ff": dff, "prune": "2:4", "timing": "per call, L2 flushed before each; mean / best of 20"}
    for name, n_out, n_in in (("up", dff, d), ("down", d, dff)):        # linear with weights [n_out x n_in]
        g = bf16_dev(workloads.gradient((T, n_out), "student_t", seed + (0 if name == "up" else 1), dtype="bf16"), "cuda")
        h = bf16_dev(workloads.normal_bf16((T, n_in), seed + 100), "cuda")
        W = bf16_dev(workloads.normal_bf16((n_out, n_in), seed + 200, std=0.02), "cuda")
        fz = bf16_dev(workloads.normal_bf16((T, n_in), seed + 300), "cuda")
        entry = {"g": [T, n_out]}
        # update: prune along tokens, dW[n_out x n_in] = theta(g)^T h
        v0, m0 = binding.mvue_prune(g, 2, 4, 0, 1, layout=TC, joint=joint)
        p_mean, p_best = tm.each(lambda: binding.mvue_prune(g, 2, 4, 0, 1, values=v0, meta=m0, layout=TC, joint=joint), 20)
        dW = torch.empty((n_out, n_in), dtype=torch.float32, device="cuda")
        ws = torch.empty(max(16, binding.mvue_gemm_workspace_bytes(0, n_out, n_in, T)), dtype=torch.uint8, device="cuda")
        u_mean, u_best = tm.each(lambda: binding.mvue_sparse_update_gemm(v0, m0, h, out=dW, workspace=ws), 20)
        gT = g.t()
        du_mean, du_best = tm.each(lambda: torch.matmul(gT, h), 20)
        flops = 2.0 * n_out * n_in * T
        entry["prune_axis0_us"] = 1e3 * p_mean
        entry["prune_axis0_roofline"] = hbm_roofline("prune_axis0_bf16_whole_tiles_kernel", prune_bytes(T, n_out, 2), p_mean, peaks)
        entry["update_us"] = 1e3 * u_mean
        entry["update_us_best"] = 1e3 * u_best
        entry["update_roofline"] = tensor_roofline("sparse_gemm_pair_kernel", flops, u_mean, peaks, issue_cold)
        entry["update_hbm_frac"] = gemm_bytes(n_out, n_in, T) / (u_mean * 1e-3) / 1e9 / peaks["hbm_gbs"]
        entry["update_dense_cublas_us"] = 1e3 * du_mean
        # backward: prune along the features, dh[T x n_in] = theta(g) W (* f'(z))
        v1, m1 = binding.mvue_prune(g, 2, 4, 1, 2, layout=TC, joint=joint)
        q_mean, _ = tm.each(lambda: binding.mvue_prune(g, 2, 4, 1, 2, values=v1, meta=m1, layout=TC, joint=joint), 20)
        dh = torch.empty((T, n_in), dtype=torch.bfloat16, device="cuda")
        wsb = torch.empty(max(16, binding.mvue_gemm_workspace_bytes(1, T, n_in, n_out)), dtype=torch.uint8, device="cuda")
        b_mean, b_best = tm.each(lambda: binding.mvue_sparse_backward_gemm(v1, m1, W, out=dh, workspace=wsb), 20)
        bf_mean, bf_best = tm.each(lambda: binding.mvue_sparse_backward_gemm(v1, m1, W, act_grad=fz, out=dh, workspace=wsb), 20)
        db_mean, _ = tm.each(lambda: torch.matmul(g, W), 20)
        dbf_mean, _ = tm.each(lambda: torch.matmul(g, W) * fz, 20)
        entry["prune_axis1_us"] = 1e3 * q_mean
        # K = n_out runs along the rows: whole blocks of 16 rows x 512 elements take the kernel without bounds checks
        axis1_kernel = "prune_axis1_bf16_pairs_kernel" if T % 16 == 0 and n_out % 512 == 0 else "prune_axis1_kernel"
        entry["prune_axis1_roofline"] = hbm_roofline(axis1_kernel, prune_bytes(T, n_out, 2), q_mean, peaks)
        entry["backward_us"] = 1e3 * b_mean
        entry["backward_us_best"] = 1e3 * b_best
        entry["backward_roofline"] = tensor_roofline("sparse_gemm_pair_kernel", flops, b_mean, peaks, issue_cold)
        entry["backward_hbm_frac"] = gemm_bytes(T, n_in, n_out, 2) / (b_mean * 1e-3) / 1e9 / peaks["hbm_gbs"]
        entry["backward_act_grad_us"] = 1e3 * bf_mean
        entry["backward_act_grad_us_best"] = 1e3 * bf_best
        entry["backward_act_grad_roofline"] = tensor_roofline("sparse_gemm_pair_kernel", flops, bf_mean, peaks, issue_cold)
        entry["backward_dense_cublas_us"] = 1e3 * db_mean
        entry["backward_act_grad_dense_torch_us"] = 1e3 * dbf_mean
        res[name] = entry
    res["note"] = ("38.7 GFLOP per product and 36 (up) / 9 (down) output tiles of 256 x 256 for 74 pairs of SMs: tile-starved; "
                   "update products are split along K. Intensity is near the ridge, so both roofline readings are given")
    return res


def tensor_bound_case(tm: Timer, n, m, peaks, joint, issue_cold, base_opt=0):
    """The large FFN layer (tokens 16384, 4096 -> 14336): the shape on which the sparse product is bound by
    the tensor cores, timed kernel by kernel next to dense cuBLAS.  Rides along in the JSON line."""
    import torch
    from paper_2203_10991_b200 import binding, workloads
    cfg = workloads.CONFIGS["ffn_large"]
    T, out, inp = cfg["T"], cfg["out"], cfg["inp"]
    TC = binding.MVUE_LAYOUT_TC
    g = bf16_dev(workloads.gradient((T, out), cfg["g_dist"], cfg["seed"], dtype="bf16"), "cuda")
    h = bf16_dev(workloads.normal_bf16((T, inp), cfg["seed"] + 100), "cuda")
    values, meta = binding.mvue_prune(g, n, m, 0, 0, layout=TC)
    dW = torch.empty((out, inp), dtype=torch.float32, device="cuda")
    ws = torch.empty(max(16, binding.mvue_gemm_workspace_bytes(0, out, inp, T)), dtype=torch.uint8, device="cuda")
    pb = prune_bytes(T, out, 2)

    def prune_with(nm, j, opt=base_opt):
        return lambda: binding.mvue_prune(g, nm[0], nm[1], 0, 1, values=values, meta=meta, layout=TC, joint=j, options=opt)

    prune_ms = tm.loop(prune_with((n, m), joint), 20)
    sys_ms = tm.loop(prune_with((2, 4), binding.MVUE_JOINT_SYSTEMATIC), 20)
    table_ms = tm.loop(prune_with((2, 4), binding.MVUE_JOINT_TABLE), 20)
    one_two_ms = tm.loop(prune_with((1, 2), joint), 20)
    sr_ms = tm.loop(prune_with((n, m), joint, base_opt | binding.MVUE_OPT_STOCHASTIC_ROUNDING), 20)
    sys32_ms = tm.loop(prune_with((2, 4), binding.MVUE_JOINT_SYSTEMATIC, binding.MVUE_OPT_NONE), 20)
    table32_ms = tm.loop(prune_with((2, 4), binding.MVUE_JOINT_TABLE, binding.MVUE_OPT_NONE), 20)
    four_eight_ms = tm.loop(lambda: binding.mvue_prune_4of8(g, 0, 1), 3, warm=1)     # approx-4:8, prune only
    prune_with((n, m), joint)()
    gemm_ms = tm.loop(lambda: binding.mvue_sparse_update_gemm(values, meta, h, out=dW, workspace=ws), 30)
    fused_ms = tm.loop(lambda: binding.mvue_fused_update_gemm(g, h, n, m, 1, out=dW), 3)
    gT = g.t()
    dense_ms = tm.loop(lambda: torch.matmul(gT, h), 30)
    issue_warm = issue_probe(binding, tm)             # the same probe right after the power-capped products
    flops = 2.0 * out * inp * T
    tf = flops / (gemm_ms * 1e-3) / 1e12
    return {"g": [T, out], "h": [T, inp], "prune": f"{n}:{m}",
            "timing": "back-to-back loop (inputs 470 MB / 134 MB per call, larger than L2)",
            "prune_ms": prune_ms, "roofline_prune": hbm_roofline("prune_axis0_bf16_whole_tiles_kernel", pb, prune_ms, peaks),
            "prune_systematic_ms": sys_ms, "prune_systematic_frac_of_hbm_peak": pb / (sys_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "prune_table_ms": table_ms, "prune_table_frac_of_hbm_peak": pb / (table_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "prune_1of2_ms": one_two_ms, "prune_1of2_frac_of_hbm_peak": pb / (one_two_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "random_bits_per_block": 16 if base_opt & binding.MVUE_OPT_EPS16 else 32,
            "prune_systematic_32bit_ms": sys32_ms,
            "prune_systematic_32bit_frac_of_hbm_peak": pb / (sys32_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "prune_table_32bit_ms": table32_ms,
            "prune_table_32bit_frac_of_hbm_peak": pb / (table32_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "prune_approx_4of8_ms": four_eight_ms,
            "prune_approx_4of8_frac_of_hbm_peak": pb / (four_eight_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "prune_stochastic_rounding_ms": sr_ms,
            "prune_stochastic_rounding_frac_of_hbm_peak": pb / (sr_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "gemm_ms": gemm_ms, "gemm_tflops_effective": tf,
            "sparse_issue_rate_cold_tflops": issue_cold, "sparse_issue_rate_after_products_tflops": issue_warm,
            "gemm_frac_of_issue_rate_after_products": tf / issue_warm,
            "dense_cublas_ms": dense_ms, "dense_cublas_tflops": flops / (dense_ms * 1e-3) / 1e12,
            # three-way comparison: separate prune + sparse product vs the fused kernel vs dense cuBLAS
            "separate_ms": prune_ms + gemm_ms, "fused_ms": fused_ms,
            "fused_tflops_effective": flops / (fused_ms * 1e-3) / 1e12,
            "roofline": tensor_roofline("sparse_gemm_pair_kernel", flops, gemm_ms, peaks, issue_cold)}


def gemm_shapes_case(tm: Timer, peaks, issue_cold):
    """Sparse products on their own over a list of shapes (M x N x K; update: fp32 out; backward: bf16 out with and without
    the f'(z) factors), dense matmul beside each: the tables of profiles/ that are not tied to a workload."""
    import torch
    from paper_2203_10991_b200 import binding, workloads
    TC = binding.MVUE_LAYOUT_TC
    shapes = [("update", 14336, 4096, 16384), ("update", 8192, 8192, 8192), ("update", 4096, 14336, 16384),
              ("update", 4096, 1024, 32768), ("update", 1024, 4096, 32768),
              ("backward", 32768, 4096, 1024), ("backward", 32768, 1024, 4096),
              ("backward", 8192, 768, 3072), ("backward", 8192, 3072, 768), ("backward", 16384, 4096, 14336)]
    rows = []
    for kind, M, N, K in shapes:
        if kind == "update":                                   # A = theta(g)^T [M x K], g [K x M]
            g = bf16_dev(workloads.gradient((K, M), "student_t", 7, dtype="bf16"), "cuda")
            v, mt = binding.mvue_prune(g, 2, 4, 0, 1, layout=TC, joint=binding.MVUE_JOINT_SYSTEMATIC)
            A_dense = g.t()
        else:                                                  # A = theta(g) [M x K], g [M x K]
            g = bf16_dev(workloads.gradient((M, K), "student_t", 7, dtype="bf16"), "cuda")
            v, mt = binding.mvue_prune(g, 2, 4, 1, 1, layout=TC, joint=binding.MVUE_JOINT_SYSTEMATIC)
            A_dense = g
        B = bf16_dev(workloads.normal_bf16((K, N), 8), "cuda")
        flops = 2.0 * M * N * K
        row = {"kind": kind, "M": M, "N": N, "K": K}
        if kind == "update":
            C = torch.empty((M, N), dtype=torch.float32, device="cuda")
            ws = torch.empty(max(16, binding.mvue_gemm_workspace_bytes(0, M, N, K)), dtype=torch.uint8, device="cuda")
            mean, best = tm.each(lambda: binding.mvue_sparse_update_gemm(v, mt, B, out=C, workspace=ws), 10)
            row.update(us=1e3 * mean, us_best=1e3 * best, roofline=tensor_roofline("sparse_gemm_pair_kernel", flops, mean, peaks, issue_cold),
                       hbm_frac=gemm_bytes(M, N, K) / (mean * 1e-3) / 1e9 / peaks["hbm_gbs"])
            dmean, _ = tm.each(lambda: torch.matmul(A_dense, B), 10)
            row["dense_us"] = 1e3 * dmean
        else:
            C = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
            fz = bf16_dev(workloads.normal_bf16((M, N), 9), "cuda")
            ws = torch.empty(max(16, binding.mvue_gemm_workspace_bytes(1, M, N, K)), dtype=torch.uint8, device="cuda")
            mean, best = tm.each(lambda: binding.mvue_sparse_backward_gemm(v, mt, B, out=C, workspace=ws), 10)
            fmean, fbest = tm.each(lambda: binding.mvue_sparse_backward_gemm(v, mt, B, act_grad=fz, out=C, workspace=ws), 10)
            row.update(us=1e3 * mean, us_best=1e3 * best, act_grad_us=1e3 * fmean, act_grad_us_best=1e3 * fbest,
                       roofline=tensor_roofline("sparse_gemm_pair_kernel", flops, mean, peaks, issue_cold),
                       act_grad_roofline=tensor_roofline("sparse_gemm_pair_kernel", flops, fmean, peaks, issue_cold),
                       hbm_frac=gemm_bytes(M, N, K, 2) / (mean * 1e-3) / 1e9 / peaks["hbm_gbs"],
                       act_grad_hbm_frac=gemm_bytes(M, N, K, 2, True) / (fmean * 1e-3) / 1e9 / peaks["hbm_gbs"])
            dmean, _ = tm.each(lambda: torch.matmul(A_dense, B), 10)
            dfmean, _ = tm.each(lambda: torch.matmul(A_dense, B) * fz, 10)
            row["dense_us"], row["dense_act_grad_us"] = 1e3 * dmean, 1e3 * dfmean
            if N % 128 == 0:
                # the same product pruning its own output along N in the epilogue, against the product followed by
                # the separate prune of its output
                emean, _ = tm.each(lambda: binding.mvue_sparse_backward_gemm_pruned(
                    v, mt, B, fz, 5, next_joint=binding.MVUE_JOINT_SYSTEMATIC, workspace=ws), 10)
                pv, pm = binding.mvue_prune(C, 2, 4, 1, 5, layout=TC, joint=binding.MVUE_JOINT_SYSTEMATIC)
                pmean, _ = tm.each(lambda: binding.mvue_prune(C, 2, 4, 1, 5, values=pv, meta=pm, layout=TC,
                                                              joint=binding.MVUE_JOINT_SYSTEMATIC), 10)
                row["act_grad_epilogue_prune_us"] = 1e3 * emean
                row["separate_prune_of_output_us"] = 1e3 * pmean
        rows.append(row)
        del g, v, mt, B, C
        torch.cuda.empty_cache()
    return {"timing": "per call, L2 flushed before each; mean / best of 10", "rows": rows}


def prune_sweep(peaks, sizes_log2=range(20, 33), step_joint=1, options=0):
    """Standalone prune+pack bandwidth over bf16 tensors of 2^k bytes ([bytes / 8192 x 4096], Student-t values), both
    pruned axes, 2:4 (pair table, systematic sampling), 1:2 and 1:4.  Every point is a CUDA graph of `reps` launches
    over rotating input copies that together exceed 2.5 x L2, replayed and timed with events, so the small sizes are
    neither launch-bound on the host nor L2-warm."""
    import torch
    from paper_2203_10991_b200 import binding, workloads
    dev = torch.device("cuda")
    TC = binding.MVUE_LAYOUT_TC
    cols = 4096
    sizes_log2 = list(sizes_log2)
    max_log2 = max(sizes_log2)
    # 256 MB of seeded values drawn on the host, tiled on the device up to the largest tensor
    seed_rows = 1 << 15
    base = workloads.gradient((seed_rows, cols), "student_t", 5, dtype="bf16")
    base_dev = bf16_dev(base, dev)
    total_rows = max(1 << (max_log2 - 13), int(2.6 * L2_BYTES) // (2 * cols) // 128 * 128)
    if total_rows > seed_rows:
        base_dev = base_dev.repeat((total_rows + seed_rows - 1) // seed_rows, 1)
    out_v = torch.empty(base_dev.numel() // 2, dtype=torch.bfloat16, device=dev)
    out_m = torch.empty(base_dev.numel() // 8 + (1 << 16), dtype=torch.uint8, device=dev)
    modes = [("2:4 table", 2, 4, binding.MVUE_JOINT_TABLE), ("2:4 systematic", 2, 4, binding.MVUE_JOINT_SYSTEMATIC),
             ("1:2", 1, 2, binding.MVUE_JOINT_TABLE), ("1:4", 1, 4, binding.MVUE_JOINT_TABLE)]
    if len(sizes_log2) <= 4:                                 # the short form keeps the step's law and the table
        modes = [md for md in modes if md[3] == step_joint and md[1:3] == (2, 4) or md[0] == "2:4 table"]
    points = []
    side = torch.cuda.Stream()
    for lg in sizes_log2:
        nbytes = 1 << lg
        rows = nbytes // (2 * cols)
        copies = max(1, min(int(2.5 * L2_BYTES / nbytes) + 1, (base_dev.numel() * 2) // nbytes))
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
                                           joint=joint, options=options)
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
            "random_bits_per_block": 16 if options & 2 else 32,
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
    g_top = bf16_dev(g_host, dev)

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

    def run_sys16_overlap():
        chain.backward_update(g_top, layers, n, m, base_seed=1, joint=binding.MVUE_JOINT_SYSTEMATIC, overlap=True,
                              options=binding.MVUE_OPT_EPS16)

    def run_sys_epilogue():
        # backward products with a long reduction axis (out = 4096) prune their own output for the layer below
        chain.backward_update(g_top, layers, n, m, base_seed=1, joint=binding.MVUE_JOINT_SYSTEMATIC, overlap=True,
                              prune_in_epilogue_min_k=4096)

    def run_sys16_epilogue():
        chain.backward_update(g_top, layers, n, m, base_seed=1, joint=binding.MVUE_JOINT_SYSTEMATIC, overlap=True,
                              prune_in_epilogue_min_k=4096, options=binding.MVUE_OPT_EPS16)

    eager_ms = timed(run_table, 5)
    table_ms = timed(graphed(run_table), 10)
    sys_ms = timed(graphed(run_sys), 10) if m == 4 else None
    overlap_ms = timed(graphed(run_sys_overlap), 10) if m == 4 else None
    epilogue_ms = timed(graphed(run_sys_epilogue), 10) if m == 4 else None
    sys16_ms = timed(graphed(run_sys16_overlap), 10) if m == 4 else None
    sys16_epilogue_ms = timed(graphed(run_sys16_epilogue), 10) if m == 4 else None
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
            # and with the long-K backward products pruning their own output in the epilogue (one prune launch less
            # per block of two layers)
            "systematic_two_stream_epilogue_prune_ms": epilogue_ms,
            # the two-stream chain with sixteen random bits per block (one generator call per eight blocks)
            "systematic_16bit_two_stream_ms": sys16_ms,
            "systematic_16bit_two_stream_tflops_effective": None if sys16_ms is None else flops / (sys16_ms * 1e-3) / 1e12,
            "systematic_16bit_two_stream_epilogue_prune_ms": sys16_epilogue_ms,
            "dense_torch_ms": dense_ms, "dense_torch_tflops": flops / (dense_ms * 1e-3) / 1e12}


def spawn_ranks(args) -> int:
    """`python bench.py --gpus N` outside torchrun: start N ranks of this script on this node (one per GPU, NCCL)."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")                    # the communicator's own log shows the rank count
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), str(Path(__file__).resolve())] + sys.argv[1:]
    return subprocess.run(cmd, env=env).returncode


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
    ap.add_argument("--eps32", dest="eps16", action="store_false",
                    help="32 random bits per block (one generator call per four blocks) in the step instead of 16 "
                         "(MVUE_OPT_EPS16: one call per eight blocks); the other width is timed beside it")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep", action="store_true",
                    help="the whole standalone prune+pack sweep over bf16 tensors of 1 MB .. 4 GB (default: three sizes)")
    ap.add_argument("--gemm-shapes", action="store_true",
                    help="add a table of sparse products on their own (update / backward, with and without f'(z)) next to dense")
    ap.add_argument("--no-extra", action="store_true",
                    help="skip the riders: other estimators, the other workloads, the sustained loop and the sweep points")
    args = ap.parse_args()
    from paper_2203_10991_b200 import workloads
    cfg = workloads.CONFIGS[args.workload]
    n, m = (int(x) for x in args.prune.split(":"))
    if args.impl == "reference":
        args.steps = 3 if args.steps is None else args.steps
        run_reference(args, cfg, n, m)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args))
    args.steps = 200 if args.steps is None else args.steps
    run_ours(args, cfg, n, m)


if __name__ == "__main__":
    main()
