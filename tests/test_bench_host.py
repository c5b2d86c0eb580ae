"""Host logic of bench.py that needs no GPU: the algorithmic byte counts behind the rooflines, the roofline records,
the rule that ties an ncu traffic figure to the sources it was captured from, and the rank launcher's command."""
import importlib.util
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parents[1]


@pytest.fixture(scope="module")
def bench():
    spec = importlib.util.spec_from_file_location("bench_under_test", ROOT / "bench.py")
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_algorithmic_bytes(bench):
    # prune+pack moves 2 + 1 + 1/8 bytes per bf16 element, 4 + 1 + 1/8 per binary32 element
    assert bench.prune_bytes(200704, 256, 2) == int(200704 * 256 * 3.125) == 160563200
    assert bench.prune_bytes(512, 256, 4) == int(512 * 256 * 5.125)
    # product: survivors (M K/2 bf16) + metadata (M K/8 bytes) + B (K N bf16) + C (M N fp32), once each
    M, N, K = 256, 2304, 200704
    assert bench.gemm_bytes(M, N, K) == M * K + M * K // 8 + 2 * K * N + 4 * M * N == 985006080
    assert bench.gemm_bytes(M, N, K, c_bytes=2, scale=True) == M * K + M * K // 8 + 2 * K * N + 2 * M * N + 2 * M * N


def test_roofline_records(bench):
    peaks = {"hbm_gbs": 6548.2, "bf16_tflops": 1670.2, "bf16_tflops_sustained": 1410.7, "source": "measured"}
    r = bench.hbm_roofline("k", 160563200, 0.0316, peaks, traffic=124000000)
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["traffic"] == 124000000
    assert r["achieved"] == pytest.approx(160563200 / 31.6e-6 / 1e9) and r["frac"] == pytest.approx(r["achieved"] / 6548.2)
    t = bench.tensor_roofline("k", 2.0 * 14336 * 4096 * 16384, 0.82, peaks, 4400.0)
    assert t["bound"] == "tensor" and t["peak"] == 4400.0 and t["frac"] == pytest.approx(t["achieved"] / 4400.0)
    assert t["frac_of_2x_dense_cublas_burst"] == pytest.approx(t["achieved"] / (2 * 1670.2))
    assert bench.tensor_roofline("k", 1e12, 1.0, peaks, None)["peak"] == bench.NOMINAL_SPARSE_BF16_TFLOPS


def test_traffic_figures_follow_their_sources(bench, monkeypatch):
    name = "sparse_gemm_pair_kernel"
    nbytes, sources, digest = bench.NCU_TRAFFIC[name]
    assert bench.ncu_traffic(name, "ffn_large") is None            # captured on conv_im2col only
    assert bench.ncu_traffic("no_such_kernel", "conv_im2col") is None
    monkeypatch.setitem(bench.NCU_TRAFFIC, name, (nbytes, sources, bench.source_digest(sources)))
    assert bench.ncu_traffic(name, "conv_im2col") == nbytes
    monkeypatch.setitem(bench.NCU_TRAFFIC, name, (nbytes, sources, "0" * 16))   # the sources have changed since
    assert bench.ncu_traffic(name, "conv_im2col") is None


def test_rank_launcher_command(bench, monkeypatch):
    seen = {}

    class Done:
        returncode = 0

    def fake_run(cmd, env=None):
        seen["cmd"], seen["env"] = cmd, env
        return Done()

    monkeypatch.setattr(bench.subprocess, "run", fake_run)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "4", "--steps", "7"])

    class Args:
        gpus = 4

    assert bench.spawn_ranks(Args()) == 0
    cmd = seen["cmd"]
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-4:] == ["--gpus", "4", "--steps", "7"] and cmd[-5].endswith("bench.py")
