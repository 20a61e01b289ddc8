"""The N > 1 bookkeeping of bench.py on two gloo ranks (CPU): slowest rank decides, bytes add up."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    from paper_2505_06901_b200 import distutil

    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert distutil.rank_info() == (rank, world, rank)
        times = [1.0 + rank, 5.0 - rank, 2.0]
        mx = distutil.max_over_ranks(times, dist)
        rate = distutil.aggregate_throughput(1e9, 0.5 * (rank + 1), world, dist)
        out.put((rank, mx, rate))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_max_over_ranks_and_weak_scaling_rate_with_two_gloo_ranks():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, mx, rate in results:
        assert mx == [2.0, 5.0, 2.0]
        assert rate == pytest.approx(2 * 1e9 / 1.0)      # 2 ranks x 1 GB over the slower rank's 1.0 s


def test_single_process_is_identity():
    from paper_2505_06901_b200 import distutil

    assert distutil.max_over_ranks([3.0, 1.0]) == [3.0, 1.0]
    assert distutil.aggregate_throughput(10.0, 2.0, 1) == 5.0


def test_gpus_flag_relaunches_under_torchrun_only_when_needed():
    """`bench.py --gpus N` started directly must start N ranks itself; under torchrun it must not, and a world size
    that contradicts the flag is an error."""
    import importlib.util
    import sys

    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(root, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    argv = ["--gpus", "4", "--steps", "7", "--warmup", "3"]
    cmd = bench.relaunch_command(bench.parse_args(argv), argv, {})
    assert cmd[:3] == [sys.executable, "-m", "torch.distributed.run"]
    assert "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd and cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-len(argv) - 1].endswith("bench.py") and cmd[-len(argv):] == argv
    assert 1024 < int(cmd[cmd.index("--master-port") + 1]) < 65536
    assert bench.relaunch_command(bench.parse_args(argv), argv, {"WORLD_SIZE": "4", "RANK": "1"}) is None
    assert bench.relaunch_command(bench.parse_args([]), [], {}) is None
    assert bench.relaunch_command(bench.parse_args(["--gpus", "1"]), ["--gpus", "1"], {}) is None
    with pytest.raises(SystemExit):
        bench.relaunch_command(bench.parse_args(argv), argv, {"WORLD_SIZE": "2"})


def test_reference_arm_prints_one_contract_line():
    """`bench.py --impl reference` (the oracle, CPU only) prints exactly one JSON line with the contract's keys."""
    import json
    import subprocess
    import sys

    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                         capture_output=True, text=True, timeout=600, cwd=root)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.strip().startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in d, key
    assert d["impl"] == "reference" and d["value"] > 0 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0
    assert "workload" in d["config"]


@pytest.mark.gpu
def test_bench_line_on_gpu_has_roofline_and_baselines():
    """The product arm on the reduced workload: one JSON line with roofline, e2e, clocks, launch count and the
    oracle's cpu_baseline; its kernels really ran (gpu_launches > 0)."""
    import json
    import subprocess
    import sys

    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--small", "--steps", "3", "--warmup", "3"],
                         capture_output=True, text=True, timeout=900, cwd=root)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.strip().startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["n_gpus"] == 1 and d["steps"] == 3 and d["warmup"] >= 3 and d["value"] > 0 and d["gpu_launches"] > 0
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and 0 < r["frac"] < 1.2 and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert r["traffic"] is None or r["traffic"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] > 0 and d["e2e"]["d2h_bytes_per_step"] > 0 and d["e2e"]["value"] > 0
    assert d["e2e"]["value"] < d["value"]                      # the copies are inside its timed region
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1 and d["cpu_baseline"]["value"] > 0
    assert "sm_mhz" in d["clocks"] and "reasons" in d["clocks"]
    assert d["vs_baseline"] is None and d["scaling"] == "weak" and "workload" in d["config"]
