"""Host-side logic of bench.py: whole-job aggregation over ranks (time = max, work = sum) on a
world-size-2 gloo group, the clock-sample parser, and the reference arm's JSON line."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)

    def rmax(v):
        t = torch.tensor([v], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def rsum(v):
        t = torch.tensor([v], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        return float(t.item())

    ms, work = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 100.0 * (rank + 1), world, rmax, rsum)
    dist.barrier()
    if rank == 0:
        with open(out, "w") as fh:
            json.dump({"ms": ms, "work": work}, fh)
    dist.destroy_process_group()


def test_two_rank_aggregation_gloo(tmp_path):
    out = str(tmp_path / "agg.json")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    got = json.load(open(out))
    assert got == {"ms": 15.0, "work": 300.0}          # slowest rank, total work
    assert bench.aggregate_over_ranks(7.0, 3.0, 1, None, None) == (7.0, 3.0)


def test_self_spawned_ranks_gloo():
    """`bench.py --gpus N` run without torchrun starts its own N ranks: the command line it builds
    (one process per GPU on 127.0.0.1, the original arguments passed on) brings up a working group."""
    cmd = bench.spawn_command(["--gpus", "2", "--steps", "3"], 2, _free_port())
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"] and "--nproc-per-node=2" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-5] == os.path.join(ROOT, "bench.py") and cmd[-4:] == ["--gpus", "2", "--steps", "3"]
    cmd[-5] = os.path.join(ROOT, "tests", "rank_probe.py")          # same launch line, CPU ranks
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr
    got = json.loads([l for l in out.stdout.splitlines() if l.startswith("{")][-1])
    assert got == {"ms": 11.0, "work": 14.0, "world": 2, "argv": ["--gpus", "2", "--steps", "3"]}


def test_traffic_table_lookup():
    amp = bench.gemm_dram_amplification("S", "fp8")
    assert amp is None or (len(amp) == 2 and amp[0] >= 1.0 and amp[1] >= 0.9)
    assert bench.gemm_dram_amplification("no such set", "fp8") is None


def test_clock_sample_parser():
    s = bench.ClockSampler(0)
    s.proc = type("P", (), {"terminate": lambda self: None, "wait": lambda self, timeout=None: 0})()
    s.lines = ["0, 1755, 1965, 950.1, 0x4, Not Active, Not Active, Not Active, Active",
               "0, 1740, 1965, 960.0, 0x4, Not Active, Not Active, Not Active, Active",
               "0, 120, 1965, 80.0, 0x1, Not Active, Not Active, Not Active, Not Active"]
    got = s.stop()
    assert got["sm_mhz"] == 1747.5 and got["sm_max_mhz"] == 1965.0 and got["reasons"] == ["sw_power_cap"]


def test_reference_arm_prints_one_json_line():
    env = dict(os.environ, OMP_NUM_THREADS="4")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--shape", "128,192,256"], capture_output=True, text=True, env=env,
                         timeout=600)
    assert out.returncode == 0, out.stderr
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["cpu_baseline"]["kind"] == "oracle" and d["value"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["gpu_launches"] == 0
