#!/usr/bin/env python
"""Benchmark of the emulated-FP64 GEMM hot path (deconstruct -> residue GEMMs -> reconstruct).

One "step" is one oz_dgemm_ex call on the HPL trailing-update configuration
(C(16384x16384) -= A(16384x1024) B(1024x16384), synthetic U(-1,1) operands), i.e. one pass of the
whole hot path.  Prints ONE JSON line (rank 0):

  value      emulated FP64 TFLOP/s = 2 m n k / time, inputs resident in HBM
  e2e        same metric through oz_dgemm_host with pinned HOST buffers (copies timed)
  roofline   the residue-GEMM kernel: 3 r plane products, low-precision FLOP/s against the
             tensor peak (measured bf16 burst peak x 2 for 8-bit operands; the fractions of the
             sustained figure, of the nominal 4.5 PFLOP/s and of a library 8-bit GEMM timed in the
             same run stand beside it), timed with CUDA events recorded on the launching stream
             between the stages
  also       the same workload on the other routes (set E, INT8 digits, set A native INT8) and
             with the operands' planes prepared once (oz_dgemm_prepared), a few steps each
  cpu_baseline  the CPU oracle, as it stands, on a bounded sample of the same workload

`--impl reference` times the CPU oracle alone (there is no other implementation of the paper).
N > 1: every rank runs the same independent problem (weak scaling, no collective in the data
path); the time is the max over ranks, the value the sum of the work.  Under torchrun the ranks are
given; run plainly with --gpus N, the script starts its own N ranks (one process per GPU).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth_inputs as syn  # noqa: E402

# DRAM traffic of the residue GEMM relative to its algorithmic bytes (reads / plane bytes, writes /
# residue bytes) comes from the table in profiles/residue_gemm_dram_traffic.md: ncu captures of a
# smaller launch, one row per kernel variant, scaled here to the full-size launch by the units.
TRAFFIC_TABLE = os.path.join(os.path.dirname(os.path.abspath(__file__)), "profiles", "residue_gemm_dram_traffic.md")


def gemm_dram_amplification(set_name: str, substrate: str):
    """(read, write) amplification of the variant, or None when the table has no row for it."""
    try:
        with open(TRAFFIC_TABLE) as fh:
            rows = [[c.strip() for c in line.strip().strip("|").split("|")] for line in fh if line.startswith("|")]
    except OSError:
        return None
    for row in rows:
        if len(row) >= 4 and row[0] == set_name and row[1] == substrate:
            try:
                return float(row[2]), float(row[3])
            except ValueError:
                return None
    return None


METRIC = "emulated FP64 TFLOPS (2mnk/s)"
UNIT = "TFLOP/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        return {"hbm_gbs": d["hbm_gbs"], "bf16": d["bf16_tflops"],
                "bf16_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        # by UUID, so that a restricted device list (CUDA_VISIBLE_DEVICES) cannot point the sampler at
        # another GPU; the plain index is the fall-back
        self.gpu = str(gpu_index)
        try:
            import torch
            uuid = str(torch.cuda.get_device_properties(gpu_index).uuid)
            self.gpu = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
        except Exception:
            pass
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-i", self.gpu, "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            f = [t.strip() for t in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax.append(float(f[2]))
            except ValueError:
                continue
            try:
                pw.append(float(f[3]))
            except ValueError:
                pw.append(0.0)
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        # samples taken under load: power draw above half of the largest seen
        top = max(pw) if pw else 0.0
        busy = [v for v, w in zip(sm, pw) if w >= 0.5 * top] or sm
        return {"sm_mhz": statistics.median(busy), "sm_max_mhz": max(smax), "reasons": sorted(reasons),
                "samples": len(sm), "samples_under_load": len(busy), "power_w_max": top}


def aggregate_over_ranks(local_ms: float, local_work: float, world: int, reduce_max, reduce_sum):
    """Whole-job numbers from per-rank ones: time = max over ranks, work = sum over ranks."""
    ms = reduce_max(local_ms) if world > 1 else local_ms
    work = reduce_sum(local_work) if world > 1 else local_work
    return ms, work


def oracle_sample_tflops(cfg, set_name: str, sample=(4096, 6144, 1024)):
    """Times the CPU oracle (whole method) on a bounded sample of the workload."""
    from oracle import oz_oracle as ozo
    m, n, k = min(sample[0], cfg.m), min(sample[1], cfg.n), min(sample[2], cfg.k)
    A, B, C0 = syn.operands(cfg, m, n, k, want_c=True)
    oset = {"S": ozo.SET_S, "E": ozo.SET_E, "A": ozo.SET_A}[set_name]
    ozo.dgemm(np.asfortranarray(A[:32]), np.asfortranarray(B[:, :32]), oset)  # load the library, warm the threads
    t0 = time.perf_counter()
    ozo.dgemm(A, B, oset, ozo.QUANT_RN, ozo.SCALE_CS, cfg.alpha, cfg.beta, C0 if cfg.beta else None)
    dt = time.perf_counter() - t0
    return 2.0 * m * n * k / dt / 1e12, ozo.num_threads(), f"{m}x{n}x{k} block of the workload, {dt:.1f} s"


def run_reference(args, cfg, set_name):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals = []
    sample = (1024, 1536, 1024)
    for i in range(args.warmup + args.steps):
        v, cores, desc = oracle_sample_tflops(cfg, set_name, sample)
        if i >= args.warmup:
            vals.append(v)
    value = len(vals) / sum(1.0 / v for v in vals)
    ms = 2.0 * sample[0] * sample[1] * sample[2] / (value * 1e12) * 1e3
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int64", "data": "synthetic",
            "config": {"workload": cfg.name, "modulus_set": set_name, "m": cfg.m, "n": cfg.n, "k": cfg.k,
                       "note": "CPU oracle; each step is a bounded sample of the workload"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def spawn_command(argv, gpus: int, port: int):
    """Command line that runs this script as `gpus` ranks on this node (one process per GPU)."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def free_port() -> int:
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        return sock.getsockname()[1]


def library_8bit_tflops(torch, seconds: float = 0.25):
    """A library 8-bit GEMM (8192^3) timed in this run: the practical ceiling of the tensor pipe on this
    GPU in its present power state.  Returns {"fp8": TFLOP/s or None, "int8": TOP/s or None}."""
    n = 8192
    out = {"fp8": None, "int8": None}

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps, total = 0, 0.0
        while total < seconds * 1e3 and reps < 200:
            e0.record()
            for _ in range(5):
                fn()
            e1.record()
            torch.cuda.synchronize()
            total += e0.elapsed_time(e1)
            reps += 5
        return 2.0 * n ** 3 * reps / (total * 1e-3) / 1e12

    try:
        a = torch.randint(-8, 8, (n, n), device="cuda", dtype=torch.int8)
        b = torch.randint(-8, 8, (n, n), device="cuda", dtype=torch.int8)
        out["int8"] = timed(lambda: torch._int_mm(a, b))
    except Exception:
        pass
    try:
        a8 = torch.randn(n, n, device="cuda").to(torch.float8_e4m3fn)
        b8 = torch.randn(n, n, device="cuda").to(torch.float8_e4m3fn).t()
        one = torch.ones((), device="cuda")
        out["fp8"] = timed(lambda: torch._scaled_mm(a8, b8, scale_a=one, scale_b=one, out_dtype=torch.bfloat16))
    except Exception:
        pass
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=3, help="synthetic configuration 1..5 (3 = HPL update)")
    ap.add_argument("--set", dest="set_name", default="S", choices=["S", "E", "A"])
    ap.add_argument("--substrate", default="fp8", choices=["fp8", "int8", "int8n"],
                    help="int8n = native INT8 residues, one plane per modulus (set A only)")
    ap.add_argument("--shape", default=None, help="m,n,k override (same distribution and seed as --config)")
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-also", action="store_true", help="skip the other routes and the library 8-bit GEMM")
    ap.add_argument("--fused", action="store_true",
                    help="storage mode F: A converted inside the product kernel (OZ_STORAGE_FUSED; n <= 128)")
    ap.add_argument("--fallback", action="store_true",
                    help="re-issue the rows that fail the exponent-span check on the native FP64 path (OZ_FALLBACK_FP64)")
    args = ap.parse_args()
    if args.impl != "reference" and args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # run plainly with --gpus N: start the N replica ranks ourselves
        raise SystemExit(subprocess.call(spawn_command(sys.argv[1:], args.gpus, free_port())))
    if args.warmup < 3 and args.impl != "reference":
        args.warmup = 3
    cfg = syn.CONFIGS[args.config]
    if args.shape:
        sm_, sn_, sk_ = [int(v) for v in args.shape.split(",")]
        cfg = syn.Config(**{**cfg.__dict__, "m": sm_, "n": sn_, "k": sk_, "name": cfg.name + "_shape_" + args.shape.replace(",", "x")})
    if args.impl == "reference":
        run_reference(args, cfg, args.set_name)
        return

    import torch
    import torch.distributed as dist
    import paper_2609_09095_b200 as oz

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    m, n, k = cfg.m, cfg.n, cfg.k
    modset = {"S": oz.OZ_SET_S, "E": oz.OZ_SET_E, "A": oz.OZ_SET_A}[args.set_name]
    sub = {"fp8": oz.OZ_SUB_FP8, "int8": oz.OZ_SUB_INT8, "int8n": oz.OZ_SUB_INT8_NATIVE}[args.substrate]
    host_route = sub | oz.OZ_QUANT_RN | oz.OZ_SCALE_CS      # the host-buffer entry point has no native path
    route = host_route | (oz.OZ_FALLBACK_FP64 if args.fallback else 0) | (oz.OZ_STORAGE_FUSED if args.fused else 0)
    r, _, _ = oz.oz_set_info(modset)
    p_store = oz.oz_plane_count(modset, route)
    p_store_a = oz.oz_plane_count_side(modset, route, 0)    # same count on both operands
    if p_store == 0:
        raise SystemExit("the native INT8 substrate needs the all-byte set: --set A --substrate int8n")
    passes = r if args.substrate == "int8n" else 3 * r    # plane products per FP64 product

    # every rank owns an independent instance of the problem (weak scaling); seeds differ per rank
    cfg_rank = syn.Config(**{**cfg.__dict__, "seed": cfg.seed + rank})
    A, B, C0 = syn.operands(cfg_rank, want_c=True)
    hA = torch.from_numpy(np.ascontiguousarray(A.T)).pin_memory()
    hB = torch.from_numpy(np.ascontiguousarray(B.T)).pin_memory()
    hC = torch.from_numpy(np.ascontiguousarray(C0.T)).pin_memory()
    del A, B, C0
    dA, dB, dC = hA.cuda(), hB.cuda(), hC.cuda()
    # the other routes timed for the `also` key (single GPU, default workload only)
    also_routes = []
    if world == 1 and not args.no_also and args.shape is None:
        for sname, subname in (("E", "fp8"), ("S", "int8"), ("S", "fp8"), ("A", "int8n")):
            if (sname, subname) != (args.set_name, args.substrate):
                also_routes.append((sname, subname))
    sets = {"S": oz.OZ_SET_S, "E": oz.OZ_SET_E, "A": oz.OZ_SET_A}
    subs = {"fp8": oz.OZ_SUB_FP8, "int8": oz.OZ_SUB_INT8, "int8n": oz.OZ_SUB_INT8_NATIVE}
    core = max([oz.oz_workspace_bytes(m, n, k, modset, route), oz.oz_workspace_bytes(m, n, k, modset, host_route)] +
               [oz.oz_workspace_bytes(m, n, k, sets[a], subs[b] | oz.OZ_QUANT_RN | oz.OZ_SCALE_CS) for a, b in also_routes])
    ws_bytes = core + 8 * (m * k + k * n + m * n) + 4096
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    oz.check(oz.oz_set_workspace(ws, ws_bytes), "oz_set_workspace")
    stream = torch.cuda.current_stream()

    def step():
        oz.check(oz.oz_dgemm_ex(m, n, k, cfg.alpha, dA, m, dB, k, cfg.beta, dC, m, modset, route, stream),
                 "oz_dgemm_ex")

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    esc_flag = [False]

    def check_status(where):
        """Device status; the result of the exponent-span check (OZ_ERR_RANGE) is informational and only recorded."""
        st = oz.oz_query_status(stream)
        if st == oz.OZ_ERR_RANGE:
            esc_flag[0] = True
        else:
            oz.check(st, where)

    sampler = ClockSampler(local_rank)
    sampler.start()          # nvidia-smi needs a moment to start: launch it before the warm-up
    for _ in range(args.warmup):
        step()
    check_status("device status after warm-up")

    # ---- timed region: K steps, per-stage events recorded by the library on the launching stream
    stage_events = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(args.steps)]
    for evs in stage_events:
        for e in evs:
            e.record(stream)  # materialise the handles
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.lines.clear()    # keep only samples taken from here on
    launches0 = oz.oz_launch_count()
    ev0.record(stream)
    for i in range(args.steps):
        oz.oz_set_stage_events(stage_events[i])
        step()
    ev1.record(stream)
    barrier()
    launches = oz.oz_launch_count() - launches0
    clocks = sampler.stop()
    oz.oz_set_stage_events(None)
    check_status("device status after the timed steps")
    fallback_rows = oz.oz_query_fallback_rows(stream) // max(args.steps + args.warmup, 1)
    local_ms = ev0.elapsed_time(ev1) / args.steps
    per_step = np.array([[evs[i].elapsed_time(evs[i + 1]) for i in range(4)] for evs in stage_events])
    stage_ms = per_step.mean(axis=0)
    step_totals = per_step.sum(axis=1)          # first to last stage event of every timed call

    # ---- end to end through the host-buffer entry point (copies inside the timed region)
    def e2e_step():
        oz.check(oz.oz_dgemm_host(m, n, k, cfg.alpha, hA, m, hB, k, cfg.beta, hC, m, modset, host_route, stream),
                 "oz_dgemm_host")

    e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.e2e_steps):
        e2e_step()
    e1.record(stream)
    barrier()
    e2e_local_ms = e0.elapsed_time(e1) / args.e2e_steps
    check_status("device status after the end-to-end steps")

    flops = 2.0 * m * n * k

    # ---- the same workload on the other routes, and with the planes of A and B prepared once
    def timed_steps(fn, steps=5, warm=2):
        for _ in range(warm):
            fn()
        torch.cuda.synchronize()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record(stream)
        for _ in range(steps):
            fn()
        t1.record(stream)
        torch.cuda.synchronize()
        return t0.elapsed_time(t1) / steps

    also = []
    for sname, subname in also_routes:
        rt2 = subs[subname] | oz.OZ_QUANT_RN | oz.OZ_SCALE_CS
        r2, _, _ = oz.oz_set_info(sets[sname])
        passes2 = r2 if subname == "int8n" else 3 * r2
        ms2 = timed_steps(lambda: oz.check(oz.oz_dgemm_ex(m, n, k, cfg.alpha, dA, m, dB, k, cfg.beta, dC, m,
                                                          sets[sname], rt2, stream), "oz_dgemm_ex"))
        check_status("device status (also)")
        also.append({"modulus_set": sname, "substrate": subname, "value": flops / (ms2 * 1e-3) / 1e12, "unit": UNIT,
                     "ms_per_step": ms2, "steps": 5,
                     "roof_frac_of_nominal": flops / (ms2 * 1e-3) / 1e12 / (4500.0 / (passes2 + 1))})
    if world == 1 and not args.no_also:
        # planes kept across calls (HPL: the panel's planes serve the whole trailing matrix): operands
        # prepared once, then products only
        opA = torch.empty(oz.oz_operand_bytes(0, m, k, modset, route), dtype=torch.uint8, device="cuda")
        opB = torch.empty(oz.oz_operand_bytes(1, n, k, modset, route), dtype=torch.uint8, device="cuda")
        oz.check(oz.oz_prepare_operand(0, m, k, dA, m, modset, route, opA, None, stream), "oz_prepare_operand")
        oz.check(oz.oz_prepare_operand(1, n, k, dB, k, modset, route, opB, None, stream), "oz_prepare_operand")
        ms3 = timed_steps(lambda: oz.check(oz.oz_dgemm_prepared(m, n, k, cfg.alpha, opA, opB, cfg.beta, dC, m, modset,
                                                                route, stream), "oz_dgemm_prepared"))
        check_status("device status (prepared)")
        also.append({"modulus_set": args.set_name, "substrate": args.substrate, "planes": "prepared once (oz_dgemm_prepared)",
                     "value": flops / (ms3 * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": ms3, "steps": 5})
        del opA, opB
        if k <= 16384:
            # accurate mode: the shifts from one extra tensor-core product of magnitude digits (3r + 1 passes)
            rt4 = route & ~oz.OZ_SCALE_CS | oz.OZ_SCALE_ACCURATE
            ms4 = timed_steps(lambda: oz.check(oz.oz_dgemm_ex(m, n, k, cfg.alpha, dA, m, dB, k, cfg.beta, dC, m, modset,
                                                              rt4, stream), "oz_dgemm_ex"))
            check_status("device status (accurate mode)")
            also.append({"modulus_set": args.set_name, "substrate": args.substrate, "scale_rule": "ACCURATE",
                         "value": flops / (ms4 * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": ms4, "steps": 5})
    lib8 = library_8bit_tflops(torch) if (world == 1 and not args.no_also) else {"fp8": None, "int8": None}

    if world > 1:
        def rmax(v):
            t = torch.tensor([v], dtype=torch.float64, device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            return float(t.item())

        def rsum(v):
            t = torch.tensor([v], dtype=torch.float64, device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.SUM)
            return float(t.item())
    else:
        rmax = rsum = None
    ms, work = aggregate_over_ranks(local_ms, flops, world, rmax, rsum)
    e2e_ms, _ = aggregate_over_ranks(e2e_local_ms, flops, world, rmax, rsum)

    if rank == 0:
        peaks = measured_peaks()
        value = work / (ms * 1e-3) / 1e12
        lowp_flops = float(passes) * flops                 # p_mma plane products (3r, or r on the native INT8 route)
        gemm_ms = float(stage_ms[2])
        # 8-bit operands: nominal 2x the bf16 rate.  The kernel is timed by its own events, a few
        # milliseconds per launch: the burst figure is its denominator; the other ceilings stand beside it.
        tensor_peak = 2.0 * peaks["bf16"]
        achieved = lowp_flops / (gemm_ms * 1e-3) / 1e12
        roof_nominal = 4500.0 / (passes + 1)               # P_low/(3r+1), or P_low/(r+1) native INT8, at B200's dense 8-bit rate
        hbm = peaks["hbm_gbs"]
        dec_bytes = 24 * (m * k + k * n) + (p_store_a * m + p_store * n) * k   # two scan passes + convert read; planes written
        rb = oz.oz_residue_elem_bytes(modset)                 # bytes per stored residue
        rec_bytes = (rb * r + 8 + (8 if cfg.beta else 0)) * m * n
        plane_bytes = float((p_store_a * m + p_store * n) * k)
        residue_bytes = float(rb) * r * m * n
        amp = gemm_dram_amplification(args.set_name, args.substrate)
        lib_peak = lib8["fp8" if args.substrate == "fp8" else "int8"]
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "fp8_e4m3" if args.substrate == "fp8" else "int8",
            "data": "synthetic",
            "config": {"workload": cfg.name, "m": m, "n": n, "k": k, "alpha": cfg.alpha, "beta": cfg.beta,
                       "modulus_set": args.set_name, "r": r, "substrate": args.substrate, "quantiser": "RN",
                       "scale_rule": "CS", "storage_mode": "F (A converted inside the product kernel)" if args.fused else "M (materialised planes)",
                       "l2": "inputs larger than L2 (126 MB): A+B %.0f MB, C %.0f MB, planes %.0f MB, residues %.0f MB"
                             % (8e-6 * (m * k + k * n), 8e-6 * m * n, 1e-6 * p_store * (m + n) * k, 1e-6 * rb * r * m * n),
                       "parallelism": f"replicas x{world}" if world > 1 else "single GPU"},
            "roof": {"definition": "P_low/(3r+1)" if passes == 3 * r else "P_low/(r+1)", "nominal_tflops": roof_nominal,
                     "frac_of_nominal": value / world / roof_nominal,
                     "at_measured_peak_tflops": tensor_peak / (passes + 1),
                     "frac_at_measured_peak": value / world / (tensor_peak / (passes + 1)),
                     "ms_per_step_x_sm_mhz": ms * clocks["sm_mhz"] if clocks.get("sm_mhz") else None},
            "roofline": {"kernel": "residue_gemm_kernel (tcgen05)", "bound": "tensor", "achieved": achieved,
                         "peak": tensor_peak, "unit": "TFLOP/s", "frac": achieved / tensor_peak,
                         "peak_source": f"{peaks['source']} bf16 burst x2 (8-bit operands); frac is against this",
                         "frac_of_nominal_4500": achieved / 4500.0,
                         "frac_of_sustained_x2": achieved / (2.0 * peaks["bf16_sustained"]),
                         "peak_library_8bit": lib_peak,
                         "peak_library_8bit_source": "torch 8192^3 8-bit GEMM (torch._scaled_mm e4m3 / torch._int_mm) timed in this run",
                         "frac_of_library_8bit": achieved / lib_peak if lib_peak else None,
                         "traffic": amp[0] * plane_bytes + amp[1] * residue_bytes if amp else None,
                         "traffic_unit": "bytes per launch (ncu dram read+write of a smaller launch of this variant, "
                                         "scaled by units; profiles/residue_gemm_dram_traffic.md)",
                         "algorithmic_dram_bytes": plane_bytes + residue_bytes,
                         "ms_per_launch": gemm_ms},
            "stages": {
                "deconstruct_A_ms": float(stage_ms[0]), "deconstruct_join_ms": float(stage_ms[1]),
                "residue_gemm_ms": gemm_ms, "reconstruct_ms": float(stage_ms[3]),
                "deconstruct_GBps": dec_bytes / ((stage_ms[0] + stage_ms[1]) * 1e-3) / 1e9,
                "reconstruct_GBps": rec_bytes / (stage_ms[3] * 1e-3) / 1e9,
                "reconstruct_bytes": rec_bytes,
                "call_ms_median": float(np.median(step_totals)), "call_ms_best": float(step_totals.min()),
                "hbm_peak_GBps": hbm, "hbm_peak_source": peaks["source"]},
            "also": also,
            "e2e": {"value": work / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": 8 * (m * k + k * n + (m * n if cfg.beta else 0)),
                    "d2h_bytes_per_step": 8 * m * n, "steps": args.e2e_steps},
            "gpu_launches": int(launches), "clocks": clocks,
            "exponent_span_check": "flagged (OZ_ERR_RANGE): the set is too small for FP64-grade accuracy on this data"
                                   if esc_flag[0] else "passed",
            "native_fp64_rows_per_step": int(fallback_rows) if args.fallback else None,
            "native_fp64_ms": float(local_ms - step_totals.mean()) if args.fallback else None,   # after the last stage event
        }
        if not args.no_cpu_baseline:
            v, cores, desc = oracle_sample_tflops(cfg, args.set_name)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc}
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
