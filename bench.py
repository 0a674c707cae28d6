#!/usr/bin/env python
"""Benchmark of the int8 GEMM hot path (TMA staging -> tcgen05 kind::i8 -> fused requant epilogue).

One "step" runs the three large GEMMs of the headline workload (4096^3, 8192^3, 16384x4096x8192; per-output-
channel requantisation, ReLU off) once each through the C-ABI library, on synthetic seeded inputs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-details]

prints ONE JSON line.  `value` is int8 TOPS (2*MACs / time) summed over all ranks with operands resident in
HBM; `e2e` is the same metric through the host-buffer entry point with the copies inside the timed region;
`roofline` is the tensor kernel's achieved rate against the measured peak; `cpu_baseline` is one full evaluation of the
CPU oracle on the same workload (every output is also compared with it); `details` lists every other configuration
(256^3, the convolutions, the tall-skinny and batched products) timed one by one after the headline measurement, each
with the oracle's wall time beside it.  `--impl reference` times the
oracle alone (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "int8 TOPS (bit-exact vs oracle) and % of B200 INT8 tensor/HBM roofline"
UNIT = "TOPS"
WORKLOAD = "config1: int8 GEMM (4096,4096,4096)+(8192,8192,8192)+(16384,4096,8192), per-channel requant, ReLU off"
NOMINAL_INT8_OVER_BF16 = 2.0          # dense 4.5 POPS int8 vs 2.25 PFLOP/s bf16
FALLBACK_BF16_TFLOPS = 1590.0
FALLBACK_HBM_GBS = 6650.0
NCU_STEP_TRAFFIC_BYTES = 690600000   # dram__bytes_read.sum + dram__bytes_write.sum over the step's three launches


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_burst": d["bf16_tflops"],
                "bf16_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_burst": FALLBACK_BF16_TFLOPS, "bf16_sustained": 1400.0,
            "source": "fallback"}


def gemm_ops(p):
    return 2.0 * p.M * p.N * p.K


def gemm_bytes(p):
    nq = p.N if p.per_channel else 1
    return p.M * p.K + p.N * p.K + p.M * p.N + 4 * p.N * (1 if p.bias is not None else 0) + 8 * nq


# ------------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    """nvidia-smi sampled in the background; samples are attributed to the timed region by their timestamps."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        """Start sampling and wait (up to 5 s) for the first sample so the timed region is covered."""
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "20", "-i", str(self.gpu)], stdout=open(self.path, "w"),
                                         stderr=subprocess.DEVNULL)
            t0 = time.time()
            while time.time() - t0 < 5.0 and os.path.getsize(self.path) == 0:
                time.sleep(0.02)
        except Exception:
            self.proc = None

    def stop(self, t_begin: float, t_end: float):
        import datetime
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "window": "timed region"}
        if self.proc is None:
            return out
        try:
            time.sleep(0.05)
            self.proc.terminate()
            self.proc.wait(timeout=5)
            rows = [l.strip().split(", ") for l in open(self.path) if l.strip()]
            os.unlink(self.path)
        except Exception:
            return out
        inside, anyload, mx = [], [], None
        for r in rows:
            if len(r) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(r[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                mhz = float(r[1]); mx = float(r[2])
            except ValueError:
                continue
            reasons = [name for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9])
                       if v.strip().lower().startswith("active")]
            anyload.append((mhz, reasons))
            if t_begin - 0.01 <= ts <= t_end + 0.01:
                inside.append((mhz, reasons))
        use = inside
        if not use:
            use = anyload
            out["window"] = "whole run (timed region shorter than the sampling period)"
        if use:
            out.update(sm_mhz=statistics.median([u[0] for u in use]), sm_max_mhz=mx,
                       reasons=sorted({x for u in use for x in u[1]}), samples=len(use))
        return out


# ------------------------------------------------------------------------------------------------ CPU oracle legs
def oracle_times(names, keep=()):
    """One full evaluation of the CPU oracle, as it stands, per configuration on the host cores.  Returns
    ({name: {"oracle_s", "cores"}}, {name: output for the names in `keep`}).  No process pool is started (OpenMP threads
    inside one C call), and it runs before the first CUDA call of the process."""
    import oracle
    from paper_2505_18574_b200 import bench_details, inputs
    oracle.build()
    times, kept = {}, {}
    for name in names:
        p = bench_details._problem(name)
        t0 = time.perf_counter()
        if isinstance(p, inputs.GemmProblem):
            out = oracle.gemm_i8(p.A, p.a_rs, p.a_cs, p.B, p.b_rs, p.b_cs, p.ldc, p.bias, p.mult, p.shift, p.per_channel,
                                 p.M, p.N, p.K, p.relu)
        elif isinstance(p, inputs.ConvProblem):
            out = oracle.conv2d_i8(p.x, p.w, p.bias, p.mult, p.shift, p.per_channel, p.N, p.H, p.W, p.C, p.K, p.R, p.S,
                                   p.stride_h, p.stride_w, p.pad_h, p.pad_w, p.relu)
        elif isinstance(p, inputs.MpcProblem):
            out = oracle.mpc_forward(p.Adyn, p.Bdyn, p.Kinf, p.x0, p.d)
        else:
            out = oracle.batched_gemm_i8(p.A, p.K, 1, p.M * p.K, p.B, p.N, 1, p.K * p.N, p.N, p.M * p.N, p.bias, p.bias_bs,
                                         p.mult, p.shift, p.per_channel, p.batch, p.M, p.N, p.K, p.relu)
        times[name] = {"oracle_s": time.perf_counter() - t0, "cores": oracle.num_threads()}
        if name in keep:
            kept[name] = out
    return times, kept


def run_reference(args, rank, world):
    """The oracle timed on the host cores, on this benchmark's workload (rank 0 only)."""
    if rank != 0:
        return
    from paper_2505_18574_b200 import inputs
    import oracle
    oracle.build()
    problems = [inputs.config1(j) for j in range(3)]
    rows = {0: 512, 1: 128, 2: 256}     # per step: a bounded slab of each problem (scaled down below for long runs)

    def step():
        macs = 0.0
        for j, p in enumerate(problems):
            r = rows[j]
            A = np.ascontiguousarray(p.A[:r])
            oracle.gemm_i8(A, p.a_rs, 1, p.B, p.b_rs, p.b_cs, p.N, p.bias, p.mult, p.shift, p.per_channel, r, p.N, p.K, p.relu)
            macs += float(r) * p.N * p.K
        return macs

    # keep the whole run to a couple of minutes: one calibration step, then shrink the slabs if K steps would take longer
    t0 = time.perf_counter()
    step()
    t_base = time.perf_counter() - t0
    budget_s = 100.0
    if (args.steps + args.warmup) * t_base > budget_s:
        f = max(budget_s / ((args.steps + args.warmup) * t_base), 1.0 / 32.0)
        rows = {j: max(16, int(r * f) // 16 * 16) for j, r in rows.items()}
    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    macs = 0.0
    for _ in range(args.steps):
        macs += step()
    dt = time.perf_counter() - t0
    tops = 2.0 * macs / dt / 1e12
    sample = "per step: " + ", ".join(f"{rows[j]} rows of {p.M}x{p.N}x{p.K}" for j, p in enumerate(problems))
    line = {"impl": "reference", "metric": METRIC, "value": tops, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "i8", "data": "synthetic",
            "config": {"workload": WORKLOAD, "note": "CPU oracle (plain C loops, OpenMP over rows) on a row slab per step"},
            "cpu_baseline": {"value": tops, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": tops, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------ GPU arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-details", action="store_true", help="skip the per-problem timings of the other workload configurations")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    from paper_2505_18574_b200 import inputs
    problems = [inputs.config1(j) for j in range(3)]

    # The CPU baseline runs before the first CUDA call of this process (rank 0, single-GPU runs only): one full oracle
    # evaluation of the three headline problems (about 15 s on 16 cores; also the reference of the full-output parity
    # check below) and of every other configuration listed in `details`.
    cpu_baseline, oracle_t, oracle_out = None, None, {}
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from paper_2505_18574_b200 import bench_details
        names = ["1a", "1b", "1c"] + ([] if args.no_details else [n for n in bench_details.ALL if n not in ("1a", "1b", "1c")])
        oracle_t, oracle_out = oracle_times(names, keep=("1a", "1b", "1c"))
        t_cfg1 = sum(oracle_t[n]["oracle_s"] for n in ("1a", "1b", "1c"))
        cpu_baseline = {"value": sum(gemm_ops(p) for p in problems) / t_cfg1 / 1e12, "unit": UNIT,
                        "cores": oracle_t["1a"]["cores"], "kind": "oracle",
                        "sample": f"the whole workload: every row of the three problems, one evaluation each ({t_cfg1:.1f} s wall)"}

    import torch
    import torch.distributed as dist
    import paper_2505_18574_b200 as i8

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    from paper_2505_18574_b200 import sharding
    if rank != 0:                       # independent problems per rank: same shapes, different draws
        problems = [inputs.make_gemm(p.M, p.N, p.K, sharding.rank_seed(p.seed, rank), per_channel=1, relu=0, name=p.name)
                    for p in problems]

    dev_t = []
    for p in problems:
        dev_t.append(dict(A=torch.from_numpy(p.A).to(dev), B=torch.from_numpy(p.B).to(dev),
                          C=torch.empty((p.M, p.N), dtype=torch.int8, device=dev), bias=torch.from_numpy(p.bias).to(dev),
                          mult=torch.from_numpy(p.mult).to(dev), shift=torch.from_numpy(p.shift).to(dev)))

    def launch(j):
        d, p = dev_t[j], problems[j]
        i8.gemm_i8(d["A"], d["B"].t(), d["C"], d["bias"], d["mult"], d["shift"], p.per_channel, p.relu)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # parity spot check on this rank's draws before timing (sampled rows against the oracle on rank 0)
    bit_exact = None
    launch(0); launch(1); launch(2)
    torch.cuda.synchronize()
    assert i8.last_device_status() == 0
    assert i8.last_path() in (i8.PATH_TENSOR, i8.PATH_TENSOR_2SM, i8.PATH_CHANNEL_MAJOR, i8.PATH_CHANNEL_MAJOR_2SM), "the tensor path did not run"
    if rank == 0 and oracle_out:
        # every element of all three outputs against the oracle's
        bit_exact = all(bool(np.array_equal(dev_t[j]["C"].cpu().numpy(), oracle_out[n][:, :problems[j].N]))
                        for j, n in enumerate(("1a", "1b", "1c")))
        oracle_out = {}

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    for _ in range(args.warmup):
        launch(0); launch(1); launch(2)
    barrier()

    n_launch = 3 * args.steps
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(n_launch + 1)]
    barrier()
    t_begin = time.time()
    evs[0].record()
    k = 0
    for _ in range(args.steps):
        for j in range(3):
            launch(j)
            k += 1
            evs[k].record()
    barrier()
    t_end = time.time()
    clocks = sampler.stop(t_begin, t_end) if rank == 0 else None
    total_ms = evs[0].elapsed_time(evs[-1])
    per_problem_ms = [0.0, 0.0, 0.0]
    for s in range(args.steps):
        for j in range(3):
            per_problem_ms[j] += evs[3 * s + j].elapsed_time(evs[3 * s + j + 1])
    per_problem_ms = [t / args.steps for t in per_problem_ms]
    assert i8.last_device_status() == 0

    total_ms_max = sharding.max_over_ranks(total_ms, dev)
    ops_step = sum(gemm_ops(p) for p in problems)
    value = sharding.whole_job_rate(ops_step * args.steps, world, total_ms_max) / 1e12

    # ---- end to end through the host-buffer entry point (pinned host memory, copies inside the timed region)
    host = []
    for p in problems:
        host.append(dict(A=torch.from_numpy(p.A).pin_memory(), B=torch.from_numpy(p.B).pin_memory(),
                         C=torch.empty((p.M, p.N), dtype=torch.int8).pin_memory(), bias=torch.from_numpy(p.bias).pin_memory(),
                         mult=torch.from_numpy(p.mult).pin_memory(), shift=torch.from_numpy(p.shift).pin_memory()))

    def e2e_step():
        for j, p in enumerate(problems):
            h = host[j]
            i8.gemm_i8_host(h["A"], h["B"], h["C"], h["bias"], h["mult"], h["shift"], p.per_channel, p.relu)

    e2e_step()                          # grows the library's device workspace once
    barrier()
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.e2e_steps):
        e2e_step()
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    e2e_value = sharding.whole_job_rate(ops_step * args.e2e_steps, world, sharding.max_over_ranks(e2e_ms, dev)) / 1e12
    h2d = sum(p.M * p.K + p.N * p.K + 4 * p.N * 3 for p in problems)
    d2h = sum(p.M * p.N for p in problems)
    e2e_exact = all(np.array_equal(host[j]["C"].numpy(), dev_t[j]["C"].cpu().numpy()) for j in range(3))

    # Strong scaling beside the per-rank replicas (several GPUs only): ONE 16384 x 4096 x 8192 problem, its rows split
    # across the ranks (no exchange step; every rank holds B), timed on the device as the max over ranks.
    strong = None
    if world > 1:
        p2, d2 = problems[2], dev_t[2]
        call = lambda: sharding.sharded_gemm_i8(d2["A"], d2["B"].t(), d2["bias"], d2["mult"], d2["shift"], p2.per_channel, p2.relu,
                                                world=world, rank=rank, out=d2["C"][:sharding.row_shard(p2.M, world, rank)[1]])
        for _ in range(3):
            call()
        barrier()
        s0 = torch.cuda.Event(enable_timing=True); s1 = torch.cuda.Event(enable_timing=True)
        s0.record()
        for _ in range(20):
            call()
        s1.record()
        barrier()
        ms = sharding.max_over_ranks(s0.elapsed_time(s1) / 20, dev)
        strong = {"problem": p2.name, "rows_per_rank": sharding.row_shard(p2.M, world, 0)[1], "ms": ms, "tops": gemm_ops(p2) / (ms * 1e-3) / 1e12,
                  "scaling": "strong"}

    details, probe = None, None
    if rank == 0 and world == 1:
        from paper_2505_18574_b200 import bench_details
        pk = measured_peaks()
        if not args.no_details:
            time.sleep(0.5)             # the per-configuration timings start from an idle GPU, not from the power-capped clock
            details = bench_details.run(dev, peak_tops=2 * pk["bf16_burst"], peak_gbs=pk["hbm_gbs"], oracle=oracle_t)
        # this library's own tensor-core issue-rate probe (operands resident in shared memory): burst and sustained
        time.sleep(0.5)                 # the burst figure is taken from an idle GPU as well
        probe = bench_details.run_peak(dev)

    if rank == 0:
        peaks = measured_peaks()
        # Which cuBLAS-derived peak applies depends on how long the timed region ran: the power cap settles the clock
        # within a few tens of milliseconds, so short regions are compared with the burst figure, long ones with the
        # sustained one.  Both fractions are printed.
        peak_burst = peaks["bf16_burst"] * NOMINAL_INT8_OVER_BF16
        peak_sustained = peaks["bf16_sustained"] * NOMINAL_INT8_OVER_BF16
        long_region = total_ms_max > 100.0
        peak_int8 = peak_sustained if long_region else peak_burst
        kernel_ms = sum(per_problem_ms)
        achieved = ops_step / (kernel_ms * 1e-3) / 1e12
        algo_bytes = sum(gemm_bytes(p) for p in problems)
        roof = {"bound": "tensor", "kernel": "gemm_i8_tc_kernel<256,6,0,8,1,1> (CTA pairs, 256x256 tiles, cta_group::2)",
                "achieved": achieved, "peak": peak_int8, "unit": "TFLOP/s", "frac": achieved / peak_int8,
                "peak_source": f"{peaks['source']}: cuBLAS bf16 {'sustained' if long_region else 'burst'} "
                               f"{peaks['bf16_sustained'] if long_region else peaks['bf16_burst']} TFLOP/s x {NOMINAL_INT8_OVER_BF16} "
                               f"(nominal int8:bf16 ratio); the timed region ran {total_ms_max:.0f} ms "
                               f"({'more' if long_region else 'less'} than 100 ms)",
                "frac_of_burst_peak": achieved / peak_burst, "frac_of_sustained_peak": achieved / peak_sustained,
                "frac_of_nominal_4500": achieved / 4500.0,
                "traffic": NCU_STEP_TRAFFIC_BYTES / 3.0, "algorithmic_bytes": algo_bytes / 3.0,
                "traffic_over_algorithmic": NCU_STEP_TRAFFIC_BYTES / algo_bytes,
                "traffic_note": "DRAM bytes read+written per launch, averaged over the step's three launches, from a recorded ncu "
                                "launch list of this command (profiles/bench_config1_launch_list.txt), not measured in this run; "
                                "the excess over the algorithmic bytes is operand tiles re-read through L2 (DRAM is at ~11 % of "
                                "its peak: not the limiter)"}
        if clocks and clocks.get("sm_mhz"):
            # 128 x 256 x 32 per 128 cycles per SM = 16384 int8 operations per clock per SM (this library's issue-rate
            # probe, `bench_details --cfg peak`), at the SM clock sampled during the timed region
            clock_peak = 148 * 16384 * clocks["sm_mhz"] * 1e6 / 1e12
            roof["peak_issue_rate_at_sampled_clock"] = clock_peak
            roof["frac_of_issue_rate_at_sampled_clock"] = achieved / clock_peak
        if probe:
            pb = next(r for r in probe if r["kind"] == "burst" and r["tile_n"] == 256)
            ps = next(r for r in probe if r["kind"].startswith("sustained"))
            roof["probe"] = {"burst_tops": pb["tops"], "sustained_tops": ps["tops"], "cycles_per_128x256x32": pb["cycles_per_mma"],
                             "burst_sm_mhz": pb["sm_mhz"], "sustained_sm_mhz": ps["sm_mhz"],
                             "what": "tcgen05.mma kind::i8 issued back to back on shared-memory-resident operands on all SMs"}
            roof["frac_of_probe_peak"] = achieved / (ps["tops"] if long_region else pb["tops"])
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": total_ms_max / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "i8", "data": "synthetic",
            "config": {"workload": WORKLOAD, "parallelism": f"independent problems per rank x{world}",
                       "l2": "inputs larger than L2: one step streams 475 MB of operands and outputs through a 126 MB L2, "
                             "so each problem's tiles are evicted before its next launch",
                       "per_problem_ms": {p.name: per_problem_ms[j] for j, p in enumerate(problems)},
                       "per_problem_tops": {p.name: gemm_ops(p) / (per_problem_ms[j] * 1e-3) / 1e12 for j, p in enumerate(problems)}},
            "roofline": roof,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": args.e2e_steps, "matches_device_path": bool(e2e_exact)},
            "gpu_launches": n_launch,
            "clocks": {"sm_mhz": clocks["sm_mhz"], "sm_max_mhz": clocks["sm_max_mhz"], "reasons": clocks["reasons"],
                       "samples": clocks["samples"], "window": clocks["window"]},
            "bit_exact_vs_oracle": bit_exact,
        }
        if strong is not None:
            line["strong_scaling_row_sharded"] = strong
        if cpu_baseline is not None:
            line["cpu_baseline"] = cpu_baseline
        if details is not None:
            line["details"] = details
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
