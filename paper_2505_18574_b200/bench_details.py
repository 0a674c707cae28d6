"""Per-problem timings of every workload configuration (GEMM 256^3, the three large GEMMs, the four
convolutions, the tall-skinny GEMM and the batched 64^3 products, a batch of 128^3 products, a 4096^3 GEMM with row-major
B; `--cfg mpc` adds the fp32 TinyMPC forward pass over
2^20 instances, `--cfg sweep` the shapes the paper prints, `--cfg peak` the tensor-core issue-rate probe that gives the
int8 roofline its measured denominator) through the C-ABI binding.

    python -m paper_2505_18574_b200.bench_details [--cfg 0,1a,2,...] [--iters N] [--no-graph]

For each problem: device time per launch from back-to-back launches between two CUDA events (arguments marshalled
once, so the loop only crosses the C ABI, as a C caller's loop would), the same from a CUDA graph of the launches
(launch gaps removed), int8 TOPS, algorithmic GB/s (every operand read once, the output written once) and the fraction
of the roofline max(ops / tensor peak, bytes / HBM peak).  Problems whose operands fit in L2 are rotated over enough
copies of their buffers to exceed it (the cold figure, the one every roofline fraction uses); `us_warm_l2` is the same
launch repeated over a single buffer set.  `run(oracle=...)` takes the wall times of the CPU baseline that the
repository's `bench.py` measures on the host cores and reports them beside each configuration.
"""
from __future__ import annotations

import argparse
import json
import os

import numpy as np

# Order of a full run: the microsecond kernels first, the three large GEMMs last.  Those run for milliseconds at the power
# cap, and the lowered clock outlasts them: timed right behind them, the 56 x 56 convolution measured 11-13 us against
# 9.1 us from an idle GPU, the next configuration 8.4 against 7.3, the ones after that unchanged.
ALL = ["0", "2", "3a", "3b", "3c", "4a", "4b", "b128", "mpc", "rmB", "1a", "1b", "1c"]
# the shapes the paper prints: "g0".."g9" (inputs.SWEEP_GEMMS) and "c0", "c1" (inputs.SWEEP_CONVS)
SWEEP = [f"g{i}" for i in range(10)] + ["c0", "c1"]
L2_BYTES = 126e6


def _problem(name):
    from . import inputs
    if name == "mpc":
        return inputs.make_mpc(1 << 20)
    if name == "rmB":
        return inputs.extra_rowmajor_b()
    if name == "b128":
        return inputs.extra_batched_128()
    if name[0] == "g":
        return inputs.sweep_gemm(int(name[1:]))
    if name[0] == "c":
        return inputs.sweep_conv(int(name[1:]))
    return {"0": inputs.config0, "1a": lambda: inputs.config1(0), "1b": lambda: inputs.config1(1),
            "1c": lambda: inputs.config1(2), "2": inputs.config2, "3a": lambda: inputs.config3(0),
            "3b": lambda: inputs.config3(1), "3c": lambda: inputs.config3(2), "4a": inputs.config4a,
            "4b": inputs.config4b}[name]()


def _make(name, dev, copies_for_l2=True):
    """Returns (problem name, one prepared call per buffer set, ops, algorithmic bytes, number of buffer sets)."""
    import torch
    from . import binding as i8
    from . import inputs
    p = _problem(name)

    def T(a):
        return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(dev)

    if isinstance(p, inputs.GemmProblem):
        ops = 2.0 * p.M * p.N * p.K
        byts = p.M * p.K + p.N * p.K + p.M * p.N + 4 * p.N + 8 * (p.N if p.per_channel else 1)
        sets = int(min(16, max(1, np.ceil(2 * L2_BYTES / byts)))) if copies_for_l2 else 1
        b, mu, sh = T(p.bias), T(p.mult), T(p.shift)
        calls = []
        for _ in range(sets):
            A, B, C = T(p.A), T(p.B), torch.empty((p.M, p.N), dtype=torch.int8, device=dev)
            Bv = B.t() if p.b_rs == 1 else B           # logical (K, N): stored (N, K) K-contiguous, or row-major as it is
            calls.append(i8.prepare("gemm_i8", A, Bv, C, b, mu, sh, p.per_channel, p.relu))
    elif isinstance(p, inputs.ConvProblem):
        ops = 2.0 * p.N * p.P * p.Q * p.K * p.R * p.S * p.C
        byts = p.x.size + p.w.size + p.N * p.P * p.Q * p.K + 12 * p.K
        sets = int(min(32, max(1, np.ceil(2 * L2_BYTES / byts)))) if copies_for_l2 else 1
        b, mu, sh = T(p.bias), T(p.mult), T(p.shift)
        calls = []
        for _ in range(sets):
            x, w, y = T(p.x), T(p.w), torch.empty((p.N, p.P, p.Q, p.K), dtype=torch.int8, device=dev)
            calls.append(i8.prepare("conv2d_i8", x, w, y, b, mu, sh, p.per_channel, p.relu, (p.stride_h, p.stride_w),
                                    (p.pad_h, p.pad_w)))
    elif isinstance(p, inputs.MpcProblem):
        # flops: per step 2*4*12 + 4 (u) and 2*12*12 + 2*12*4 + 12 (x), the last step without the state update
        ops = p.batch * (p.nhorizon * 100.0 + (p.nhorizon - 1) * 396.0)
        byts = p.batch * (48 + 32 * p.nhorizon)
        sets = 1
        x0, d = T(p.x0), T(p.d)
        u = torch.empty((p.batch, p.nhorizon, 4), dtype=torch.float32, device=dev)
        calls = [lambda: i8.mpc_forward_f32(p.Adyn, p.Bdyn, p.Kinf, x0, d, u)]
    else:
        ops = 2.0 * p.batch * p.M * p.N * p.K
        byts = p.A.size + p.B.size + p.batch * p.M * p.N + p.bias.size * 4
        sets = 1
        A, B, C = T(p.A), T(p.B), torch.empty((p.batch, p.M, p.N), dtype=torch.int8, device=dev)
        b, mu, sh = T(p.bias), T(p.mult), T(p.shift)
        calls = [i8.prepare("batched_gemm_i8", A, B, C, b, mu, sh, p.per_channel, p.relu)]

    return p.name, calls, ops, byts, sets


def _on_stream(calls, stream):
    """Prepared calls carry the stream that was current when they were made; graph capture runs on a side stream."""
    return [c.with_stream(stream) if hasattr(c, "with_stream") else c for c in calls]


def run_peak(dev=None):
    """The tensor-core issue-rate probe: burst (a fraction of a millisecond) and sustained (the last of several
    launches of ~80 ms each, by when the power cap has settled the clock) for the 256-wide instruction, and the per-
    instruction cycle counts of the narrower ones."""
    from . import binding as i8
    out = []
    for n in (256, 128, 64):
        r = i8.probe_mma_rate(n, reps=4096)            # warm-up
        r = i8.probe_mma_rate(n, reps=4096)
        r["kind"] = "burst"
        out.append(r)
    last = None
    for _ in range(6):
        last = i8.probe_mma_rate(256, reps=1 << 20)
    last["kind"] = "sustained (sixth of six back-to-back launches)"
    out.append(last)
    return out


def run(dev=None, cfgs=None, iters=50, graph=True, peak_tops=None, peak_gbs=None, oracle=None):
    """`oracle`: {configuration: {"oracle_s", "cores"}}, CPU-baseline wall times measured by the caller, reported beside
    each configuration."""
    import torch
    from . import binding as i8
    dev = dev or torch.device("cuda", 0)
    out = []
    for name in (cfgs or ALL):
        pname, calls, ops, byts, sets = _make(name, dev)

        def launch(i, calls=calls):
            calls[i % sets]()
        for i in range(max(5, sets)):
            launch(i)
        torch.cuda.synchronize()
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(iters):
            launch(i)
        e1.record(); torch.cuda.synchronize()
        us_loop = e0.elapsed_time(e1) / iters * 1e3
        us_graph = None
        if graph:
            g = torch.cuda.CUDAGraph(); s = torch.cuda.Stream()
            with torch.cuda.stream(s):
                gcalls = _on_stream(calls, s)
                gcalls[0](); torch.cuda.synchronize()
                with torch.cuda.graph(g, stream=s):
                    for i in range(iters):
                        gcalls[i % sets]()
            torch.cuda.synchronize()
            g.replay(); torch.cuda.synchronize()
            e0.record(); g.replay(); e1.record(); torch.cuda.synchronize()
            us_graph = e0.elapsed_time(e1) / iters * 1e3
        us = min(us_loop, us_graph) if us_graph is not None else us_loop
        # the same launch over ONE buffer set (operands and output stay in L2 between launches): reported beside the
        # cold figure, never used for a roofline claim
        us_warm = None
        if graph and sets > 1:
            gw = torch.cuda.CUDAGraph(); sw = torch.cuda.Stream()
            with torch.cuda.stream(sw):
                wcall = _on_stream(calls, sw)[0]
                wcall(); torch.cuda.synchronize()
                with torch.cuda.graph(gw, stream=sw):
                    for i in range(iters):
                        wcall()
            torch.cuda.synchronize()
            gw.replay(); torch.cuda.synchronize()
            e0.record(); gw.replay(); e1.record(); torch.cuda.synchronize()
            us_warm = e0.elapsed_time(e1) / iters * 1e3
        rec = {"problem": pname, "us_per_launch": us, "us_loop": us_loop, "us_graph": us_graph, "tops": ops / us / 1e6,
               "gbs": byts / us / 1e3, "us_warm_l2": us_warm, "path": i8.last_path(), "buffer_sets": sets,
               "device_status": i8.last_device_status()}
        if peak_tops and peak_gbs:
            t_roof = max(ops / (peak_tops * 1e12), byts / (peak_gbs * 1e9)) * 1e6
            rec["roofline_us"] = t_roof
            rec["roofline_frac"] = t_roof / us
            rec["bound"] = "tensor" if ops / (peak_tops * 1e12) >= byts / (peak_gbs * 1e9) else "hbm"
            t_nom = max(ops / 4500e12, byts / 8000e9) * 1e6
            rec["roofline_frac_nominal"] = t_nom / us
        if oracle and name in oracle:
            rec["oracle_s"] = oracle[name]["oracle_s"]
            rec["oracle_cores"] = oracle[name]["cores"]
            rec["oracle_tops"] = ops / oracle[name]["oracle_s"] / 1e12
        out.append(rec)
    return out


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("--cfg", default=",".join(ALL), help="comma list of configurations, 'sweep' for the paper's printed shapes, 'peak' for the issue-rate probe")
    ap.add_argument("--iters", type=int, default=50)
    ap.add_argument("--no-graph", action="store_true")
    a = ap.parse_args()
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    pk = os.path.join(root, "MEASURED_PEAKS.json")
    peak_tops, peak_gbs = 2 * 1590.0, 6650.0
    if os.path.exists(pk):
        d = json.load(open(pk)); peak_tops, peak_gbs = 2 * d["bf16_tflops"], d["hbm_gbs"]
    if a.cfg == "peak":
        for r in run_peak():
            print(json.dumps(r), flush=True)
    else:
        cfgs = SWEEP if a.cfg == "sweep" else a.cfg.split(",")
        for r in run(cfgs=cfgs, iters=a.iters, graph=not a.no_graph, peak_tops=peak_tops, peak_gbs=peak_gbs):
            print(json.dumps(r), flush=True)
