#!/usr/bin/env python
"""Benchmark of the Conv-BN-SiLU forward + backward path on B200.

A "step" is one forward call, one backward-data call and one backward-weight call of the C ABI for every
Conv-BN-SiLU layer of the workload (default: the 77 layers of the YOLOv8m-class detector at batch 16,
640 x 640; each layer on its own seeded synthetic tensors of the right shape).  One JSON line is printed:

  value / ms_per_step : whole-job TFLOP/s (2*M*K*Cout per GEMM, three GEMMs per layer) and ms per step with all
                        tensors resident in HBM, timed with CUDA events over exactly --steps steps;
  e2e                 : the same through nb_conv_bn_silu_step_host from pinned host buffers, copies inside the timing;
  roofline            : per-kernel-site device times from an instrumented pass (events around every launch) for the
                        site that takes the largest share, against the measured peak;
  cpu_baseline        : the fp64 CPU oracle timed on this host on a bounded sample of the same workload.

`--impl reference` times the CPU oracle alone (the paper ships no code to install as a reference).
Multi-GPU (`torchrun`): the path does not shard, so every rank runs an independent replica (weak scaling).
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "conv_bn_silu_fwd_bwd_bf16_tflops"
UNIT = "TFLOP/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}


# DRAM traffic of one launch divided by its algorithmic bytes, measured with ncu (dram__bytes_read.sum +
# dram__bytes_write.sum) on SINGLE-kernel captures of small cases whose tensors exceed L2: benchmark configuration 3 for
# the three GEMM kernels (79 MB tensors), configuration 2 (157 MB tensors) for the elementwise passes.  Reads equal the
# algorithmic bytes; part of what a kernel writes is still in L2 when it ends, hence ratios below 1.  roofline.traffic of
# a full-size launch is this ratio times the launch's algorithmic bytes (traffic grows in proportion to the tensor sizes).
NCU_TRAFFIC_OVER_ALGORITHMIC = {
    "conv_fprop": 0.75, "conv_dgrad": 0.76, "conv_wgrad": 1.03,
    "bn_silu_apply": 0.86, "bn_silu_bwd_reduce": 1.01, "bn_silu_bwd_dy": 0.92,
}


def cpu_model() -> str:
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def spread(ms_list):
    """mean / median / min of per-step device times (milliseconds)."""
    v = sorted(ms_list)
    n = len(v)
    med = v[n // 2] if n % 2 else 0.5 * (v[n // 2 - 1] + v[n // 2])
    return {"mean": sum(v) / n, "median": med, "min": v[0], "max": v[-1], "steps": n}


def write_per_layer(path, blocks, per_shape, peaks):
    """Markdown table: per distinct layer shape, the instrumented device time of each kernel site per launch and what it
    means against the measured peaks (the times include a few microseconds of launch latency per kernel)."""
    counts = {}
    for b in blocks:
        counts[b.shape.key] = counts.get(b.shape.key, 0) + 1
    lines = ["| layer shape (Cin, Cout, k, stride, H) | layers | fprop us (TFLOP/s, % of peak) | dgrad us | wgrad+reduce us | apply us (GB/s) | bwd reduce us (GB/s) | dy us (GB/s) |",
             "|---|---|---|---|---|---|---|---|"]
    for key, rec in per_shape.items():
        s, st = rec["shape"], rec["sites"]
        us = lambda site: (st[site][0] / st[site][1] * 1e3) if site in st else 0.0
        def gemm(site, extra=None):
            t = us(site) + (us(extra) if extra else 0.0)
            if t <= 0:
                return "-"
            tf = s.gemm_flops / (t * 1e-6) / 1e12
            return "%.1f (%.0f, %.0f %%)" % (t, tf, 100.0 * tf / peaks["bf16_tflops"])
        def ew(site):
            t = us(site)
            if t <= 0:
                return "-"
            return "%.1f (%.0f)" % (t, site_work(site, s)[1] / (t * 1e-6) / 1e9)
        lines.append("| (%d, %d, %d, %d, %d) | %d | %s | %s | %s | %s | %s | %s |" % (
            s.c_in, s.c_out, s.k, s.stride, s.h, counts[key], gemm("conv_fprop"), gemm("conv_dgrad"), gemm("conv_wgrad", "wgrad_splitk_reduce"),
            ew("bn_silu_apply"), ew("bn_silu_bwd_reduce"), ew("bn_silu_bwd_dy")))
    with open(path, "w") as f:
        f.write("\n".join(lines) + "\n")


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS if k in p} | {"source": "measured"}
    return dict(FALLBACK_PEAKS) | {"source": "fallback"}


def workload_layers(name: str):
    from paper_2609_10632_b200 import workloads as wl

    if name.startswith("cfg"):
        return wl.config_shapes(int(name[3:]))
    raise SystemExit(f"unknown workload {name}")


def step_flops(layers) -> float:
    return float(sum(3 * s.gemm_flops for s in layers))


# ----------------------------------------------------------------------------- algorithmic work per kernel site
def site_work(site: str, s):
    """(flops, bytes) one launch of `site` must perform/move for layer shape s (bf16 activations, fp16 saved y)."""
    out_e = s.m * s.c_out
    in_b = 2 * s.n * s.h * s.w * s.c_in
    w_b = 2 * s.kdim * s.c_out
    if site == "conv_fprop":
        return s.gemm_flops, in_b + w_b + 2 * out_e
    if site == "conv_dgrad":
        return s.gemm_flops, in_b + w_b + 2 * out_e
    if site == "conv_wgrad":
        return s.gemm_flops, in_b + 2 * out_e + 4 * s.kdim * s.c_out
    if site == "bn_stats":
        return 3 * out_e, 2 * out_e
    if site == "bn_silu_apply":
        return 10 * out_e, 4 * out_e
    if site == "bn_silu_bwd_reduce":
        return 15 * out_e, 4 * out_e
    if site == "bn_silu_bwd_dy":
        return 18 * out_e, 6 * out_e
    if site == "dgrad_weight_transform":
        return 0, 2 * w_b
    return 0, 0


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def __exit__(self, *a):
        if self.proc:
            time.sleep(0.15)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                self.proc.kill()

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for nm, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------- CPU oracle timing
def time_oracle(layers, budget_s: float):
    """Time the oracle (forward + backward of whole blocks) on a bounded sample of the workload: every distinct layer
    shape once, at a reduced batch chosen so that the pass takes roughly `budget_s` seconds (batch 1 is timed first to
    size it).  Returns (TFLOP/s, seconds, flops, cores, description)."""
    import oracle
    from paper_2609_10632_b200 import workloads as wl

    oracle.build()
    cores = oracle.num_threads()

    def one_pass(batch):
        distinct = wl.distinct_shapes([s.with_batch(min(batch, s.n)) for s in layers])
        flops, secs = 0.0, 0.0
        for i, (s, _mult) in enumerate(distinct):
            inp = wl.make_inputs(s, cfg_id=5, layer_id=i, bf16=True)
            t0 = time.perf_counter()
            oracle.cbs_fwd_bwd(inp.x, inp.w, inp.gamma, inp.beta, inp.g, s.stride, 1e-3)
            secs += time.perf_counter() - t0
            flops += 3 * s.gemm_flops
        return flops, secs, len(distinct)

    full_batch = max(s.n for s in layers)
    flops, secs, nshapes = one_pass(1)
    batch = 1
    if full_batch > 1 and secs > 0:
        batch = int(max(1, min(full_batch, budget_s / secs)))
        if batch > 1:
            flops, secs, nshapes = one_pass(batch)
    desc = f"{nshapes} distinct layer shapes at batch {batch} (of {full_batch}), one fwd+bwd each, fp64 direct loops"
    return flops / secs / 1e12, secs, flops, cores, desc


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    layers = workload_layers(args.workload)
    total = args.steps + args.warmup
    budget = max(1.0, min(30.0, 120.0 / max(1, total)))
    vals, secs_all = [], []
    desc, cores = "", 0
    for i in range(total):
        v, secs, flops, cores, desc = time_oracle(layers, budget)
        if i >= args.warmup:
            vals.append(v)
            secs_all.append(secs)
    value = sum(vals) / len(vals)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * sum(secs_all) / len(secs_all), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "note": "fp64 CPU oracle on a bounded sample per step; ms_per_step is the sample's time"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "cpu": cpu_model(), "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def max_over_ranks(ms: float, dist, device) -> float:
    """The step time of a multi-process run is the slowest rank's (replicas only: no data-path collective, the only
    communication of the benchmark is this reduction and the barriers around the timed region)."""
    if dist is None:
        return ms
    import torch

    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world: int, flops_per_replica: float, ms_step: float) -> float:
    """TFLOP/s of all replicas together: every rank does the same work (weak scaling) in the slowest rank's time."""
    return world * flops_per_replica / (ms_step * 1e-3) / 1e12


# ----------------------------------------------------------------------------- GPU arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--workload", default="cfg5", help="cfg1..cfg5 (cfg5 = the detector's 77 Conv-BN-SiLU layers at batch 16)")
    ap.add_argument("--per-layer", default=None, help="write a per-layer-shape table of the instrumented kernel times to this file")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--e2e-streams", type=int, default=6, help="streams of the end-to-end arm (1 = no overlap of copies and compute)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--f16", action="store_true", help="run the per-layer step in NB_MODE_F16_TC (fp16 operands, the paper's own 16-bit format) "
                    "instead of bf16; the chained-detector and end-to-end objects are skipped")
    ap.add_argument("--no-chain", action="store_true", help="skip the chained C2f units measurement (extra object of the JSON line)")
    ap.add_argument("--no-optimizer", action="store_true", help="skip the fused clip + SGD-Nesterov step measurement (extra object of the JSON line)")
    ap.add_argument("--no-eval-forward", action="store_true", help="skip the evaluation-mode forward measurement (extra object of the JSON line)")
    ap.add_argument("--no-profile", action="store_true")
    ap.add_argument("--cpu-budget", type=float, default=20.0, help="seconds of oracle work for cpu_baseline")
    ap.add_argument("--force-simt", action="store_true", help="run the convolutions on the CUDA-core kernels")
    ap.add_argument("--no-wgrad-stream", action="store_true", help="queue the weight gradients on the main stream instead of a second stream")
    ap.add_argument("--no-graph", action="store_true", help="launch every kernel from the host instead of replaying a CUDA graph of one step")
    ap.add_argument("--sustain-seconds", type=float, default=2.0, help="length of the additional sustained region in seconds of device time (0 = skip)")
    ap.add_argument("--no-configs", action="store_true", help="skip the per-configuration figures (cfg2, cfg3, cfg4a, cfg4b)")
    ap.add_argument("--only-chain", action="store_true", help="run only the chained-detector measurement and print its object (with --no-graph: "
                    "eager launches, for a profiler's launch list)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.warmup < 3:
        print(f"note: warmup {args.warmup} < 3 breaks the timing rules", file=sys.stderr)

    import torch

    from paper_2609_10632_b200 import binding as nb
    from paper_2609_10632_b200 import workloads as wl
    from paper_2609_10632_b200.block import CbsBlock

    nb.load()  # fails loudly if the CUDA library is missing
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if args.only_chain:
        print(json.dumps({"detector_chain": run_detector_chain(args, dev, local, load_peaks(), step_flops(workload_layers("cfg5")))}), flush=True)
        return
    dist = None
    if world > 1:
        import torch.distributed as dist_mod

        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)

    layers = workload_layers(args.workload)
    flags = nb.NB_CBS_FLAG_FORCE_SIMT if args.force_simt else 0
    plans_probe = [nb.Plan.for_shape(s, flags=flags, device=local) for s in layers]
    ws_bytes = max(max(p.fwd_bytes, p.bwd_bytes) for p in plans_probe)
    del plans_probe
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    mode = nb.NB_MODE_F16_TC if args.f16 else nb.NB_MODE_BF16_TC
    if args.f16:
        args.no_chain = args.no_e2e = True
    blocks = [CbsBlock(s, mode=mode, flags=flags, device=local, workspace=ws) for s in layers]
    for i, b in enumerate(blocks):
        b.fill_random(seed=1000 + i)
    resident = sum(sum(t.numel() * t.element_size() for t in (b.x, b.w, b.g, b.y, b.a, b.dy, b.dx, b.dw)) for b in blocks)
    flops = step_flops(layers)
    stream = torch.cuda.current_stream()

    # The weight gradient of a layer depends only on dy and x, so it goes to a second stream (with a workspace of its
    # own) and overlaps the kernels that follow on the main stream; the step ends when both streams have finished.
    wgrad_stream = None if args.no_wgrad_stream else torch.cuda.Stream(device=dev)
    wgrad_ws = None if args.no_wgrad_stream else torch.empty(ws_bytes, dtype=torch.uint8, device=dev)

    def one_step():
        if wgrad_stream is None:
            for b in blocks:
                b.step()
            return
        main = torch.cuda.current_stream()
        wgrad_stream.wait_stream(main)
        for b in blocks:
            b.step(wgrad_stream=wgrad_stream, wgrad_workspace=wgrad_ws)
        main.wait_stream(wgrad_stream)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        one_step()
    for b in blocks:
        b.poll()
    barrier()
    # The step is launch-bound on its small layers (about 770 kernels): capture one step of C-ABI calls into a CUDA
    # graph and replay it.  Every call only enqueues kernels on the current stream, so the capture holds exactly the
    # kernels an eager step launches.
    l0 = nb.nb_cbs_launch_count()
    graph = None
    if not args.no_graph:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            one_step()
        torch.cuda.current_stream().wait_stream(side)
        l0 = nb.nb_cbs_launch_count()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            one_step()
        launches_per_step = nb.nb_cbs_launch_count() - l0
        run_step = graph.replay
        for _ in range(2):
            run_step()
    else:
        run_step = one_step
        launches_per_step = None
    barrier()
    stream = torch.cuda.current_stream()
    l0 = nb.nb_cbs_launch_count()
    # Exactly --steps steps between two events; an event after every step gives the spread (mean / median / min).
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    with ClockSampler(local) as clocks:
        marks[0].record(stream)
        for i in range(args.steps):
            run_step()
            marks[i + 1].record(stream)
        barrier()
    launches = launches_per_step * args.steps if launches_per_step is not None else nb.nb_cbs_launch_count() - l0
    for b in blocks:
        b.poll()
    ms_total = marks[0].elapsed_time(marks[-1])
    per_step = spread([marks[i].elapsed_time(marks[i + 1]) for i in range(args.steps)])
    ms_total = max_over_ranks(ms_total, dist, dev)
    ms_step = ms_total / args.steps
    value = whole_job_value(world, flops, ms_step)
    peaks = load_peaks()
    # The same step for at least --sustain-seconds of device time (default 2 s), with its own clock record: the timed
    # region above lasts a fraction of a second at boost clock, this one shows what a long run settles at.
    sustained = None
    if args.sustain_seconds > 0:
        n_sus = max(args.steps, int(args.sustain_seconds * 1e3 / ms_step) + 1)
        smarks = [torch.cuda.Event(enable_timing=True) for _ in range(n_sus + 1)]
        barrier()
        with ClockSampler(local) as sclocks:
            smarks[0].record(stream)
            for i in range(n_sus):
                run_step()
                smarks[i + 1].record(stream)
            barrier()
        for b in blocks:
            b.poll()
        sus_ms = max_over_ranks(smarks[0].elapsed_time(smarks[-1]), dist, dev)
        sustained = spread([smarks[i].elapsed_time(smarks[i + 1]) for i in range(n_sus)]) | {
            "ms_per_step": sus_ms / n_sus, "value": whole_job_value(world, flops, sus_ms / n_sus), "unit": UNIT, "seconds": sus_ms * 1e-3, "clocks": sclocks.summary()}

    # ---------------- instrumented pass: per-site device times (events around every launch; calls wait for each kernel)
    roofline, kernels = None, {}
    if not args.no_profile:
        for b in blocks:
            nb.nb_cbs_profile_enable(b.plan, True)
        prof_steps = max(1, min(args.steps, 3))
        for _ in range(prof_steps):
            one_step()
        torch.cuda.synchronize()
        agg = {}
        per_shape = {}  # distinct layer shape -> site -> [ms, launches]
        for b in blocks:
            for site, (ms, n) in nb.nb_cbs_profile_read(b.plan).items():
                if n == 0:
                    continue
                ps = per_shape.setdefault(b.shape.key, {"shape": b.shape, "count": 0, "sites": {}})["sites"].setdefault(site, [0.0, 0])
                ps[0] += ms
                ps[1] += n
                f, by = site_work(site, b.shape)
                a = agg.setdefault(site, {"ms": 0.0, "launches": 0, "flops": 0.0, "bytes": 0.0})
                a["ms"] += ms
                a["launches"] += n
                a["flops"] += f * n
                a["bytes"] += by * n
            nb.nb_cbs_profile_enable(b.plan, False)
        tot_ms = sum(a["ms"] for a in agg.values()) or 1.0
        tensor_sites = {"conv_fprop", "conv_dgrad", "conv_wgrad"}
        if args.per_layer and rank == 0:
            write_per_layer(args.per_layer, blocks, per_shape, peaks)
        for site, a in agg.items():
            sec = a["ms"] * 1e-3
            k = {"launches": a["launches"], "ms_per_step": a["ms"] / prof_steps, "share": a["ms"] / tot_ms}
            if site in tensor_sites:
                k["tflops"] = a["flops"] / sec / 1e12
                k["gbs_algorithmic"] = a["bytes"] / sec / 1e9
            else:
                k["gbs"] = a["bytes"] / sec / 1e9
            kernels[site] = k
        top = max(agg, key=lambda s: agg[s]["ms"])
        a = agg[top]
        sec = a["ms"] * 1e-3
        if top in tensor_sites:
            ach = a["flops"] / sec / 1e12
            # a GEMM site that moves more bytes than its flops justify is HBM-bound (arithmetic intensity under the ridge)
            ridge = peaks["bf16_tflops"] * 1e12 / (peaks["hbm_gbs"] * 1e9)
            if a["flops"] / max(a["bytes"], 1.0) >= ridge:
                roofline = {"kernel": top, "bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s"}
            else:
                roofline = {"kernel": top, "bound": "hbm", "achieved": a["bytes"] / sec / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
        else:
            roofline = {"kernel": top, "bound": "hbm", "achieved": a["bytes"] / sec / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
        roofline["frac"] = roofline["achieved"] / roofline["peak"]
        ratio = NCU_TRAFFIC_OVER_ALGORITHMIC.get(top)
        roofline["traffic"] = ratio * a["bytes"] / a["launches"] if ratio else None
        roofline["traffic_note"] = ("DRAM bytes per launch = algorithmic bytes per launch (%.3g, average over the site's launches of one step) x %s, the "
                                    "ratio ncu measured on a single-kernel capture of a small case of the same kernel; inside a step most layers' "
                                    "tensors are found in the 126 MB L2, so the real traffic is lower" % (a["bytes"] / a["launches"], ratio))
        roofline["peak_source"] = peaks["source"] + (" (burst figure: kernels timed one at a time)" if roofline["bound"] == "tensor" else "")
        roofline["avg_launch_ms"] = a["ms"] / a["launches"]
        roofline["share_of_step"] = a["ms"] / tot_ms

    # ---------------- the evaluation-mode forward (running statistics; one fused kernel per tensor-core layer)
    eval_fwd = None
    if not args.no_eval_forward:
        eval_fwd = run_eval_forward(args, blocks, dev, flops / 3.0, peaks, kernels)

    # ---------------- the fused optimiser step over the detector's 243 gradient tensors
    opt_step = None
    if not args.no_optimizer and args.workload == "cfg5":
        opt_step = run_optimizer_step(args, blocks, dev, local, peaks)

    # ---------------- the whole detector as CHAINED blocks (split / add / concat / pool / upsample glue included)
    chain = None
    if not args.no_chain and args.workload == "cfg5":
        chain = run_detector_chain(args, dev, local, peaks, flops)

    # ---------------- end to end from pinned host buffers through the C ABI
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(args, layers, blocks, flags, local, dev, dist, world, flops)

    # ---------------- the other benchmark configurations, one by one (cfg2 stem, cfg3, cfg4a, cfg4b)
    cfgs = None
    if not args.no_configs and args.workload == "cfg5" and not args.f16:
        cfgs = run_configs(args, dev, local, peaks, ws, wgrad_ws)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, secs, fl, cores, desc = time_oracle(layers, args.cpu_budget)
        cpu = {"value": v, "unit": UNIT, "cores": cores, "cpu": cpu_model(), "kind": "oracle", "sample": f"{desc}; {secs:.1f} s"}

    if rank == 0:
        paths = {"fprop": 0, "dgrad": 0, "wgrad": 0}
        for b in blocks:
            for k in paths:
                paths[k] += b.plan.paths[k]
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "ms_per_step_spread": per_step, "sustained": sustained, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f16" if args.f16 else "bf16", "data": "synthetic",
            "config": {
                "workload": f"{args.workload}: {len(layers)} Conv-BN-SiLU layers, batch {layers[0].n}, fwd + bwd_data + bwd_weight per layer "
                            f"(stem data gradient included), each layer on its own tensors",
                "l2_policy": f"inputs larger than L2: {resident / 1e9:.2f} GB of tensors are touched per step",
                "gflop_per_step": flops / 1e9, "multi_gpu": "replicas only", "cuda_graph": graph is not None, "wgrad_on_second_stream": wgrad_stream is not None, "tensor_core_layers": paths, "layers": len(layers),
                "frac_of_nominal_bf16_peak": value / world / NOMINAL["bf16_tflops"],
                "frac_of_measured_sustained_bf16_peak": value / world / peaks["bf16_tflops_sustained"],
            },
            "clocks": clocks.summary(), "gpu_launches": int(launches), "e2e": e2e, "roofline": roofline, "cpu_baseline": cpu,
            "kernels": kernels, "configs": cfgs, "eval_forward": eval_fwd, "optimizer_step": opt_step, "detector_chain": chain,
        }
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def run_configs(args, dev, local, peaks, ws, wgrad_ws):
    """Benchmark configurations 2, 3, 4a and 4b on their own: one training step of that layer as a CUDA-graph replay (weight
    gradient on the main stream: a single layer has nothing to overlap it with), repeated with an L2 flush between
    replays left out on purpose for cfg2 / cfg3, whose tensors (157 MB / 79 MB each) exceed L2 anyway; per kernel site
    the device time of an instrumented pass and what it means against the measured peaks."""
    import torch

    from paper_2609_10632_b200 import binding as nb
    from paper_2609_10632_b200 import workloads as wl
    from paper_2609_10632_b200.block import CbsBlock

    out = {}
    shapes = [("cfg2", wl.config_shapes(2)[0]), ("cfg3", wl.config_shapes(3)[0])] + list(zip(("cfg4a", "cfg4b"), wl.config_shapes(4)))
    for name, s in shapes:
        blk = CbsBlock(s, device=local)
        blk.fill_random(seed=4000)
        for _ in range(3):
            blk.step()
        torch.cuda.synchronize()
        blk.poll()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            blk.step()
        n = 100
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        marks = [torch.cuda.Event(enable_timing=True) for _ in range(n + 1)]
        marks[0].record()
        for i in range(n):
            graph.replay()
            marks[i + 1].record()
        torch.cuda.synchronize()
        blk.poll()
        sp = spread([marks[i].elapsed_time(marks[i + 1]) for i in range(n)])
        fl = 3 * s.gemm_flops
        rec = {"shape": [s.n, s.h, s.w, s.c_in, s.c_out, s.k, s.stride], "ms_per_step": sp["mean"], "ms_median": sp["median"], "ms_min": sp["min"],
               "tflops": fl / (sp["mean"] * 1e-3) / 1e12, "frac_of_measured_bf16_peak": fl / (sp["mean"] * 1e-3) / 1e12 / peaks["bf16_tflops"], "kernels": {}}
        nb.nb_cbs_profile_enable(blk.plan, True)
        for _ in range(5):
            blk.step()
        torch.cuda.synchronize()
        for site, (ms, cnt) in nb.nb_cbs_profile_read(blk.plan).items():
            if cnt == 0:
                continue
            f, by = site_work(site, s)
            us = ms / cnt * 1e3
            k = {"us": us}
            if site in ("conv_fprop", "conv_dgrad", "conv_wgrad"):
                k["tflops"] = f / (us * 1e-6) / 1e12
                k["frac_of_measured_bf16_peak"] = k["tflops"] / peaks["bf16_tflops"]
            elif by:
                k["gbs"] = by / (us * 1e-6) / 1e9
                k["frac_of_measured_hbm_peak"] = k["gbs"] / peaks["hbm_gbs"]
            rec["kernels"][site] = k
        nb.nb_cbs_profile_enable(blk.plan, False)
        out[name] = rec
        del blk, graph
        torch.cuda.empty_cache()
    return out


def run_eval_forward(args, blocks, dev, fwd_flops, peaks, kernels):
    """The evaluation-mode forward of every layer (nb_conv_bn_silu_infer: running statistics, no saved tensors) as a
    CUDA-graph replay on this rank; reported beside the training step, not part of `value`."""
    import torch

    from paper_2609_10632_b200 import binding as nb

    gen = torch.Generator(device=dev)
    gen.manual_seed(4242)
    ws = torch.empty(max(max(b.plan.infer_bytes for b in blocks), 256), dtype=torch.uint8, device=dev)
    stats = []
    for b in blocks:
        c = b.shape.c_out
        stats.append((0.2 * torch.randn(c, generator=gen, device=dev), 0.25 + 0.5 * torch.rand(c, generator=gen, device=dev)))

    def fwd_all():
        for b, (rm, rv) in zip(blocks, stats):
            nb.nb_conv_bn_silu_infer(b.plan, b.x, b.w, b.gamma, b.beta, rm, rv, b.a, ws)

    for _ in range(max(3, args.warmup)):
        fwd_all()
    torch.cuda.synchronize()
    l0 = nb.nb_cbs_launch_count()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        fwd_all()
    launches = nb.nb_cbs_launch_count() - l0
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.steps):
        graph.replay()
    ev1.record()
    torch.cuda.synchronize()
    for b in blocks:
        b.poll()
    ms = ev0.elapsed_time(ev1) / args.steps
    train_fwd = sum(kernels[k]["ms_per_step"] for k in ("conv_fprop", "bn_stats", "bn_finalize", "bn_silu_apply") if k in kernels) if kernels else None
    tf = fwd_flops / (ms * 1e-3) / 1e12
    return {"call": "nb_conv_bn_silu_infer", "ms_per_pass": ms, "tflops": tf, "frac_of_measured_bf16_peak": tf / peaks["bf16_tflops"],
            "launches_per_pass": int(launches), "fused_layers": sum(1 for b in blocks if b.plan.infer_fused), "layers": len(blocks),
            "training_forward_kernels_ms": train_fwd, "cuda_graph": True}


def run_detector_chain(args, dev, local, peaks, step_flops_value):
    """The 77 blocks run as the detector's dataflow (workloads.detector_graph): every block consumes the previous blocks'
    activations and gradients, joined by the glue calls (channel split / concat, residual add, 5x5 max-pools, 2x
    upsampling, gradient accumulation at fan-out).  Forward + backward from a uniform[0,1] image batch and random
    gradients at the six head tensors, as one CUDA-graph replay.  Same convolution work as the per-layer step."""
    import torch

    from paper_2609_10632_b200 import binding as nb
    from paper_2609_10632_b200 import workloads as wl
    from paper_2609_10632_b200.detector import GraphRunner

    ops, layers, outs, plain = wl.detector_graph(16, 640, plain_head=True)  # up to the six raw head outputs
    run = GraphRunner(ops, layers, outs, device=local, plain_layers=plain)
    run.fill_parameters(seed=7000)
    for pl in run.plain:
        pl["w"].normal_(0.0, 0.05)
        pl["bias"].normal_(0.0, 0.5)
    run.buf["img"].uniform_(0.0, 1.0)
    for name in outs:
        run.grad[name].normal_()

    side = None if args.no_wgrad_stream else torch.cuda.Stream(device=dev)
    side_ws = None if side is None else torch.empty(max(b.plan.bwd_bytes for b in run.blocks), dtype=torch.uint8, device=dev)
    # the optimiser step over the chain's 243 gradient tensors: fp32 masters and momentum here, the blocks' bf16 filters are
    # the working copies it rewrites; BN gains / shifts and the plain biases are fp32 parameters updated in place
    items = []
    for b in run.blocks:
        items.append((b.dw, b.w.float().reshape(-1).clone(), torch.zeros(b.w.numel(), dtype=torch.float32, device=dev), b.w, 0))
        items.append((b.dgamma, b.gamma, torch.zeros_like(b.gamma), None, 1))
        items.append((b.dbeta, b.beta, torch.zeros_like(b.beta), None, 2))
    for pl in run.plain:
        items.append((pl["dw"], pl["w"].float().reshape(-1).clone(), torch.zeros(pl["w"].numel(), dtype=torch.float32, device=dev), pl["w"], 0))
        items.append((pl["dbias"], pl["bias"], torch.zeros_like(pl["bias"]), None, 2))
    sgd = nb.SgdPlan(items, device=local)
    sgd_ws = torch.empty(sgd.workspace_bytes, dtype=torch.uint8, device=dev)
    sgd.upload(sgd_ws)
    hyper = dict(lr=[1e-4, 1e-4, 1e-4], weight_decay=[3.75e-4, 0.0, 0.0], momentum=0.937, max_norm=10.0)  # Table 1 (small lr: random gradients)

    def step(with_update=False):
        run.forward()
        if side is None:
            run.backward()
        else:
            main = torch.cuda.current_stream()
            side.wait_stream(main)
            run.backward(wgrad_stream=side, wgrad_workspace=side_ws)
            main.wait_stream(side)
        if with_update:
            sgd.step(sgd_ws, first_step=False, **hyper)

    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize()
    run.poll()
    if args.no_graph:  # eager launches only (a profiler's launch list); no timing claims
        l0 = nb.nb_cbs_launch_count()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for _ in range(args.steps):
            step()
        ev1.record()
        torch.cuda.synchronize()
        run.poll()
        return {"ms_per_step": ev0.elapsed_time(ev1) / args.steps, "launches_per_step": int((nb.nb_cbs_launch_count() - l0) / args.steps),
                "glue_launches_fwd_bwd": list(run.glue_launches()), "cuda_graph": False}
    l0 = nb.nb_cbs_launch_count()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    launches = nb.nb_cbs_launch_count() - l0
    graph.replay()
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.steps):
        graph.replay()
    ev1.record()
    torch.cuda.synchronize()
    run.poll()
    ms = ev0.elapsed_time(ev1) / args.steps
    # the same with the clip + SGD-Nesterov update of all 243 tensors behind it: one training iteration minus the loss
    sgd.step(sgd_ws, first_step=True, **hyper)
    torch.cuda.synchronize()
    graph2 = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph2):
        step(with_update=True)
    graph2.replay()
    torch.cuda.synchronize()
    ev0.record()
    for _ in range(args.steps):
        graph2.replay()
    ev1.record()
    torch.cuda.synchronize()
    run.poll()
    ms_upd = ev0.elapsed_time(ev1) / args.steps
    finite = all(bool(torch.isfinite(b.w.float()).all()) for b in run.blocks[:3])
    gf, gb = run.glue_launches()
    tf = step_flops_value / (ms * 1e-3) / 1e12
    return {"what": "77 chained Conv-BN-SiLU blocks + 6 plain head convolutions + glue, image -> raw head outputs, fwd + bwd, batch 16, 640 x 640", "wgrad_on_second_stream": side is not None, "ms_per_step": ms, "tflops": tf,
            "frac_of_measured_bf16_peak": tf / peaks["bf16_tflops"], "launches_per_step": int(launches), "glue_launches_fwd_bwd": [gf, gb],
            "ms_per_step_with_optimizer_update": ms_upd, "optimizer_tensors": len(items), "weights_finite_after_updates": finite, "cuda_graph": True}


def run_optimizer_step(args, blocks, dev, local, peaks):
    """nb_sgd_clip_nesterov_step over the detector's 243 trainable tensors (the 77 layers' dw / dgamma / dbeta as gradients
    and their bf16 filters as working copies, plus the six plain head convolutions), timed as a CUDA-graph replay."""
    import torch

    from paper_2609_10632_b200 import binding as nb
    from paper_2609_10632_b200 import workloads as wl

    gen = torch.Generator(device=dev)
    gen.manual_seed(777)
    items, elems, lp_elems = [], 0, 0

    def add(grad, lp, group):
        nonlocal elems, lp_elems
        n = grad.numel()
        master = (lp.float().clone() if lp is not None else torch.randn(n, generator=gen, device=dev) * 0.05).reshape(-1)
        items.append((grad, master, torch.empty(n, dtype=torch.float32, device=dev), lp, group))
        elems += n
        lp_elems += n if lp is not None else 0

    for b in blocks:
        add(b.dw, b.w, 0)
        add(b.dgamma, None, 1)
        add(b.dbeta, None, 2)
    for cin, cout in wl.detector_plain_head_convs():
        add(torch.randn(cout * cin, generator=gen, device=dev) * 0.01, torch.empty(cout * cin, dtype=torch.bfloat16, device=dev), 0)
        add(torch.randn(cout, generator=gen, device=dev) * 0.01, None, 2)
    plan = nb.SgdPlan(items, device=local)
    ws = torch.empty(plan.workspace_bytes, dtype=torch.uint8, device=dev)
    plan.upload(ws)
    norm = torch.zeros(1, dtype=torch.float32, device=dev)
    hyper = dict(lr=[0.01, 0.01, 0.01], weight_decay=[3.75e-4, 0.0, 0.0], momentum=0.937, max_norm=10.0)  # Table 1
    plan.step(ws, first_step=True, total_norm=norm, **hyper)
    for _ in range(max(3, args.warmup)):
        plan.step(ws, first_step=False, total_norm=norm, **hyper)
    torch.cuda.synchronize()
    l0 = nb.nb_cbs_launch_count()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        plan.step(ws, first_step=False, total_norm=norm, **hyper)
    launches = nb.nb_cbs_launch_count() - l0
    graph.replay()
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.steps):
        graph.replay()
    ev1.record()
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1) / args.steps
    # norm pass reads g; update reads g, p, momentum and writes p, momentum (4 bytes each) and the bf16 copy of the filters
    algo_bytes = elems * 4 * 6 + lp_elems * 2
    gbs = algo_bytes / (ms * 1e-3) / 1e9
    return {"call": "nb_sgd_clip_nesterov_step", "tensors": len(items), "parameters": int(elems), "ms_per_step": ms, "launches_per_step": int(launches),
            "algorithmic_bytes": int(algo_bytes), "gbs": gbs, "frac_of_measured_hbm_peak": gbs / peaks["hbm_gbs"], "grad_norm": float(norm.item()),
            "cuda_graph": True, "note": "the 311 MB of gradients, parameters and momentum fit the 126 MB L2 only in part: warm replays re-read some of them from L2"}


def run_e2e(args, layers, blocks, flags, local, dev, dist, world, flops):
    """Whole steps through nb_conv_bn_silu_step_host: pinned host inputs -> device -> three calls -> pinned host outputs."""
    import torch

    from paper_2609_10632_b200 import binding as nb

    host = {}  # per distinct shape: pinned input and output buffers (inputs filled from the device tensors)
    scratch_bytes = 0
    h2d = d2h = 0
    for b in blocks:
        s = b.shape
        scratch_bytes = max(scratch_bytes, b.plan.step_host_scratch_bytes())
        if s.key not in host:
            pin = lambda t: torch.empty(t.shape, dtype=t.dtype).pin_memory()
            hin = {k: pin(getattr(b, k)) for k in ("x", "w", "gamma", "beta", "g")}
            for k, t in hin.items():
                t.copy_(getattr(b, k))
            hout = {k: pin(getattr(b, k)) for k in ("a", "dx", "dw", "dgamma", "dbeta")}
            host[s.key] = (hin, hout)
        hin, hout = host[s.key]
        h2d += sum(t.numel() * t.element_size() for t in hin.values())
        d2h += sum(t.numel() * t.element_size() for t in hout.values())
    # Several streams (--e2e-streams, default 6), each with its own device scratch, take the layers in turn: while one layer computes, the next
    # layer's inputs arrive over PCIe and the previous layer's results leave (the two copy directions run concurrently).
    # Layers of the same shape share a plan and may then be in flight on different streams at once, so the plans of this arm
    # are created with NB_CBS_FLAG_SEPARATE_FINALIZE: all scratch of a call then lies in the workspace it was given (a default
    # plan sums its statistics in accumulators of its own, which only one call at a time may use).
    nstreams = max(1, args.e2e_streams)
    plans = {}
    for b in blocks:
        if b.shape.key not in plans:
            plans[b.shape.key] = nb.Plan.for_shape(b.shape, flags=flags | (nb.NB_CBS_FLAG_SEPARATE_FINALIZE if nstreams > 1 else 0), device=local)
    scratches = [torch.empty(scratch_bytes, dtype=torch.uint8, device=dev) for _ in range(nstreams)]
    main = torch.cuda.current_stream()
    streams = [main] if nstreams == 1 else [torch.cuda.Stream(device=dev) for _ in range(nstreams)]

    def one():
        for i, b in enumerate(blocks):
            hin, hout = host[b.shape.key]
            k = i % nstreams
            nb.nb_conv_bn_silu_step_host(plans[b.shape.key], hin["x"], hin["w"], hin["gamma"], hin["beta"], hin["g"], hout["a"], hout["dx"],
                                         hout["dw"], hout["dgamma"], hout["dbeta"], scratches[k], stream=streams[k])

    def fork():  # the side streams start after everything already queued on the main stream
        if nstreams > 1:
            e = torch.cuda.Event()
            e.record(main)
            for st in streams:
                st.wait_event(e)

    def join():  # the main stream continues after all side streams
        if nstreams > 1:
            for st in streams:
                e = torch.cuda.Event()
                e.record(st)
                main.wait_event(e)

    steps = max(1, min(args.steps, 20))  # (the main arm's step count, up to 20: a step moves 7.3 GB over PCIe)
    fork()
    one()
    join()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(main)
    fork()
    for _ in range(steps):
        one()
    join()
    ev1.record(main)
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1)
    ms = max_over_ranks(ms, dist, dev)
    return {"value": whole_job_value(world, flops, ms / steps), "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
            "ms_per_step": ms / steps, "steps": steps, "streams": nstreams}


if __name__ == "__main__":
    main()
