#!/usr/bin/env python
"""Benchmark of the ScaleKV per-scale hot path on B200.

One "step" = one full pass of the workload: after a reset, for every scale k and every layer,
append -> attend -> compress (no compress after the last scale).  The metric is scale-steps per
second (one scale-step = append + attend + compress of every layer at one scale); passes per
second is printed beside it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload pass2b] [--impl reference]

Prints one JSON line.  Inputs are seeded synthetic tensors (see paper_2505_19602_b200/synth.py),
generated on the device before the timed region.  With --gpus N > 1 (under torchrun) every rank
runs an independent replica on its own batch: the path shards by batch with no collective.
"""
import argparse
import dataclasses
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "scale_steps_per_sec"
# DRAM traffic of the attend kernel: (dram__bytes_read.sum + dram__bytes_write.sum) / algorithmic bytes over the two
# launches of an ncu capture of one layer of the headline workload, its two largest scales (592.2 + 956.3 = 1548.5 MB
# measured against 1676 MB algorithmic: part of the appended rows is still in L2 when a launch ends).  The capture runs
# one layer of the workload; traffic grows in proportion to the bytes a launch must move, so the roofline object reports
# this ratio times the average algorithmic bytes per launch.  Captured on the kernel as of the commit named below
# (profiles/attend_tc_kernel_pass2b_1layer.md); set ATTEND_TRAFFIC_RATIO to None when attend_tc.cuh changes after it.
ATTEND_TRAFFIC_RATIO = 1110.5 / 1128.4
ATTEND_TRAFFIC_SOURCE = ("ncu capture of attend_tc_kernel at commit 319ec61 (one layer, scales 12 and 13), scaled to the "
                         "average launch by algorithmic bytes")
UNIT = "scale-steps/s"
E2E_HOST_LAYERS = 4


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="scalekv", choices=["scalekv", "reference"])
    ap.add_argument("--workload", default="pass2b")
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (profiling on a small case)")
    ap.add_argument("--full-cache", action="store_true", help="KEEP_ALL budgets instead of drafter/refiner budgets")
    ap.add_argument("--overall-pct", type=float, default=0.0,
                    help="overall budget in per cent of the cached tokens (the 4 / 10 / 20 sweep of the 16-scale workload): "
                         "refiner budget = overall / 3.25, drafter budget = 10 x refiner; default: 30 %% / 3 %%")
    ap.add_argument("--delta", type=float, default=None,
                    help="budget table from Eq. 4 with the paper's constants (650 tokens per head and layer on average, "
                         "B_r(0) = 600) and this refiner decay rate (Sec. 4.3 sweeps 0 .. 70) instead of 30 %% / 3 %%")
    ap.add_argument("--policy", default="scalekv", choices=["scalekv", "sliding", "sinks", "snapkv", "pyramid"],
                    help="keep-rule timed on the same store at equal total budget: the paper's (default) or one of the "
                         "comparison policies of Sec. 4.1 (see include/scalekv.h, scalekv_policy_budgets)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-side-stream", action="store_true")
    ap.add_argument("--no-graph", action="store_true",
                    help="launch the timed passes call by call instead of replaying a CUDA graph of one pass")
    ap.add_argument("--cpu-sample-slices", type=int, default=16)
    return ap.parse_args()


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); power.append(float(r[2]))
            except ValueError:
                continue
            for name, v in zip(["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"], r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_burst": p["bf16_tflops"], "bf16_sustained": p["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


def workload_from_args(args):
    from paper_2505_19602_b200 import synth

    wl = synth.WORKLOADS[args.workload]
    if args.layers:
        nd = max(1, round(wl.n_drafters * args.layers / wl.n_layers)) if wl.n_drafters else 0
        wl = dataclasses.replace(wl, n_layers=args.layers, n_drafters=nd)
    return wl


# --------------------------------------------------------------------------------------------
# CPU oracle legs (cpu_baseline of the main line; the whole of --impl reference)
# --------------------------------------------------------------------------------------------
def oracle_threads():
    try:
        from threadpoolctl import threadpool_info

        n = [i.get("num_threads", 1) for i in threadpool_info()]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def oracle_slice_pass(wl, layer, b, h, budgets, windows):
    """One slice's full pass on the CPU oracle.  Returns seconds."""
    import numpy as np

    from oracle import scalekv_oracle as orc
    from paper_2505_19602_b200 import synth

    one = dataclasses.replace(wl)
    cache = orc.SliceCache(wl.n_tokens, wl.head_dim)
    data = []
    for k in range(wl.n_scales):
        Q, K, V = synth.scale_inputs(one, layer, k)
        data.append(tuple(t[b, h].double().numpy() for t in (Q, K, V)))
    t0 = time.perf_counter()
    for k in range(wl.n_scales):
        Q, K, V = data[k]
        cache.append(K, V)
        cache.attend(Q)
        if k + 1 < wl.n_scales:
            w = windows[k] if windows[k] is not None else list(range(wl.n_tokens[k]))
            cache.compress(Q[w], w, budgets[layer][k])
    return time.perf_counter() - t0


def oracle_rate(wl, budgets, windows, n_sample):
    """scale-steps/s of the oracle extrapolated from a sample of slices (slices are independent)."""
    small = dataclasses.replace(wl, batch=1, n_heads=1)        # same per-slice shapes, cheap to generate
    layers = sorted(set(round(i * (wl.n_layers - 1) / max(n_sample - 1, 1)) for i in range(n_sample)))
    secs = [oracle_slice_pass(small, l, 0, 0, budgets, windows) for l in layers]
    per_slice = sum(secs) / len(secs)
    total = per_slice * wl.n_slices
    return wl.n_scales / total, f"{len(layers)} slices (layers {layers}, batch 0, head 0), full {wl.n_scales}-scale pass each, " \
                                f"{per_slice:.2f} s per slice-pass, extrapolated to {wl.n_slices} slices"


def host_policy(wl, args):
    """Budgets and windows.  Roles of the timed workloads come from scalekv_layer_stats when a GPU
    is present; the reference arm (CPU only) uses the planted drafter layers directly."""
    from oracle import scalekv_oracle as orc

    windows = [orc.window_centroids(a, a, wl.window) for a in wl.sides]
    return windows


def reference_budgets(wl, full_cache):
    from oracle import scalekv_oracle as orc
    from paper_2505_19602_b200 import synth

    if full_cache or wl.n_drafters == 0 and wl.name != "layer2b":
        return [[orc.KEEP_ALL] * wl.n_scales for _ in range(wl.n_layers)]
    n = wl.n_tokens
    if wl.n_drafters == 0:
        b = orc.budget_tokens(0.10, n)
        return [[b] * wl.n_scales for _ in range(wl.n_layers)]
    planted = set(synth.drafter_layers(wl))
    bd, br = orc.budget_tokens(0.30, n), orc.budget_tokens(0.03, n)
    return [[bd if l in planted else br] * wl.n_scales for l in range(wl.n_layers)]


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = workload_from_args(args)
    windows = host_policy(wl, args)
    budgets = reference_budgets(wl, args.full_cache)
    rates = []
    note = ""
    t_all = time.perf_counter()
    for i in range(args.warmup + args.steps):
        r, note = oracle_rate(wl, budgets, windows, 4)
        if i >= args.warmup:
            rates.append(r)
    value = statistics.mean(rates)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1000.0 * wl.n_scales / value, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "layers": wl.n_layers, "batch": wl.batch, "heads": wl.n_heads, "head_dim": wl.head_dim,
                   "scales": wl.n_scales, "budget": "full" if args.full_cache else "drafter 30% / refiner 3%"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                         "sample": "per step: " + note},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0, "wall_s": time.perf_counter() - t_all,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------------------------
# Multi-rank plumbing (no data-path collective: every rank owns its own batch of images)
# --------------------------------------------------------------------------------------------
def rank_workload(wl, rank, world):
    """The workload of one rank: same shapes, its own seed, so that every rank owns a different batch."""
    return dataclasses.replace(wl, seed=wl.seed + 1000 * rank) if world > 1 else wl


def max_over_ranks(x, world, device="cpu"):
    """Slowest rank's time: the job is done when the last rank is."""
    if world <= 1:
        return float(x)
    import torch
    import torch.distributed as dist

    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(n_scales, steps, world, ms_max):
    """Whole-job scale-steps per second: all ranks' scale-steps over the slowest rank's time."""
    return n_scales * steps * world / (ms_max / 1000.0)


# --------------------------------------------------------------------------------------------
# CUDA arm
# --------------------------------------------------------------------------------------------
def run_scalekv(args):
    import torch
    import torch.distributed as dist

    from paper_2505_19602_b200 import binding, pipeline, synth

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    wl = workload_from_args(args)
    wl = rank_workload(wl, rank, world)
    peaks = load_peaks()
    windows = pipeline.windows_for(wl.sides, wl.window)

    # budgets: drafter / refiner roles per scale from the offline statistics on seeded inputs
    t0 = time.perf_counter()
    if args.full_cache:
        budgets = [[binding.KEEP_ALL] * wl.n_scales for _ in range(wl.n_layers)]
        role_note = "full cache"
    elif wl.n_drafters > 0:
        asi, roles = pipeline.calibrate_roles(wl, wl.n_drafters, device=local_rank)
        if args.overall_pct > 0:
            r1000 = max(1, round(args.overall_pct * 1000 / 3.25))          # refiner share in 1/100000 of T_c
            budgets = pipeline.budget_table(wl, roles, drafter_frac=10 * r1000 / 100000, refiner_frac=r1000 / 100000)
        else:
            budgets = pipeline.budget_table(wl, roles)
        if args.delta is not None:
            budgets = [[int(x) for x in row] for row in binding.scalekv_make_budgets(roles, 650, 600, args.delta)]
        planted = synth.drafter_layers(wl)
        # Eq. 2 cannot tell the roles apart while the history is shorter than K' (then the top-K' mass is all of the
        # history mass and ASI = c (1 - c) is symmetric): count the recovery over the scales with a longer history
        n_cum = [sum(wl.n_tokens[:k]) for k in range(wl.n_scales)]
        ks = [k for k in range(1, wl.n_scales - 1) if n_cum[k] > 4 * 16]
        hits = sum(int(roles[l][k]) for k in ks for l in planted)
        role_note = (f"{wl.n_drafters} drafters per scale from scalekv_layer_stats; {hits}/{len(planted) * len(ks)} planted "
                     f"drafters recovered at the {len(ks)} scales whose history exceeds 4 K'")
        if args.delta is not None:
            role_note += f"; Eq. 4 table: 650 average, B_r(0) = 600, delta = {args.delta:g}"

    else:
        b = binding.scalekv_budget_tokens(0.10, wl.sides)
        budgets = [[b] * wl.n_scales for _ in range(wl.n_layers)]
        role_note = "uniform 10%"
    calib_s = time.perf_counter() - t0
    # the comparison policies run at the total budget of the table above: its mean over layers, window included
    select, window_kind = None, "centroids"
    if args.policy != "scalekv":
        args.no_e2e = args.no_cpu_baseline = True      # those legs run the paper's rule; an A/B line is kernel timing only
        w_obs = min(wl.window, binding.MAX_WINDOW)
        k_ref = wl.n_scales - 2
        mean_cache = sum(min(budgets[l][k_ref], 10 ** 9) + w_obs for l in range(wl.n_layers)) / wl.n_layers
        if args.policy in ("sliding", "sinks"):
            table = binding.scalekv_policy_budgets("uniform", wl.n_layers, wl.n_scales, mean_cache)
            select = {"policy": "recent", "n_sink": 4 if args.policy == "sinks" else 0}
        else:
            table = binding.scalekv_policy_budgets("uniform" if args.policy == "snapkv" else "pyramid", wl.n_layers, wl.n_scales,
                                                   mean_cache - w_obs, 20.0)
            select = {"policy": "score", "pool_kernel": 7}
            window_kind = "last"
            windows = [binding.scalekv_window_last(a, a, w_obs) for a in wl.sides]
        budgets = [[int(x) for x in row] for row in table]
        role_note = f"policy {args.policy} at {mean_cache:.1f} cached tokens per head and layer on average"

    def make_kv():
        return binding.ScaleKV(wl.n_layers, wl.batch, wl.n_heads, wl.head_dim, wl.dtype, wl.sides, wl.sides, budgets,
                               max_window=min(wl.window, binding.MAX_WINDOW), device=local_rank,
                               side_stream=not args.no_side_stream, window_kind=window_kind)

    kv = make_kv()
    inputs = pipeline.PassInputs(wl, device=local_rank)
    work = pipeline.pass_work(wl, budgets, windows, recent=select is not None and select["policy"] == "recent",
                              one_call_steps=True)
    torch.cuda.synchronize()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    pass_marks = []

    def timed_passes(n_pass, graph=None):
        # one event per pass boundary on stream_main (a pass starts with a reset, which joins the side
        # stream): the region as a whole gives the reported time, the boundaries its spread
        marks = [torch.cuda.Event(enable_timing=True) for _ in range(n_pass + 1)]
        for i in range(n_pass):
            with torch.cuda.stream(kv.stream_main):
                marks[i].record()
                if graph is not None:
                    graph.replay()
            if graph is None:
                pipeline.run_pass(kv, inputs, windows, select=select)
        kv.scalekv_join()
        with torch.cuda.stream(kv.stream_main):
            marks[n_pass].record()
        kv.scalekv_sync()
        pass_marks[:] = [marks[i].elapsed_time(marks[i + 1]) for i in range(n_pass)]
        return marks[0].elapsed_time(marks[n_pass])

    for _ in range(args.warmup):
        pipeline.run_pass(kv, inputs, windows, select=select)
    kv.scalekv_sync()
    # A pass is the same sequence of launches every time (the schedule, the budgets and the buffers are
    # fixed), so it is captured once into a CUDA graph - stream_main plus the side stream that compress
    # forks to - and the timed region replays it: the GPU is then never waiting for the host.
    graph, graph_note = None, "off (--no-graph)"
    launches0 = kv.scalekv_launch_count()
    if not args.no_graph:
        try:
            graph = torch.cuda.CUDAGraph()
            torch.cuda.synchronize()
            # thread_local: other threads (a process group's watchdog under torchrun) may call CUDA meanwhile
            with torch.cuda.graph(graph, stream=kv.stream_main, capture_error_mode="thread_local"):
                pipeline.run_pass(kv, inputs, windows, select=select)
                kv.scalekv_join()
            with torch.cuda.stream(kv.stream_main):
                graph.replay()                         # one untimed replay
            kv.scalekv_sync()
            graph_note = "on"
        except Exception as exc:                       # a capture that did not go through: start over, call by call
            graph, graph_note = None, f"off (capture failed: {type(exc).__name__})"
            torch.cuda.synchronize()
            kv.close()
            kv = make_kv()
            pipeline.run_pass(kv, inputs, windows, select=select)
            kv.scalekv_sync()
            launches0 = kv.scalekv_launch_count()
    launches_per_pass = kv.scalekv_launch_count() - launches0
    launches0 = kv.scalekv_launch_count()
    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    ms = timed_passes(args.steps, graph)
    barrier()
    launches = launches_per_pass * args.steps if graph is not None else kv.scalekv_launch_count() - launches0
    pass_spread = {"min": min(pass_marks), "median": statistics.median(pass_marks), "max": max(pass_marks)}
    # the same region again with CUDA events around every launch, each on the stream it is launched on:
    # the attend durations measured here (compress overlapping on the side stream, as in the timed
    # passes) feed the roofline object; the events themselves cost a few per cent, so `value` comes
    # from the passes above
    kv.scalekv_profile_enable(1)
    ms_events = timed_passes(args.steps)
    prof_timed = kv.scalekv_profile_read()
    clocks = sampler.stop()
    ms = max_over_ranks(ms, world, "cuda")
    value = job_throughput(wl.n_scales, args.steps, world, ms)

    # per-scale-step latency: events on stream_main at the scale boundaries of the same passes (a scale-step's
    # compress of its last layers may still run on the side stream when the next scale-step starts)
    kv.scalekv_profile_enable(0)
    per_pass = []
    per_scale_mode = "call by call (eager): at the small scales the host's launch rate, not the GPU, sets the time"
    scale_graphs = None
    if graph is not None:
        # one CUDA graph per scale-step, captured while a pass runs (capture, then replay to execute it), each
        # ending with a join of the side stream: what the events then bracket is GPU time
        try:
            kv.scalekv_reset()
            kv.scalekv_sync()
            scale_graphs = []
            for k in range(wl.n_scales):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=kv.stream_main, capture_error_mode="thread_local"):
                    pipeline.scale_step(kv, inputs, windows, k, select=select)
                    kv.scalekv_join()
                with torch.cuda.stream(kv.stream_main):
                    g.replay()
                kv.scalekv_sync()
                scale_graphs.append(g)
            per_scale_mode = "one CUDA graph per scale-step, the side stream joined at every scale boundary"
        except Exception:
            scale_graphs = None
            torch.cuda.synchronize()
            kv.close()
            kv = make_kv()
    for _ in range(args.steps):
        if scale_graphs is None:
            marks = []
            pipeline.run_pass(kv, inputs, windows, marks=marks, select=select)
        else:
            marks = [torch.cuda.Event(enable_timing=True) for _ in range(wl.n_scales + 2)]
            with torch.cuda.stream(kv.stream_main):
                marks[0].record()
            kv.scalekv_reset()
            with torch.cuda.stream(kv.stream_main):
                marks[1].record()
                for k in range(wl.n_scales):
                    scale_graphs[k].replay()
                    marks[k + 2].record()
        kv.scalekv_sync()
        per_pass.append([marks[i].elapsed_time(marks[i + 1]) for i in range(len(marks) - 1)])
    scale_graphs = None
    cols = list(zip(*per_pass))
    scale_flop = work["per_scale_flop"]
    per_scale = {"reset_ms_median": statistics.median(cols[0]),
                 "scale_steps": [{"scale": k + 1, "n_k": wl.n_tokens[k], "ms_median": statistics.median(cols[k + 1]),
                                  "ms_min": min(cols[k + 1]),
                                  "attend_TFLOPps": scale_flop[k] / (statistics.median(cols[k + 1]) / 1e3) / 1e12}
                                 for k in range(wl.n_scales)],
                 "mode": per_scale_mode,
                 "note": "CUDA events on stream_main at scale boundaries; one scale-step = append + attend + compress of "
                         "every layer at that scale; attend_TFLOPps = the scale's attention flop over the step's time"}

    # the same passes once more with compress serialised onto stream_main: every kernel timed alone
    kv.scalekv_profile_enable(2)
    for _ in range(args.steps):
        pipeline.run_pass(kv, inputs, windows, select=select)
    prof_alone = kv.scalekv_profile_read()
    kv.scalekv_profile_enable(0)
    att_ms, att_n = prof_timed["attend"]
    att_tflops = work["attend_flop"] * args.steps / (att_ms / 1000.0) / 1e12 if att_ms > 0 else 0.0
    peak_tf = peaks["bf16_sustained"] if wl.dtype == "bf16" else None
    kernels = {}
    for name, key in (("append", "append_bytes"), ("score", "score_bytes"), ("select", "select_bytes"),
                      ("compact", "compact_bytes"), ("compress", "compress_bytes")):
        kms, kn = prof_alone[name]
        if kn == 0:
            continue
        gbs = work[key] * args.steps / (kms / 1000.0) / 1e9 if kms > 0 else 0.0
        kernels[name] = {"ms_per_pass": kms / args.steps, "launches_per_pass": kn / args.steps, "algorithmic_GBps": gbs,
                         "frac_of_hbm_peak": gbs / peaks["hbm_gbs"], "timed": "alone (compress serialised onto stream_main)"}
    al_ms, al_n = prof_alone["attend"]
    kernels["attend"] = {"ms_per_pass": att_ms / args.steps, "launches_per_pass": att_n / args.steps, "TFLOPps": att_tflops,
                         "ms_per_pass_alone": al_ms / args.steps,
                         "TFLOPps_alone": work["attend_flop"] * args.steps / (al_ms / 1000.0) / 1e12 if al_ms > 0 else 0.0,
                         "algorithmic_GB_per_pass": work["attend_min_bytes"] / 1e9}
    roofline = {"bound": "tensor", "kernel": "attend_tc_kernel", "achieved": att_tflops, "peak": peak_tf, "unit": "TFLOP/s",
                "frac": (att_tflops / peak_tf) if peak_tf else None,
                "traffic": (ATTEND_TRAFFIC_RATIO * work["attend_min_bytes"] / max(work["attend_launches"], 1)
                            if ATTEND_TRAFFIC_RATIO and wl.dtype == "bf16" else None),
                "traffic_unit": "bytes per launch (average launch)",
                "traffic_source": ATTEND_TRAFFIC_SOURCE if (ATTEND_TRAFFIC_RATIO and wl.dtype == "bf16") else None,
                "peak_source": f"{peaks['source']} bf16 sustained (kernel timed inside a long step)",
                "avg_launch_ms": att_ms / max(att_n, 1),
                "flop_per_launch_avg": work["attend_flop"] / max(work["attend_launches"], 1),
                "ms_per_pass_with_events": ms_events / args.steps}
    hbm_bytes = work["compress_bytes"]
    ser_ms = (work["attend_flop"] / (peaks["bf16_sustained"] * 1e12) + hbm_bytes / (peaks["hbm_gbs"] * 1e9)) * 1e3
    pass_ms = ms / args.steps
    roofline["pass_roofline_ms_serial"] = ser_ms
    roofline["pass_frac_serial"] = ser_ms / pass_ms

    # end to end from pinned host buffers through scalekv_step_host
    e2e = None
    if not args.no_e2e:
        n_max = max(wl.n_tokens)
        dt = synth.torch_dtype(wl.dtype)
        # pinned host copies of the inputs of E2E_HOST_LAYERS layers (a full set would pin 33 GB); layer l reads set
        # l mod E2E_HOST_LAYERS, so consecutive steps copy from different host pages
        host = {}
        n_host = min(E2E_HOST_LAYERS, wl.n_layers)
        for r in range(n_host):
            for k in range(wl.n_scales):
                host[(r, k)] = tuple(t.cpu().pin_memory() for t in inputs.data[(r, k)])
        Oh = [torch.empty(wl.batch, wl.n_heads, n_max, wl.head_dim, dtype=dt).pin_memory() for _ in range(2)]
        staging = torch.empty(8 * wl.batch * wl.n_heads * n_max * wl.head_dim, dtype=dt, device="cuda")
        torch.cuda.synchronize()

        def e2e_pass():
            kv.scalekv_reset()
            for k in range(wl.n_scales):
                nk = wl.n_tokens[k]
                last = k + 1 == wl.n_scales
                for l in range(wl.n_layers):
                    Qh, Kh, Vh = host[(l % n_host, k)]
                    kv.scalekv_step_host(l, k, Qh, Kh, Vh, Oh[(l + k) & 1], staging, window_pos=None if last else windows[k])
            kv.scalekv_sync()                  # every output has reached the host
        e2e_steps = max(1, min(args.steps, 3))
        e2e_pass()
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            e2e_pass()
        barrier()
        e2e_s = time.perf_counter() - t0
        e2e_s = max_over_ranks(e2e_s, world, "cuda")
        esz = 2 if wl.dtype == "bf16" else 4
        tok_bytes = sum(wl.n_tokens) * wl.batch * wl.n_heads * wl.head_dim * esz * wl.n_layers
        e2e = {"value": wl.n_scales * e2e_steps * world / e2e_s, "unit": UNIT, "h2d_bytes_per_step": 3 * tok_bytes,
               "d2h_bytes_per_step": tok_bytes, "steps": e2e_steps,
               "note": "scalekv_step_host per layer and scale: pinned host Q/K/V -> device, append + attend + compress, O -> "
                       "pinned host; the copies of neighbouring steps overlap the kernels; one sync per pass; layer l reads "
                       f"the pinned host tensors of layer l mod {n_host}"}
        del staging

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, note = oracle_rate(wl, budgets, windows, args.cpu_sample_slices)
        cpu = {"value": v, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle", "sample": note}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": pass_ms, "ms_per_step_spread": pass_spread, "passes_per_sec": args.steps * world / (ms / 1000.0), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
            "config": {"workload": wl.name, "layers": wl.n_layers, "batch": wl.batch, "heads": wl.n_heads,
                       "head_dim": wl.head_dim, "scales": wl.n_scales, "tokens": sum(wl.n_tokens),
                       "budget": role_note + (f"; overall {args.overall_pct} %" if args.overall_pct > 0 else ""),
                       "policy": args.policy,
                       "window": wl.window, "parallelism": f"replica x{world} (batch-sharded, no collective)",
                       "l2_policy": f"inputs larger than L2: {inputs.bytes() / 1e9:.1f} GB of Q/K/V per pass",
                       "side_stream": not args.no_side_stream, "cuda_graph": graph_note, "calibration_s": round(calib_s, 1),
                       "attend_kernel": "tcgen05" if (wl.dtype == "bf16" and wl.head_dim == 128) else "fp32 FMA"},
            "roofline": roofline, "kernels": kernels, "per_scale": per_scale, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches,
            "clocks": clocks, "work_per_pass": {k: v for k, v in work.items() if k != "per_scale_flop"},
        }
        print(json.dumps(line))
    kv.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_scalekv(args)


if __name__ == "__main__":
    main()
