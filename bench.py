#!/usr/bin/env python
"""Benchmark of the PruneTrain hot path on B200.

One step = one pass of the whole hot path on the pruned ResNet-50 workload (batch 64, 224x224, 53 conv layers,
per-layer keep ratios drawn from a seed to give ~60 % of dense FLOPs):
  zero-group detection + keep-set scan + channel-union compaction of the dense-shaped model  ->
  conv fwd of every layer, conv dgrad + wgrad in reverse order                                ->
  fused group-lasso momentum-SGD step over all conv weights.
BN, ReLU, pooling, residual adds and the classifier are not on the path and not in the step.

Prints ONE JSON line (rank 0). `--impl reference` times the CPU oracle instead (a deliberately plain program).
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

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

PROFILE_LAUNCH_LIST = os.path.join(ROOT, "profiles", "step_launch_list_resnet50_keep060_b64.txt")


def ncu_pass_traffic(kind):
    """dram__bytes_read.sum + dram__bytes_write.sum over the launches of one conv pass of the default workload, as the tracked
    ncu summary records them (a line 'pass_dram_bytes fwd=... dgrad=... wgrad=...'); None if the summary has no such line.
    A captured launch's writes mostly retire from the 126 MB L2 after it has ended, so the figure is dominated by reads."""
    try:
        for line in open(PROFILE_LAUNCH_LIST):
            if line.startswith("# pass_dram_bytes"):
                kv = dict(t.split("=") for t in line.split()[2:])
                return float(kv[kind])
    except Exception:
        pass
    return None


METRIC = "pruned ResNet-50 train-step conv TFLOP/s (useful FLOPs / whole step)"
UNIT = "TFLOP/s"


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d["bf16_tflops_sustained"], "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "50", "-i", str(index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons, pw = [], [], set(), []
        for line in self.f.read().splitlines():
            c = [t.strip() for t in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1])); mx.append(float(c[2])); pw.append(float(c[3]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        self.f.close()
        os.unlink(self.f.name)
        if sm:
            out = {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                   "samples": len(sm), "power_w_max": max(pw)}
        return out


def workload(args):
    from paper_1901_09290_b200 import workloads as W
    seed = W.BASE_SEED + 4
    if args.net != "resnet50":
        # the paper's CIFAR models (Tab. 1) as extra workloads; the default and the headline stay the ImageNet ResNet-50
        net = W.resnet32() if args.net == "resnet32" else W.vgg(int(args.net[3:]))
        if args.net == "resnet32" and args.keep is None:
            # the CIFAR-shaped stack as its configuration states it: keep ratios drawn per space from 0.4-0.9 (the seed of
            # the parity tests of that configuration), channel union at the residual adds
            seed = W.BASE_SEED + 2
            counts = W.random_keep(net, seed)
            name = "resnet32-32x32-keep-drawn-0.4-0.9"
        else:
            keep = 0.6 if args.keep is None else args.keep
            counts = W.uniform_keep(net, keep)
            name = f"{args.net}-32x32-uniform-keep-{keep:g}"
    elif args.keep is not None:
        net = W.resnet50()
        counts = W.uniform_keep(net, args.keep)
        name = f"resnet50-uniform-keep-{args.keep:g}"
    else:
        net = W.resnet50()
        counts = W.staged_keep_to_flops(net, seed, 0.60)
        name = "resnet50-224-53conv-keep-drawn-to-0.60-flops"
    kept = W.choose_kept(net, counts, seed)
    return net, counts, kept, seed, name


# ------------------------------------------------------------------------------------------ CPU oracle legs
def oracle_step_sample(net_p, N_s, layer_ids, seed):
    """One bounded sample of the step on the host cores with the oracle as it stands: fwd + dgrad + wgrad of the
    given layers at batch N_s, and the lasso step, detection of those layers. Returns (seconds, useful conv FLOPs)."""
    import numpy as np
    import oracle
    from paper_1901_09290_b200 import workloads as W
    flops = 0
    data = []
    for li in layer_ids:
        l = net_p.layers[li]
        x = (W.gen_image if li == 0 else W.gen_act)(N_s, l.H, l.H, l.C, seed + li).numpy()
        w = W.bf16_round(W.gen_weight(l.K, l.R, l.R, l.C, seed + 1000 + li)).numpy()
        dy = W.gen_dy(N_s, l.P, l.P, l.K, seed + 2000 + li).numpy()
        v = W.gen_small(w.shape, seed + 3000 + li).numpy()
        data.append((l, li, x, w, dy, v))
    t0 = time.perf_counter()
    for l, li, x, w, dy, v in data:
        oracle.conv_fwd(x, w, l.stride, l.pad)
        fl = 2 * N_s * l.P * l.P * l.K * l.C * l.R * l.R
        flops += 2 * fl
        if li > 0:
            oracle.conv_dgrad(dy, w, l.H, l.H, l.stride, l.pad)
            flops += fl
        dw = oracle.conv_wgrad(x, dy, l.R, l.R, l.stride, l.pad)
        oracle.lasso_sgd(w, dw.astype(np.float32), v, 1e-4, 0.1, 0.9, reg_in=(li > 0))
        oracle.find_zero_groups(w)
    return time.perf_counter() - t0, flops


CPU_SAMPLE_BATCH = 2          # both arms time the oracle on the same bounded sample: every layer of the workload at this batch


def cpu_sample(net_p):
    ids = list(range(len(net_p.layers)))
    return ids, CPU_SAMPLE_BATCH, (f"batch {CPU_SAMPLE_BATCH}, all {len(ids)} layers of the workload: fwd+dgrad+wgrad+lasso+detection "
                                   "per layer, as the oracle stands")


def run_reference(args):
    """--impl reference: the oracle on the host cores, same metric and config, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_1901_09290_b200 import workloads as W
    net, counts, kept, seed, name = workload(args)
    net_p = W.with_sizes(net, counts)
    ids, nb, sample = cpu_sample(net_p)
    for _ in range(args.warmup):
        oracle_step_sample(net_p, nb, ids, seed)
    T, F = 0.0, 0
    for _ in range(args.steps):
        t, f = oracle_step_sample(net_p, nb, ids, seed)
        T += t
        F += f
    val = F / T / 1e12
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": T / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": name, "batch": args.batch, "image": net.layers[0].H, "kept_params": sum(l.K * l.C * l.R * l.R for l in net_p.layers)},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------------------------------ multi-rank aggregation
def max_over_ranks(ms: float, world: int, device="cuda") -> float:
    """Step time of the job = the slowest rank's device time."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(flops_per_rank: float, world: int, ms_total: float, steps: int) -> float:
    """Whole-job TFLOP/s: every rank processes its own batch (weak scaling), the job takes the slowest rank's time."""
    return world * flops_per_rank / (ms_total / steps * 1e-3) / 1e12


def chained_step_times(ctx, ts, args, seed):
    """The same pruned network as ONE chained training step (convolution -> batch norm -> ReLU, max pooling after the stem,
    residual adds, the whole backward pass, the lasso step), replayed from a CUDA graph: with the normalisation statistics
    taken in the convolution epilogues and with the stand-alone normalisation (weight gradients and projection shortcuts on
    side streams), and once more with everything on one stream. Not the headline metric (whose workload has no
    normalisation layers in it); reported beside it."""
    import torch
    from paper_1901_09290_b200 import harness
    res = {}
    for fused, ws_n, key in ((True, 2, "fused_statistics"), (False, 2, "stand_alone_normalisation"), (True, 0, "fused_statistics_one_stream")):
        cs = harness.ChainedStep(ctx, ts.net, args.batch, seed + 5, fused_stats=fused, algo=args.algo, wgrad_streams=ws_n)
        cs.step()
        torch.cuda.synchronize()
        l0 = ctx.launch_count()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            cs.step()
        launches = ctx.launch_count() - l0
        for _ in range(3):
            g.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n = 10
        a.record()
        for _ in range(n):
            g.replay()
        b.record()
        torch.cuda.synchronize()
        ctx.poll()
        ms = a.elapsed_time(b) / n
        res[key] = {
            "ms_per_step": ms, "launches": launches, "conv_tflops_over_step": cs.conv_flops() / (ms * 1e-3) / 1e12}
        del cs, g
        torch.cuda.empty_cache()
    ctx.set_wgrad_cta_limit(ts.wgrad_ctas)
    res["note"] = ("53 convolutions each followed by batch norm (training statistics) + ReLU, 3x3/2 max pooling after the stem, 16 "
                   "residual adds, backward to every weight / gamma / beta gradient, lasso step; CUDA graph replay; the weight gradients on two side streams beside the backward chain (one stream in the third entry)")
    return res


# ------------------------------------------------------------------------------------------ GPU leg
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_1901_09290_b200 import binding as B
    from paper_1901_09290_b200 import harness
    from paper_1901_09290_b200 import workloads as W

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but WORLD_SIZE is {world}")
    if local >= torch.cuda.device_count():
        raise SystemExit(f"bench.py: rank {rank} needs GPU {local}, the machine has {torch.cuda.device_count()}")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    pk = peaks()
    ctx = B.Context(local)
    net, counts, kept, seed, name = workload(args)
    # N > 1 default: independent replicas (no data-path collective). --data-parallel: every rank holds the same model (same
    # seed; the synthetic batch is then the same too, which the timing does not depend on) and the weight gradients are
    # averaged by one NCCL all-reduce before the update.
    dp = world > 1 and args.data_parallel
    ts = harness.TrainStep(ctx, net, counts, kept, args.batch, seed + (0 if dp else 17 * rank), algo=args.algo, host_inputs=True,
                           world=world if dp else 1, wgrad_ctas=args.wgrad_ctas, wgrad_streams=args.wgrad_streams)
    flops = ts.conv_flops()
    tot_flops = sum(flops.values())
    stream = torch.cuda.current_stream()

    MIN_TIMED_S = 0.5

    def timed(fn, steps):
        """Device time of `steps` steps (max over ranks). The timed region is kept at or above half a second: the K requested
        steps are repeated back to back r times inside one pair of events (r chosen from a first pass of K steps) and the
        total is divided by r, so that a short K still gives a sustained-clock figure. Returns (ms for K steps, r)."""
        def run(n):
            barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(n):
                fn()
            e1.record(stream)
            barrier()
            return max_over_ranks(e0.elapsed_time(e1), world)
        first = run(steps)
        r = max(1, int(MIN_TIMED_S * 1e3 / max(first, 1e-3)) + 1)
        if r == 1:
            return first, 1
        return run(steps * r) / r, r

    if args.profile_steps and args.profile_chained:
        # the same for the chained step (convolutions + batch norm + pooling + residual adds, forward and backward)
        from paper_1901_09290_b200 import harness
        cs = harness.ChainedStep(ctx, ts.net, args.batch, seed + 5, fused_stats=True, algo=args.algo)
        for _ in range(1 + args.profile_steps):
            cs.step()
            torch.cuda.synchronize()
        ctx.poll()
        if rank == 0:
            print(json.dumps({"profile_steps": args.profile_steps, "step": "chained", "workload": name}))
        return
    if args.profile_steps:
        # a short run for profilers: one warm-up step, then the requested steps, nothing else
        ts.step()
        torch.cuda.synchronize()
        for _ in range(args.profile_steps):
            ts.step()
        torch.cuda.synchronize()
        ctx.poll()
        if rank == 0:
            print(json.dumps({"profile_steps": args.profile_steps, "launches_per_step": None, "workload": name}))
        return
    ts.step()                                   # one eager step sets up tables and kernel attributes
    torch.cuda.synchronize()
    if not args.no_graph:
        ts.build_graph(two_streams=not args.one_stream)
    for _ in range(max(args.warmup, 3)):
        ts.step()
    barrier()
    ctx.poll()
    l0 = ctx.launch_count()
    sampler = ClockSampler(local) if rank == 0 else None
    ms, reps_timed = timed(ts.step, args.steps)
    n_timed = args.steps * (reps_timed + (1 if reps_timed > 1 else 0))      # steps run inside the timed regions (first pass + repeats)
    per_step_launches = (ctx.launch_count() - l0) / max(1, n_timed) + (ts.graph_launches if getattr(ts, "graph", None) is not None else 0)
    launches = int(round(per_step_launches * args.steps))
    # end-to-end: image batch from pinned host memory, regulariser value and new sizes read back, every step
    for _ in range(2):
        ts.step_e2e()
    ms_e2e, _ = timed(ts.step_e2e, args.steps)
    clocks = sampler.stop() if sampler else None
    ctx.poll()

    # per-phase and per-layer device times (CUDA events around each ABI call, same stream), for the roofline
    nL = len(ts.net.layers)
    reps = max(2, min(5, args.steps))
    acc = {"fwd": [0.0] * nL, "dgrad": [0.0] * nL, "wgrad": [0.0] * nL}
    phase = {}

    def ev_time(fn):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        fn()
        b.record(stream)
        return a, b

    # Conv passes: every launch of a pass kind is captured into one CUDA graph with an (external) event between
    # launches, so the per-layer times are device times with no host launch gaps, and the layers' buffers (6 GB in
    # total) keep the L2 cold between launches. Falls back to eager event timing if external events are unavailable.
    def time_pass_in_graph(kind):
        calls = []
        for li in (range(nL) if kind == "fwd" else range(nL - 1, -1, -1)):
            if kind == "dgrad" and li == 0:
                continue
            fn = {"fwd": ts.conv_fwd, "dgrad": ts.conv_dgrad, "wgrad": ts.conv_wgrad}[kind]
            calls.append((li, fn))
        try:
            evs = [torch.cuda.Event(enable_timing=True, external=True) for _ in range(len(calls) + 1)]
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                cs = torch.cuda.current_stream()
                evs[0].record(cs)
                for i, (li, fn) in enumerate(calls):
                    fn(li)
                    evs[i + 1].record(cs)
            g.replay()
            torch.cuda.synchronize()
            for _ in range(reps):
                g.replay()
                torch.cuda.synchronize()
                for i, (li, fn) in enumerate(calls):
                    acc[kind][li] += evs[i].elapsed_time(evs[i + 1]) / reps
            return "graph"
        except Exception:
            for li in range(nL):
                acc[kind][li] = 0.0
            for _ in range(reps):
                pend = [(li, ev_time(lambda: fn(li))) for li, fn in calls]
                torch.cuda.synchronize()
                for li, (a, b) in pend:
                    acc[kind][li] += a.elapsed_time(b) / reps
            return "eager"

    timing_mode = [time_pass_in_graph(k) for k in ("fwd", "dgrad", "wgrad")]
    # Each pass alone with the stream assignment it has inside the step (weight gradients of different layers side by
    # side on their streams, shortcuts beside their blocks): the device time of the pass as the step launches it.
    sched = {}
    if getattr(ts, "graph", None) is not None and not args.one_stream:
        for kind in ("fwd", "dgrad", "wgrad"):
            gk = ts.capture_pass(kind)
            gk.replay()
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(reps):
                gk.replay()
            b.record(stream)
            torch.cuda.synchronize()
            sched[kind] = a.elapsed_time(b) / reps
    # Update and reconfiguration phases, each alone: replayed from a CUDA graph where the call has no host synchronisation
    # (as the step launches it), with the L2 flushed before every repetition (in the step the convolutions in between do that)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    def time_alone(fn, graph=True):
        fn()
        torch.cuda.synchronize()
        g = None
        if graph:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                fn()
        tot = 0.0
        for _ in range(reps):
            flush.fill_(1)
            a, b = ev_time(g.replay if g is not None else fn)
            torch.cuda.synchronize()
            tot += a.elapsed_time(b) / reps
        return tot

    md = ts.md
    v_saved = [v.clone() for v in md.v]
    phase["reconfigure"] = time_alone(ts.reconfigure, graph=False)                      # contains the plan's host synchronisation
    phase["detect"] = time_alone(lambda: B.pt_find_zero_groups(ctx, md.arr, 1e-4, False, md.ws))
    phase["gather"] = time_alone(lambda: B.pt_reconfigure(ctx, md.graph(), ts.new2old, ts.mp.graph()))
    phase["plan_incl_host_sync"] = time_alone(lambda: B.pt_reconfigure_plan(ctx, md.graph(), ts.new2old), graph=False)
    phase["lasso"] = time_alone(ts.lasso)
    ts.lasso_norms()
    phase["lasso_carried"] = time_alone(ts.lasso_carried)
    phase["lasso_dense_model"] = time_alone(lambda: B.pt_group_lasso_sgd_step(ctx, md.arr, 1e-4, 0.0, 0.9, 0.0, md.reg, md.ws))
    B.pt_group_lasso_norms(ctx, md.arr, md.reg, md.ws)
    phase["lasso_carried_dense_model"] = time_alone(lambda: B.pt_group_lasso_sgd_step_carried(ctx, md.arr, 1e-4, 0.0, 0.9, 0.0, md.reg, md.ws))
    for w, sv in zip(md.v, v_saved):
        w.copy_(sv)
    del flush
    ts.reconfigure()
    ctx.poll()

    which_id = {"fwd": 0, "dgrad": 1, "wgrad": 2}
    per_layer = []
    t_roof_sum, t_meas_sum = 0.0, 0.0
    tc_peak = pk["bf16_tflops_sustained"] * 1e12
    bw_peak = pk["hbm_gbs"] * 1e9
    for kind in ("fwd", "dgrad", "wgrad"):
        for li, l in enumerate(ts.net.layers):
            if kind == "dgrad" and li == 0:
                continue
            fl = 2 * args.batch * l.P * l.P * l.K * l.C * l.R * l.R
            by = ts.layer_bytes(li, which_id[kind])
            t = acc[kind][li] * 1e-3
            roof = max(fl / tc_peak, by / bw_peak)
            t_roof_sum += roof
            t_meas_sum += t
            per_layer.append({"layer": l.name, "pass": kind, "C": l.C, "K": l.K, "R": l.R, "stride": l.stride, "H": l.H,
                              "us": t * 1e6, "tflops": fl / t / 1e12, "gbs": by / t / 1e9,
                              "bound": "tensor" if fl / tc_peak > by / bw_peak else "hbm", "roofline_frac": roof / t})
    # the layers above the ridge (tensor-bound by their algorithmic FLOPs and bytes), fwd and dgrad: the subset the tensor-peak
    # target is meant for. Weight gradients are left out of it because their serial times are taken at a third of the SMs.
    sub = [r for r in per_layer if r["bound"] == "tensor" and r["pass"] != "wgrad"]
    sub_fl = sum(r["tflops"] * r["us"] for r in sub)           # TFLOP/s x us = MFLOP
    sub_us = sum(r["us"] for r in sub)
    tensor_subset = {"launches": len(sub), "tflops": sub_fl / sub_us if sub_us else None,
                     "pct_of_measured_sustained": 100 * sub_fl / sub_us * 1e12 / tc_peak if sub_us else None,
                     "best_layer_pct": max((100 * r["tflops"] * 1e12 / tc_peak for r in sub), default=None),
                     "timing": "fwd and dgrad launches whose FLOPs / tensor peak exceed their bytes / HBM rate, one after the other"}
    floor_ms = {k: 1e3 * sum(max(2 * args.batch * l.P * l.P * l.K * l.C * l.R * l.R / tc_peak, ts.layer_bytes(li, which_id[k]) / bw_peak)
                             for li, l in enumerate(ts.net.layers) if not (k == "dgrad" and li == 0)) for k in which_id}
    serial_ms = {k: sum(v) for k, v in acc.items()}           # launches of a pass one after the other
    conv_ms = sched if sched else serial_ms                     # passes as the step schedules them
    conv_total_ms = sum(conv_ms.values())
    dom = max(conv_ms, key=conv_ms.get)
    dom_flops = flops[dom]
    dom_t = conv_ms[dom] * 1e-3
    n_dom = nL - (1 if dom == "dgrad" else 0)
    dom_bytes = sum(ts.layer_bytes(li, which_id[dom]) for li in range(nL) if not (dom == "dgrad" and li == 0))
    value = whole_job_value(tot_flops, world, ms, args.steps)
    e2e_val = whole_job_value(tot_flops, world, ms_e2e, args.steps)
    h2d, d2h = ts.e2e_bytes()
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms / args.steps, "timed_region": {"steps_per_pass": args.steps, "passes_averaged": reps_timed,
                                                         "seconds": ms * reps_timed * 1e-3}, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16",
        "arithmetic": "bf16 operands, f32 accumulate (convs); f32 (lasso/SGD); u8/i32 (detection, compaction)",
        "data": "synthetic",
        "config": {"workload": name, "batch_per_gpu": args.batch, "image": net.layers[0].H, "conv_layers": nL,
                   "kept_params": ts.mp.n_params(), "dense_params": ts.md.n_params(),
                   "useful_conv_flops_per_step": tot_flops, "l2": "inputs larger than L2 (per-layer activations 20-400 MB, ~6 GB per step)",
                   "parallelism": ("data parallel: one NCCL all-reduce (mean) of the weight gradients per step" if dp else
                                   "independent data-parallel replicas, no collective") if world > 1 else "1 GPU",
                   "algo": args.algo,
                   "launch": "eager" if args.no_graph else ("CUDA graph replay after the reconfiguration's host sync; "
                                                            + ("1 stream" if args.one_stream else f"streams along the network's data dependencies: dgrad chain, projection shortcuts beside their blocks, wgrads round-robin on {ts.wgrad_streams} streams at <= {ts.wgrad_ctas} CTAs each" + (f" nominal; per-launch limits {min(ts.wgrad_limit.values())}..{max(ts.wgrad_limit.values())} CTAs from a work-per-CTA dynamic programme, every three consecutive launches within the SM count, the last three sharing the SMs as {[ts.wgrad_limit[k] for k in (2, 1, 0)]}" if ts.wgrad_limit else "")))},
        "e2e": {"value": e2e_val, "unit": UNIT, "ms_per_step": ms_e2e / args.steps, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "pipeline": "one pinned-host image copy per step on a copy stream into the other of two stem-input buffers (one CUDA graph per buffer), overlapping the current step's kernels"},
        "gpu_launches": launches,
        "clocks": clocks,
        "phases_ms": {"conv_fwd": conv_ms["fwd"], "conv_dgrad": conv_ms["dgrad"], "conv_wgrad": conv_ms["wgrad"],
                      "lasso_sgd_pruned": phase["lasso"], "detect_plan_compact": phase["reconfigure"],
                      "lasso_sgd_dense_model": phase["lasso_dense_model"], "lasso_sgd_carried_pruned": phase["lasso_carried"],
                      "note": "conv passes: each pass alone as the step schedules it (wgrads of different layers side by side)"
                              if sched else "conv passes: sum of the launches one after the other"},
        "phases_serial_ms": {"conv_fwd": serial_ms["fwd"], "conv_dgrad": serial_ms["dgrad"], "conv_wgrad": serial_ms["wgrad"]},
        "conv_tflops": tot_flops / (conv_total_ms * 1e-3) / 1e12,
        "conv_pct_of_bf16_peak": {"measured_sustained": 100 * tot_flops / (conv_total_ms * 1e-3) / tc_peak,
                                  "nominal_2250": 100 * tot_flops / (conv_total_ms * 1e-3) / 2.25e15},
        "conv_mixed_roofline_frac": t_roof_sum / t_meas_sum,
        "conv_tensor_bound_subset": tensor_subset,
        "per_layer_timing": timing_mode[0],
        "lasso_gbs": {"pruned_model": ts.lasso_bytes(ts.mp) / (phase["lasso"] * 1e-3) / 1e9,
                      "dense_model": ts.lasso_bytes(ts.md) / (phase["lasso_dense_model"] * 1e-3) / 1e9,
                      "bytes_per_param": 26,
                      "carried_pruned_model": 22 * ts.mp.n_params() / (phase["lasso_carried"] * 1e-3) / 1e9,
                      "carried_dense_model": 22 * ts.md.n_params() / (phase["lasso_carried_dense_model"] * 1e-3) / 1e9,
                      "carried_bytes_per_param": 22, "peak": pk["hbm_gbs"], "peak_source": pk["source"]},
        "reconf_gbs": ts.reconf_bytes() / (phase["reconfigure"] * 1e-3) / 1e9,
        "reconf": {"whole_call_incl_host_sync_ms": phase["reconfigure"], "detect_ms": phase["detect"], "gather_ms": phase["gather"],
                   "plan_incl_host_sync_ms": phase["plan_incl_host_sync"],
                   "detect_gbs": 4 * ts.md.n_params() / (phase["detect"] * 1e-3) / 1e9,
                   "gather_gbs": 18 * ts.mp.n_params() / (phase["gather"] * 1e-3) / 1e9,
                   "kernels_gbs": ts.reconf_bytes() / ((phase["detect"] + phase["gather"]) * 1e-3) / 1e9},
        "roofline": {"kernel": f"conv_{dom} (all {n_dom} launches of a step, as the step schedules them)",
                     # the pass's own FLOPs and bytes decide which roof bounds it
                     "bound": "tensor" if dom_flops / tc_peak > dom_bytes / bw_peak else "hbm",
                     "achieved": (dom_flops / dom_t / 1e12) if dom_flops / tc_peak > dom_bytes / bw_peak else (dom_bytes / dom_t / 1e9),
                     "peak": pk["bf16_tflops_sustained"] if dom_flops / tc_peak > dom_bytes / bw_peak else pk["hbm_gbs"],
                     "unit": "TFLOP/s" if dom_flops / tc_peak > dom_bytes / bw_peak else "GB/s",
                     # sum over the pass's layers of max(FLOPs / tensor peak, bytes / HBM rate), over the pass's scheduled time
                     "frac": floor_ms[dom] / conv_ms[dom],
                     "frac_all_passes": sum(floor_ms.values()) / conv_total_ms,
                     "tensor_only": {"achieved_tflops": dom_flops / dom_t / 1e12, "frac_of_sustained_bf16": dom_flops / dom_t / tc_peak},
                     "hbm_only": {"achieved_gbs": dom_bytes / dom_t / 1e9, "frac_of_copy_rate": dom_bytes / dom_t / bw_peak},
                     "traffic": ncu_pass_traffic(dom) if (args.net == "resnet50" and args.keep is None and args.batch == 64 and args.algo in (0, 2)) else None,
                     "traffic_note": "dram bytes of the pass's launches in the tracked ncu summary (profiles/); mostly reads: a launch's "
                                     "writes retire from L2 after it has ended",
                     "algorithmic_bytes": dom_bytes,
                     "peak_source": pk["source"]},
    }
    if world == 1 and not args.no_chained and args.net == "resnet50":
        out["chained_step"] = chained_step_times(ctx, ts, args, seed)
    if rank == 0:
        if args.per_layer:
            os.makedirs(os.path.dirname(os.path.abspath(args.per_layer)), exist_ok=True)
            json.dump(per_layer, open(args.per_layer, "w"), indent=0)
        if world == 1 and not args.no_cpu_baseline:
            import oracle
            net_p = ts.net
            ids, nb, sample = cpu_sample(net_p)
            oracle_step_sample(net_p, nb, ids[:4], seed)            # warm the thread pool
            t, f, n_rep = 0.0, 0, 0
            while t < 10.0 and n_rep < 8:                            # about 10-20 s of CPU work
                t1, f1 = oracle_step_sample(net_p, nb, ids, seed)
                t += t1; f += f1; n_rep += 1
            out["cpu_baseline"] = {"value": f / t / 1e12, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                                   "sample": f"{sample}; {n_rep} repetitions, {t:.1f} s"}
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--batch", type=int, default=64)
    ap.add_argument("--data-parallel", action="store_true",
                    help="N > 1: average the weight gradients over the ranks with one NCCL all-reduce per step (default: replicas)")
    ap.add_argument("--keep", type=float, default=None, help="uniform keep ratio instead of the seeded per-space draw")
    ap.add_argument("--net", default="resnet50", choices=["resnet50", "resnet32", "vgg11", "vgg13", "vgg16"],
                    help="shape table; resnet50 (224x224) is the headline workload, the others are the paper's 32x32 CIFAR models")
    ap.add_argument("--wgrad-ctas", type=int, default=49, help="CTA limit of a weight-gradient launch")
    ap.add_argument("--wgrad-streams", type=int, default=3,
                    help="streams the weight gradients go round-robin on; streams x CTA limit must not exceed the SM count")
    ap.add_argument("--algo", type=int, default=2,
                    help="2 (default): the tcgen05 kernels only, a shape they decline is an error; 0: fall back to the CUDA-core kernels; 1: CUDA-core kernels")
    ap.add_argument("--per-layer", default=None, help="write the per-layer table (JSON) here")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-chained", action="store_true", help="skip the chained-step timing (conv + batch norm + pooling + residuals)")
    ap.add_argument("--no-graph", action="store_true", help="launch every kernel eagerly instead of replaying a CUDA graph")
    ap.add_argument("--one-stream", action="store_true", help="capture the step on one stream (no dgrad/wgrad overlap)")
    ap.add_argument("--profile-chained", action="store_true", help="with --profile-steps: run the chained step instead")
    ap.add_argument("--profile-steps", type=int, default=0,
                    help="run only this many steps after one warm-up and print no timing: for a launch list (the one-pass "
                         "gpu__time_duration capture); captures with more metrics belong on a small case (layerbench, --net resnet32)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # no launcher: start the N ranks here (one process per GPU, rendezvous on the loopback address)
        spawn_ranks(args.gpus, _rank_main, (sys.argv[1:],))
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


def _rank_main(argv):
    sys.argv = [sys.argv[0]] + list(argv)
    main()


def _spawn_entry(rank, world, port, fn, fn_args):
    os.environ.update({"RANK": str(rank), "LOCAL_RANK": str(rank), "WORLD_SIZE": str(world), "MASTER_ADDR": "127.0.0.1",
                       "MASTER_PORT": str(port)})
    fn(*fn_args)


def spawn_ranks(n, fn, fn_args=()):
    """Runs fn(*fn_args) in n processes with RANK / LOCAL_RANK / WORLD_SIZE / MASTER_* set as a launcher would; raises if a
    rank fails."""
    import socket
    import torch.multiprocessing as mp
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    mp.spawn(_spawn_entry, args=(n, port, fn, fn_args), nprocs=n, join=True)


if __name__ == "__main__":
    main()
