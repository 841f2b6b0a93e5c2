#!/usr/bin/env python
"""Benchmark of the fused tile-partitioned training step.

    python bench.py --gpus N --steps K --warmup W [--workload C3] [--impl reference]

A step is one pass of the whole hot path (forward, loss delta, backward with input gradient,
cross-tile reduction of the partial gradient sets, SGD update) over one batch of synthetic input.
Rank 0 prints ONE JSON line.  Without --workload the run measures the three benchmark workloads
C3 (the largest; the headline of the line), C1 and C2 (under "workloads"), each with its roofline,
end-to-end and CPU-oracle numbers, after measuring the fp32 FMA rate of the GPU with a register-only
kernel of the library (the peak the fp32 roofline fractions are quoted against).  With --gpus N > 1
(launched by torchrun, one rank per GPU) every rank runs the one-GPU path on its own batch of the
headline workload (weak scaling) and the summed gradients are all-reduced over NCCL before the
update.  --impl reference times the CPU oracle instead.
"""
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

from paper_2409_09083_b200 import synth  # noqa: E402

METRIC = "train-step images/sec (fwd+bwd+dW reduce+SGD)"
UNIT = "images/s"
HEADLINE = "C3"
# nominal fp32 FMA rate, used only if the measurement kernel cannot run: 148 SMs x 128 lanes x 2 flop x 1.965 GHz
FP32_NOMINAL_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12
# Launch kinds of the library's per-launch timing (ftp_plan_timing): name, and how many forward-equivalents of the
# executed group's multiply-accumulates the launch performs (None: a memory-bound helper)
KIND = {0: ("pack_filters", None), 1: ("fwd_group", 1), 2: ("loss_delta", None), 3: ("bwd_group", 2), 4: ("halo_sum", None),
        5: ("reduce_sgd", None), 6: ("delta_act", None), 7: ("filter_grad_rows", 1), 8: ("delta_conv_rows", 1),
        9: ("unroll_windows", None), 10: ("fold_windows", None)}
KERNEL = {("fwd_group", "fp32"): "fwd_group_kernel / conv_rows_kernel", ("bwd_group", "fp32"): "bwd_group_kernel / thin_bwd_kernel",
          ("filter_grad_rows", "fp32"): "filter_grad_rows_kernel", ("delta_conv_rows", "fp32"): "conv_rows_kernel (input delta)",
          ("fwd_group", "bf16"): "conv_tc_rows_kernel / fwd_group_tc_kernel", ("bwd_group", "bf16"): "bwd_group_tc_kernel",
          ("filter_grad_rows", "bf16"): "filter_grad_tc_rows_kernel", ("delta_conv_rows", "bf16"): "conv_tc_rows_kernel (input delta)"}
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu captures summarised
# under profiles/ (static: null for every kernel / workload without a capture of the current code)
NCU_TRAFFIC = {("C3", "fp32", "fwd_group"): 128.4e6, ("C3", "fp32", "filter_grad_rows"): 245.8e6,
               ("C3", "fp32", "delta_conv_rows"): 159.3e6, ("C3", "fp32", "bwd_group"): 950.4e6,
               ("C3", "bf16", "fwd_group"): 84.7e6, ("C3", "bf16", "filter_grad_rows"): 153.2e6, ("C3", "bf16", "delta_conv_rows"): 201.5e6}


def measured_bf16_peak():
    """Sustained dense bf16 TFLOP/s measured on this machine's B200s (generated file), else the fallback."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["bf16_tflops_sustained"]), "of measured (MEASURED_PEAKS.json, sustained cuBLAS bf16)"
    except (OSError, KeyError, ValueError):
        return 1400.0, "of fallback (1.4 PFLOP/s sustained)"


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=None, choices=["C0", "C1", "C2", "C3"],
                    help="measure this workload only (default: C3 as the headline, C1 and C2 beside it)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--precision", default="fp32", choices=["fp32", "bf16"],
                    help="fp32: CUDA-core path (tolerance 1e-4); bf16: tcgen05 tensor-core path, bf16 maps, fp32 accumulation (2e-2)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--min-seconds", type=float, default=2.0,
                    help="the K timed steps are repeated until this much time has passed; the median repeat is reported")
    ap.add_argument("--tc-blocks", type=int, default=0, choices=[0, 1, 2],
                    help="bf16 path: thread blocks per SM (0 = planner default)")
    ap.add_argument("--cost-model", type=int, default=0, choices=[-1, 0, 1],
                    help="planner's time model for cutting the requested groups: 0 planner default, 1 on, -1 off (fixed rule)")
    ap.add_argument("--stationary", type=int, default=0, choices=[-1, 0, 1],
                    help="one-conv groups on their own kernels (fp32: weight-stationary; bf16: banded tensor-core kernels): 0 planner default, "
                         "-1 never (fused stacks only)")
    ap.add_argument("--strict-groups", action="store_true", help="execute the requested grouping profile as it is (no cuts)")
    ap.add_argument("--no-bf16", action="store_true", help="skip the second measurement on the bf16 tensor-core path")
    return ap.parse_args()


def config_of(wl, extra=None):
    cfg = {"workload": f"{wl.name}: {len(wl.layers)}-layer YOLOv2-style stack, batch {wl.N}x{wl.C}x{wl.H}x{wl.W} fp32, "
                       f"tile grid {wl.grid[0]}x{wl.grid[1]}, requested groups {[list(g) for g in wl.groups]}, MSE loss, SGD lr {wl.lr}",
           "global_batch": wl.N, "tile_grid": list(wl.grid), "groups": [list(g) for g in wl.groups],
           "input_delta": True}
    cfg.update(extra or {})
    return cfg


def time_oracle(wl, images, steps, warmup):
    """Seconds per oracle training step on `images` images of the workload (as it stands)."""
    from oracle import reference as orc
    x, params, target = synth.draw(wl, N=images)
    layers = list(wl.layers)
    times = []
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        orc.step(layers, x, params, wl.lr, target=target)
        dt = time.perf_counter() - t0
        if i >= warmup:
            times.append(dt)
    return sum(times) / len(times), orc.num_threads()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = synth.workload(args.workload or HEADLINE)
    images = 1
    sec, cores = time_oracle(wl, images, args.steps, args.warmup)
    value = images / sec
    sample = f"each step = one full training step of the fp64 oracle on {images} image of {wl.name} at full resolution"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(wl, {"sample_images_per_step": images}),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.path = tempfile.mktemp(suffix=".csv")
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for row in open(self.path):
                f = [c.strip() for c in row.split(",")]
                if len(f) < 8:
                    continue
                try:
                    sm.append(float(f[0])); mx.append(float(f[1]))
                except ValueError:
                    continue
                for name, v in zip(names, f[4:8]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def measure_fma_peak(ftp, torch, local):
    """fp32 FMA rate of this GPU, TFLOP/s: the library's register-only FMA loop (ftp_fma_peak) timed with CUDA
    events, best of five launches of about 50 ms, with the SM clock sampled meanwhile."""
    out = torch.empty(1024 * torch.cuda.get_device_properties(local).multi_processor_count, dtype=torch.float32, device="cuda")
    try:
        ftp.ftp_fma_peak(out, 2000)
        torch.cuda.synchronize()
        sampler = ClockSampler(local)
        best = 0.0
        for _ in range(5):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            flops = ftp.ftp_fma_peak(out, 100000)
            b.record()
            torch.cuda.synchronize()
            best = max(best, flops / (a.elapsed_time(b) / 1e3) / 1e12)
        clocks = sampler.stop()
        return {"tflops": best, "source": "measured in this run: register-only fp32 FMA loop on all SMs (ftp_fma_peak), best of 5",
                "sm_mhz": clocks["sm_mhz"], "tflops_x_1000_over_sm_mhz": best * 1000.0 / clocks["sm_mhz"] if clocks["sm_mhz"] else None,
                "nominal_tflops": FP32_NOMINAL_TFLOPS}
    except Exception as e:                                    # noqa: BLE001 - the benchmark goes on with the nominal figure
        return {"tflops": FP32_NOMINAL_TFLOPS, "source": f"nominal 148 SMs x 128 lanes x 2 x 1.965 GHz (measurement failed: {e})",
                "sm_mhz": None, "nominal_tflops": FP32_NOMINAL_TFLOPS}


def run_ours(args):
    import torch
    import paper_2409_09083_b200 as ftp
    from paper_2409_09083_b200 import dp

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the training step has no CPU path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    fma = measure_fma_peak(ftp, torch, local) if rank == 0 else None
    ctx = dict(args=args, rank=rank, world=world, local=local, dist=dist, ftp=ftp, dp=dp, torch=torch, fma=fma)
    head = args.workload or HEADLINE
    line = measure(ctx, head, args.precision)
    if rank == 0:
        def with_bf16(name, into):
            if world == 1 and args.precision == "fp32" and not args.no_bf16:
                second = measure(ctx, name, "bf16", extras=False)
                into["bf16_tensor_core_path"] = {k: second[k] for k in ("value", "unit", "ms_per_step", "dtype", "roofline",
                                                                        "breakdown_ms_per_step", "gpu_launches", "e2e", "loss")}
                into["bf16_tensor_core_path"]["executed_groups"] = second["config"]["executed_groups"]
                try:        # the same step as fused sub-tile stacks only (what the one-conv kernels replace)
                    into["bf16_tensor_core_path"]["fused_stacks_only"] = measure(ctx, name, "bf16", light=True, stationary=-1)
                except Exception as e:                        # noqa: BLE001
                    into["bf16_tensor_core_path"]["fused_stacks_only"] = {"unavailable": str(e)}
        with_bf16(head, line)
        if args.workload is None and world == 1:
            line["workloads"] = {}
            for name in ("C1", "C2"):
                sub = measure(ctx, name, args.precision)
                with_bf16(name, sub)
                if args.precision == "fp32":
                    # the same step with the requested grouping profile executed as it is (fused sub-tile stacks
                    # of whole requested groups), and with fused stacks only under the planner's own cuts
                    for key, opts in (("requested_profile_as_is", dict(strict_groups=True, stationary=-1)),
                                      ("fused_stacks_only", dict(stationary=-1))):
                        try:
                            sub[key] = measure(ctx, name, "fp32", light=True, **opts)
                        except Exception as e:                # noqa: BLE001 - e.g. the requested groups do not fit as they are
                            sub[key] = {"unavailable": str(e)}
                line["workloads"][name] = {k: sub[k] for k in sub if k not in ("metric", "unit", "n_gpus", "higher_is_better", "scaling",
                                                                            "vs_baseline", "data", "fp32_fma_peak")}
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def measure(ctx, name, precision, extras=True, light=False, **plan_opts):
    """Times the training step of one workload at one precision; returns the JSON line (rank 0) or None.
    light: only the timed steps (for the comparison runs with other planner options, given as plan_opts)."""
    args, rank, world, local, dist = ctx["args"], ctx["rank"], ctx["world"], ctx["local"], ctx["dist"]
    ftp, dp, torch = ctx["ftp"], ctx["dp"], ctx["torch"]
    wl = synth.workload(name).with_(seed=rank)                # per-GPU batch is fixed: weak scaling
    x, params, target = synth.draw(wl)
    if world > 1:                                             # same initial parameters on every rank
        params = synth.draw(wl.with_(seed=0))[1]
    tcp = precision == "bf16"
    plan = ftp.ftp_plan(wl.layers, wl.N, wl.C, wl.H, wl.W, wl.grid, wl.groups, precision=1 if tcp else 0,
                        tc_blocks_per_sm=args.tc_blocks if tcp else 0, cost_model=args.cost_model,
                        **dict(dict(stationary=args.stationary, strict_groups=args.strict_groups), **plan_opts))
    ws = plan.new_workspace()
    xd, pd, td = (torch.from_numpy(a).cuda() for a in (x, params, target))
    dx = torch.empty_like(xd)
    grad = torch.empty_like(pd)
    loss = torch.zeros(1, dtype=torch.float32, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")      # > 126 MB L2
    steps = args.steps

    def step():
        if world == 1:
            ftp.ftp_step(plan, xd, pd, wl.lr, ws, target=td, loss_out=loss, dx=dx)
        else:
            # every executed group's gradient slice is all-reduced on a communication stream as soon as it is
            # complete, while the groups before it are back-propagated; the update follows the last slice
            ex = dp.cuda_overlap(torch, dist, grad, world)
            ftp.ftp_step_grad_groups(plan, xd, pd, grad, ws, ex.ready, target=td, loss_out=loss, dx=dx)
            ex.finish(wl.lr, lambda g, lr: ftp.ftp_sgd(pd, g, lr), join=ex.join)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed_steps(fn):
        """K steps, each bracketed by events on the launching stream with an L2 flush before it; returns total ms."""
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        barrier()
        for i, (a, b) in enumerate(ev):
            flush.zero_()                                     # evict the previous step from L2 (not timed)
            a.record()
            fn(i)
            b.record()
            torch.cuda.synchronize()
        barrier()
        total = sum(a.elapsed_time(b) for a, b in ev)
        if dist is not None:
            t = torch.tensor([total], dtype=torch.float64, device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            total = float(t.item())
        return total

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    plan.check(ws)          # a bounded device-side wait that ran out would invalidate everything below

    # The K timed steps run as a user's would, without per-launch instrumentation, and are repeated until
    # min_seconds have passed (every rank the same number of times); the median repeat is the reported one.
    sampler = ClockSampler(local) if rank == 0 else None
    launches0 = plan.launch_count()
    repeats = []
    t_begin = time.perf_counter()
    while True:
        repeats.append(timed_steps(lambda i: step()))
        budget = args.min_seconds * (0.25 if light else 1.0)
        more = torch.tensor([1.0 if time.perf_counter() - t_begin < budget and len(repeats) < 50 else 0.0], device="cuda")
        if dist is not None:
            dist.broadcast(more, 0)
        if more.item() == 0.0:
            break
    launches = (plan.launch_count() - launches0) // len(repeats)
    total_ms = statistics.median(repeats)
    if light:
        if sampler:
            sampler.stop()
        return {"value": world * wl.N * steps / (total_ms / 1e3), "unit": UNIT, "ms_per_step": total_ms / steps,
                "executed_groups": [list(g) for g in plan.exec_groups()],
                "stationary_groups": [bool(plan.group_mode(i)[0]) for i in range(len(plan.exec_groups()))],
                "gpu_launches": int(launches), "workspace_bytes": plan.workspace_bytes}
    # K more steps with an event pair around every launch of the library (ftp_plan_timing) for the per-kernel
    # breakdown and the launch durations of the roofline: the events do not change a kernel's duration, but
    # their records between the launches would lengthen the step, so they stay out of the timed steps.
    plan.timing(True)
    per_kind = {}
    for _ in range(steps):
        flush.zero_()
        step()
        torch.cuda.synchronize()
        for kind, group, ms in plan.timing_read():
            per_kind[(kind, group)] = per_kind.get((kind, group), 0.0) + ms
    barrier()
    plan.timing(False)
    clocks = sampler.stop() if sampler else None

    # end to end: batch and target start in pinned host memory every step, the loss comes back to the host
    e2e = None
    if world == 1:
        # Two pinned host batches take turns, as a data loader would hand them over.  Every step's interval
        # holds the step on this step's batch (its copies were started during the step before), the copies
        # of the NEXT batch from pinned host memory (ftp_prefetch_host on a copy stream; the interval ends
        # only when they are through as well) and the read of the loss.
        xh = [torch.from_numpy(x).pin_memory(), torch.from_numpy(x.copy()).pin_memory()]
        th = [torch.from_numpy(target).pin_memory(), torch.from_numpy(target.copy()).pin_memory()]
        lh = torch.zeros(1, dtype=torch.float32).pin_memory()
        copy_stream = torch.cuda.Stream()
        main = torch.cuda.current_stream()
        for i in range(2):
            ftp.ftp_step_host(plan, xh[i], th[i], pd, wl.lr, lh, ws, dx=dx)
        ftp.ftp_prefetch_host(plan, xh[0], th[0], ws, copy_stream)
        torch.cuda.synchronize()

        def host_step(i):
            ftp.ftp_step_host(plan, xh[i % 2], th[i % 2], pd, wl.lr, lh, ws, dx=dx)
            ftp.ftp_prefetch_host(plan, xh[(i + 1) % 2], th[(i + 1) % 2], ws, copy_stream)
            main.wait_stream(copy_stream)
        e2e_ms = timed_steps(host_step)
        _ = float(lh[0])
        e2e = {"value": wl.N * steps / (e2e_ms / 1e3), "unit": UNIT,
               "h2d_bytes_per_step": int(xh[0].numel() * 4 + th[0].numel() * 4), "d2h_bytes_per_step": 4,
               "pipeline": "next batch prefetched from pinned host memory during the step (ftp_prefetch_host)"}

    if rank != 0:
        return None

    eg = plan.exec_groups()
    modes = [plan.group_mode(i) for i in range(len(eg))]
    layers = list(wl.layers)
    shapes = synth.map_shapes(layers, wl.C, wl.H, wl.W)

    def group_macs(gi):
        a, b = eg[gi]
        return sum(l.cout * l.cin * l.k * l.k * shapes[i + 1][1] * shapes[i + 1][2]
                   for i, l in enumerate(layers) if l.kind == "conv" and a <= i + 1 <= b)
    macs = synth.forward_macs_per_image(wl.layers, wl.C, wl.H, wl.W)
    ms_step = total_ms / steps
    breakdown, per_group, flops_kind, launches_kind = {}, {}, {}, {}
    for (kind, group), ms in per_kind.items():
        kname, fwd_equiv = KIND[kind]
        breakdown[kname] = breakdown.get(kname, 0.0) + ms / steps
        launches_kind[kname] = launches_kind.get(kname, 0) + 1
        if group >= 0:
            per_group[f"{kname}[{group}]"] = per_group.get(f"{kname}[{group}]", 0.0) + ms / steps
            if fwd_equiv:
                flops_kind[kname] = flops_kind.get(kname, 0.0) + 2.0 * fwd_equiv * group_macs(group) * wl.N
    # the dominant kernel = the arithmetic kernel class with the largest share of the step
    if tcp:
        peak, src, bound = *measured_bf16_peak(), "tensor"
    else:
        peak, src, bound = ctx["fma"]["tflops"], ctx["fma"]["source"], "alu"
    per_kernel = {k: {"ms_per_step": breakdown[k], "algorithmic_flops_per_step": f,
                      "achieved_tflops": f / (breakdown[k] / 1e3) / 1e12, "frac": f / (breakdown[k] / 1e3) / 1e12 / peak,
                      "launches_per_step": launches_kind[k]}
                  for k, f in flops_kind.items() if breakdown.get(k, 0.0) > 0}
    dom = max(per_kernel, key=lambda k: per_kernel[k]["ms_per_step"])
    d = per_kernel[dom]
    roofline = {"bound": bound, "kernel": KERNEL.get((dom, precision), dom), "achieved": d["achieved_tflops"], "peak": peak,
                "unit": "TFLOP/s", "frac": d["frac"], "traffic": NCU_TRAFFIC.get((wl.name, precision, dom)),
                "traffic_unit": "bytes per launch (static, from the ncu captures under profiles/; null: no capture of the current kernel)",
                "peak_source": src, "launches_per_step": d["launches_per_step"],
                "avg_launch_ms": d["ms_per_step"] / d["launches_per_step"],
                "algorithmic_flops_per_step": d["algorithmic_flops_per_step"],
                "per_kernel": per_kernel,
                "step_frac_of_peak": 6.0 * macs * wl.N / (ms_step / 1e3) / 1e12 / peak}
    exec_desc = [f"{list(g)}{'*' if m[0] else ''}" for g, m in zip(eg, modes)]
    cfg = config_of(wl, {"global_batch": wl.N * world, "precision": precision, "executed_groups": [list(g) for g in eg],
                         "stationary_groups": [bool(m[0]) for m in modes], "partial_sets": [m[1] for m in modes],
                         "parallelism": f"dp{world}", "l2": "flushed between timed steps (256 MiB write)",
                         "timing": f"value: median of {len(repeats)} repeats of K steps without per-launch events; breakdown and roofline: "
                                   "K more steps with an event pair around every launch",
                         "repeats": len(repeats), "workspace_bytes": plan.workspace_bytes, "redundancy_fwd": plan.redundancy})
    cfg["workload"] += f"; executed as groups {' '.join(exec_desc)} (* = one-conv group run weight-stationary{', its filter gradient on the bf16 path' if tcp else ''})"
    line = {"metric": METRIC, "value": world * wl.N * steps / (total_ms / 1e3), "unit": UNIT, "n_gpus": world,
            "steps": steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if tcp else "f32", "data": "synthetic",
            "config": cfg, "clocks": clocks, "gpu_launches": int(launches), "breakdown_ms_per_step": breakdown,
            "per_group_ms_per_step": per_group, "roofline": roofline, "loss": float(loss.item())}
    if not tcp:
        line["fp32_fma_peak"] = ctx["fma"]
    if e2e is not None:
        line["e2e"] = e2e
    if world == 1 and extras and not args.no_cpu_baseline:
        images = 1 if len(wl.layers) > 8 else min(wl.N, 2)
        sec, cores = time_oracle(wl, images, 1, 0)
        line["cpu_baseline"] = {"value": images / sec, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"one fp64 oracle training step on {images} image(s) of {wl.name} at full resolution, "
                                          "scaled per image"}
    return line


def main():
    args = parse()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
