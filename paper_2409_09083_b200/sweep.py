"""Sweep of the training step over batch size, tile grid, group profile and precision on the 16-layer
stack (the axes of the paper's grouping / batch-size experiments, Section 5, on synthetic data).

    python -m paper_2409_09083_b200.sweep [--stack yolo16] [--batches 1,4,16] [--grids 1,3,5] [--size 608] [--steps 5]
                                         [--profiles pairs,planner]

Prints one JSON line per point: images/s, ms per step, executed groups, redundancy, workspace.
Needs a CUDA device; every step runs in the library.
"""
import argparse
import json

from . import synth


def profiles(layers):
    """name -> (requested groups, max_group_convs).  The first three are executed as requested as far as
    they fit in shared memory; "pairs" is one all-in-one group cut by the fixed rule (two convs per
    executed group, ending at a pool); "planner" lets the planner cut it its default way, i.e. where
    its time model puts the minimum."""
    return {"all-in-one": (((1, len(layers)),), -1),
            "per-maxpool": (synth.groups_per_maxpool(layers), -1),
            "per-layer": (synth.groups_per_layer(layers), -1),
            "pairs": (((1, len(layers)),), 2),
            "planner": (((1, len(layers)),), 0)}


def time_point(ftp, torch, layers, N, size, grid, groups, precision, steps, warmup=3, max_group_convs=0):
    wl = synth.Workload("sweep", tuple(layers), N, 3, size, size, (grid, grid), tuple(groups))
    x, params, target = synth.draw(wl)
    plan = ftp.ftp_plan(wl.layers, N, wl.C, wl.H, wl.W, wl.grid, wl.groups, precision=precision,
                        max_group_convs=max_group_convs)
    ws = plan.new_workspace()
    xd, pd, td = (torch.from_numpy(a).cuda() for a in (x, params, target))
    dx = torch.empty_like(xd)
    loss = torch.zeros(1, dtype=torch.float32, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for _ in range(warmup):
        ftp.ftp_step(plan, xd, pd, wl.lr, ws, target=td, loss_out=loss, dx=dx)
    plan.check(ws)
    total = 0.0
    for _ in range(steps):
        flush.zero_()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        ftp.ftp_step(plan, xd, pd, wl.lr, ws, target=td, loss_out=loss, dx=dx)
        b.record()
        torch.cuda.synchronize()
        total += a.elapsed_time(b)
    ms = total / steps
    return {"images_per_s": N / (ms / 1e3), "ms_per_step": ms, "executed_groups": plan.exec_groups(),
            "redundancy_fwd": plan.redundancy, "workspace_mb": plan.workspace_bytes / 1e6, "loss": float(loss.item())}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--batches", default="1,4,16")
    ap.add_argument("--grids", default="1,3,5")
    ap.add_argument("--stack", default="yolo16", choices=["yolo8", "yolo16"])
    ap.add_argument("--size", type=int, default=608)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--precisions", default="fp32,bf16")
    ap.add_argument("--profiles", default="", help="comma-separated subset of the profile names (default: all)")
    args = ap.parse_args()
    import torch
    import paper_2409_09083_b200 as ftp
    layers = synth.stack_yolo16() if args.stack == "yolo16" else synth.stack_yolo8()
    for prec in args.precisions.split(","):
        for N in (int(v) for v in args.batches.split(",")):
            for grid in (int(v) for v in args.grids.split(",")):
                for name, (groups, mgc) in profiles(layers).items():
                    if args.profiles and name not in args.profiles.split(","):
                        continue
                    try:
                        r = time_point(ftp, torch, layers, N, args.size, grid, groups, 1 if prec == "bf16" else 0, args.steps,
                                       max_group_convs=mgc)
                    except ftp.FtpError as e:
                        r = {"error": str(e)}
                    print(json.dumps({"precision": prec, "batch": N, "grid": grid, "profile": name, **r}), flush=True)
                    torch.cuda.empty_cache()


if __name__ == "__main__":
    main()
