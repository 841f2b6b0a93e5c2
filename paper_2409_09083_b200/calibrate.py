"""Fits the weights of the planner's time model (ftp_plan_cost) to measurements on the GPU at hand.

    python -m paper_2409_09083_b200.calibrate [--max-convs 3] [--out measurements.jsonl]

The paper picks its grouping profile by weighing halo recomputation against boundary exchanges
(Sections 4.2 and 5.3) without printing the procedure.  The planner estimates the time of one pass
of an executed group as a weighted sum of work terms; this script measures, for every candidate
group of one to three convs of the 8- and 16-layer stacks at several batch sizes and tile grids, the
kernel time of its forward and backward pass inside a whole training step (every other layer is a
group of its own, so the group finds its input the way it does in a real step), reads the terms of
the same plan, fits non-negative weights by least squares on the relative errors, and prints the
table in the form the planner's source holds, with the error of the fit.  Needs a CUDA device and
scipy; every step runs in the library.
"""
import argparse
import json
import statistics

import numpy as np

from . import synth

SETTINGS = [("yolo16", 608, 16, 5), ("yolo16", 608, 4, 3), ("yolo8", 416, 4, 3), ("yolo8", 416, 8, 4),
            ("yolo16", 608, 1, 3), ("yolo16", 608, 2, 6), ("yolo8", 416, 16, 2)]      # stack, size, batch, grid


def candidates(layers, max_convs):
    """(single-op profile, [(first, last)]): groups that start after a cut and end at one, a conv never
    parted from the pool after it."""
    L = len(layers)
    cut_ok = lambda e: e == L or not (layers[e - 1].kind == "conv" and layers[e].kind == "pool")
    cuts = [e for e in range(1, L + 1) if cut_ok(e)]
    starts = [1] + [e + 1 for e in cuts if e < L]
    out = []
    for s in starts:
        for e in cuts:
            if e >= s and sum(1 for l in layers[s - 1:e] if l.kind == "conv") <= max_convs:
                out.append((s, e))
    return list(zip(starts, cuts)), out


def measure(ftp, torch, max_convs, log):
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")          # > L2
    rows = []
    for stack, size, N, grid in SETTINGS:
        layers = synth.stack_yolo16() if stack == "yolo16" else synth.stack_yolo8()
        L = len(layers)
        c, h, w = synth.map_shapes(layers, 3, size, size)[-1]
        wl = synth.Workload("calibrate", tuple(layers), N, 3, size, size, (grid, grid), ((1, L),))
        params0 = torch.from_numpy(synth.draw(wl, N=1)[1]).cuda()
        gen = torch.Generator(device="cuda").manual_seed(0)
        x = torch.rand((N, 3, size, size), device="cuda", generator=gen)
        target = torch.randn((N, c, h, w), device="cuda", generator=gen)
        loss = torch.zeros(1, device="cuda")
        singles, cands = candidates(layers, max_convs)
        for s, e in cands:
            groups = tuple([g for g in singles if g[1] < s] + [(s, e)] + [g for g in singles if g[0] > e])
            gi = groups.index((s, e))
            for prec in (0, 1):
                try:
                    plan = ftp.ftp_plan(layers, N, 3, size, size, (grid, grid), groups, precision=prec, strict_groups=True)
                except ftp.FtpError:
                    continue                                                   # no sub-tile of the group fits
                ws, pd, tf, tb = plan.new_workspace(), params0.clone(), [], []
                plan.timing(True)
                for it in range(5):
                    flush.zero_()
                    ftp.ftp_step(plan, x, pd, 1e-3, ws, target=target, loss_out=loss)
                    torch.cuda.synchronize()
                    recs = plan.timing_read()
                    if it >= 2:
                        tf.append(sum(ms for k, g, ms in recs if g == gi and k == 1) * 1e3)
                        tb.append(sum(ms for k, g, ms in recs if g == gi and k in (3, 4)) * 1e3)
                plan.check(ws)
                row = dict(stack=stack, size=size, N=N, grid=grid, first=s, last=e, prec=prec,
                           us=[statistics.median(tf), statistics.median(tb)],
                           terms=[plan.cost(0, gi, s > 1)[0], plan.cost(1, gi, s > 1)[0]])
                rows.append(row)
                if log:
                    log.write(json.dumps(row) + "\n")
                    log.flush()
                del plan, ws
    return rows


def fit(rows):
    from scipy.optimize import nnls
    print("const double kCostWeights[2][2][kCostTerms] = {")
    for prec, name in ((0, "fp32: forward, backward"), (1, "bf16")):
        print("    {   // %s" % name)
        errs = []
        for ps in (0, 1):
            R = [r for r in rows if r["prec"] == prec]
            A = np.array([r["terms"][ps] for r in R])
            t = np.array([r["us"][ps] for r in R])
            w = nnls(A / t[:, None], np.ones(len(t)))[0]
            e = np.abs(np.log((A @ w) / t))
            errs.append("pass %d: %d groups, |log(estimate / measured)| median %.3f, 90th percentile %.3f, max %.3f"
                        % (ps, len(R), np.median(e), np.percentile(e, 90), e.max()))
            print("        {" + ", ".join("%.4g" % v for v in w) + "},")
        print("    },   // " + "; ".join(errs))
    print("};")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--max-convs", type=int, default=3)
    ap.add_argument("--out", default="", help="also write the measurements, one JSON line per (group, precision)")
    ap.add_argument("--fit", default="", help="skip the measurement and fit the lines of this file")
    args = ap.parse_args()
    if args.fit:
        rows = [json.loads(l) for l in open(args.fit)]
    else:
        import torch
        import paper_2409_09083_b200 as ftp
        log = open(args.out, "w") if args.out else None
        rows = measure(ftp, torch, args.max_convs, log)
    fit(rows)


if __name__ == "__main__":
    main()
