"""Parity of the CUDA path (through the C-ABI binding) with the fp64 oracle, element by element
on the same seeded inputs.  Tolerance of the fp32 path: per tensor
max|gpu - oracle| / max|oracle| <= 1e-4 for activations, input gradients and weight gradients.

Max-pool arg-max and leaky-ReLU sign are discrete decisions taken on floating-point values; a
near-tie decided differently in fp32 and fp64 moves a whole delta to another pixel.  Gradient
parity is therefore checked on inputs where both precisions decide alike: small cases whose
oracle-side decision margins are verified to be far above fp32 rounding, and larger cases with
dyadic data whose forward pass is exact in fp32 (activations then also match bit for bit, exact
ties included).  Activations are checked on the paper-like inputs at every size."""
import numpy as np
import pytest
import torch

import paper_2409_09083_b200 as ftp
from paper_2409_09083_b200 import binding, synth
from _util import (FP32_TOL, draw_unambiguous, rel_err, run_gpu, run_gpu_step, run_oracle)

pytestmark = pytest.mark.gpu

W = synth.Workload
conv, pool = synth.conv, synth.pool

SMALL = {
    "C0": (synth.workload("C0"), {}),
    "C0-1x1grid": (synth.workload("C0").with_(grid=(1, 1)), {}),
    "C0-per-layer": (synth.workload("C0").with_(groups=((1, 1), (2, 2), (3, 3))), {}),
    "C0-subtiled": (synth.workload("C0"), dict(max_subtile=3)),
    "C0-16tiles": (synth.workload("C0").with_(grid=(16, 16)), {}),          # one output pixel per tile
    "one-conv": (W("a", (conv(3, 8, 3),), 2, 3, 20, 28, (2, 2), ((1, 1),), x_dist="normal"), {}),
    "conv1x1-odd-channels": (W("b", (conv(5, 13, 1),), 2, 5, 10, 14, (2, 3), ((1, 1),), x_dist="normal"), {}),
    "conv5-pool-conv": (W("c", (conv(2, 6, 5), pool(), conv(6, 4, 3)), 1, 2, 24, 24, (2, 2), ((1, 3),), x_dist="normal"), {}),
    "conv7": (W("d", (conv(1, 3, 7),), 1, 1, 18, 22, (2, 2), ((1, 1),), x_dist="normal"), {}),
    "conv-pool": (W("e", (conv(3, 8, 3), pool()), 1, 3, 16, 24, (2, 2), ((1, 2),), x_dist="normal"), {}),
    "pool-first": (W("f", (pool(), conv(3, 8, 3), pool(), pool()), 1, 3, 32, 48, (2, 2), ((1, 4),), x_dist="normal"), {}),
    "pool|conv-split": (W("g", (conv(3, 6, 3), pool(), conv(6, 5, 3)), 3, 3, 12, 20, (3, 2), ((1, 1), (2, 3)), x_dist="normal"), {}),
    # fused conv+pool ops whose delta is staged in more than one slice (20 and 24 channels, 16 at a time),
    # with 7 x 7 and 5 x 5 windows, in one group and cut between them; filters staged a few channels at a time
    "conv7-pool-conv5-pool": (W("h", (conv(4, 20, 7), pool(), conv(20, 24, 5), pool()), 1, 4, 12, 16, (2, 2), ((1, 4),), x_dist="normal"),
                              dict(strict_groups=True)),
    "conv7-pool|conv5-pool": (W("i", (conv(4, 20, 7), pool(), conv(20, 24, 5), pool()), 1, 4, 12, 16, (1, 2), ((1, 2), (3, 4)), x_dist="normal"), {}),
}


@pytest.mark.parametrize("name", sorted(SMALL))
def test_small_cases_match_oracle(name):
    wl, opts = SMALL[name]
    wl, x, params, target, ref = draw_unambiguous(wl)
    got = run_gpu(wl, x, params, target=target, **opts)
    assert rel_err(got["y"], ref["y"]) <= FP32_TOL
    ref = run_oracle(wl, x, params, dy=got["dy"])     # same loss delta on both sides
    assert rel_err(got["dx"], ref["dx"]) <= FP32_TOL
    assert rel_err(got["dparams"], ref["dparams"]) <= FP32_TOL


@pytest.mark.parametrize("name", ["C0", "conv5-pool-conv", "pool|conv-split"])
def test_step_updates_parameters_like_the_oracle(name):
    wl, opts = SMALL[name]
    wl, x, params, target, ref = draw_unambiguous(wl)
    lr = 0.05
    ref = run_oracle(wl, x, params, target=target, lr=lr)
    got = run_gpu_step(wl, x, params, target, lr, **opts)
    assert got["loss"] == pytest.approx(ref["loss"], rel=1e-5)
    assert rel_err(got["new_params"] - params, ref["new_params"] - params) <= FP32_TOL
    assert rel_err(got["dx"], ref["dx"]) <= FP32_TOL
    # without dx the same update must come out
    got2 = run_gpu_step(wl, x, params, target, lr, want_dx=False, **opts)
    assert np.array_equal(got2["new_params"], got["new_params"])


Y8 = W("y8", tuple(synth.stack_yolo8()), 2, 3, 64, 96, (3, 3), ((1, 8),))
Y16 = W("y16", tuple(synth.stack_yolo16()), 1, 3, 96, 160, (5, 5), ((1, 4), (5, 8), (9, 16)))
WIDE = W("wide", (conv(3, 16, 3), pool(), conv(16, 512, 1), pool(), conv(512, 1024, 3), conv(1024, 512, 1)), 2, 3, 40, 56,
         (2, 2), ((1, 2), (3, 4), (5, 5), (6, 6)))
DYADIC = {
    "yolo8-one-group": (Y8, 3, {}),
    "yolo8-strict-one-group": (Y8, 3, dict(strict_groups=True)),
    "yolo8-two-groups-4x4": (Y8.with_(grid=(4, 4), groups=((1, 4), (5, 8))), 3, {}),
    "yolo8-per-layer": (Y8.with_(groups=synth.groups_per_layer(Y8.layers)), 3, {}),
    "yolo8-per-maxpool": (Y8.with_(groups=synth.groups_per_maxpool(Y8.layers)), 3, {}),
    "yolo8-subtile4": (Y8.with_(grid=(2, 2), groups=((1, 4), (5, 8))), 3, dict(max_subtile=4)),
    "yolo8-ragged-5x7grid": (Y8.with_(H=88, W=104, grid=(5, 7), groups=((1, 2), (3, 8))), 3, {}),
    "yolo8-1x1grid": (Y8.with_(grid=(1, 1), N=3), 3, {}),
    "yolo16-three-groups": (Y16, 2, {}),
    "yolo16-all-in-one": (Y16.with_(groups=((1, 16),), grid=(2, 3)), 2, {}),
    # the shapes of the layers behind the 16-layer stack (512 -> 1024 3x3, 1024 -> 512 1x1 on a map of a few hundred
    # pixels): filters of 19 MB against maps of 0.6 MB, one-conv groups and two of them fused
    "wide-1024": (WIDE, 3, {}),
    "wide-1024-fused-pair": (WIDE.with_(groups=((1, 4), (5, 6))), 3, dict(strict_groups=True)),
}


@pytest.mark.parametrize("name", sorted(DYADIC))
def test_mid_size_stacks_match_oracle(name):
    wl, nnz, opts = DYADIC[name]
    wl = synth.with_slope(wl, 0.5)
    x, params, target = synth.draw_dyadic(wl, nnz=nnz)
    ref = run_oracle(wl, x, params, target=target)
    got = run_gpu(wl, x, params, target=target, **opts)
    assert np.array_equal(got["y"].astype(np.float64), ref["y"])       # forward is exact
    assert rel_err(got["dx"], ref["dx"]) <= FP32_TOL
    assert rel_err(got["dparams"], ref["dparams"]) <= FP32_TOL


def test_result_does_not_depend_on_grid_or_groups_and_is_reproducible():
    wl = Y8
    x, params, target = synth.draw(wl, bias_std=0.1)
    rng = np.random.default_rng(1)
    dy = rng.standard_normal((wl.N, 128, 8, 12)).astype(np.float32)
    base = run_gpu(wl.with_(grid=(1, 1)), x, params, dy=dy, strict_groups=True)
    again = run_gpu(wl.with_(grid=(1, 1)), x, params, dy=dy, strict_groups=True)
    for k in ("y", "dx", "dparams"):
        assert np.array_equal(base[k], again[k]), f"{k} differs from run to run"
    variants = [dict(grid=(3, 3)), dict(grid=(4, 2), groups=((1, 4), (5, 8))),
                dict(grid=(2, 5), groups=synth.groups_per_layer(wl.layers)), dict(grid=(8, 12)),
                dict(grid=(2, 2), opts=dict(max_group_convs=-1)), dict(grid=(3, 2), opts=dict(max_group_convs=1)),
                dict(grid=(3, 3), opts=dict(cost_model=1)), dict(grid=(3, 3), opts=dict(cost_model=-1)),
                # less shared memory: the conv+pool input delta without its staging area, and with smaller ones
                # (first split that fits and fixed-rule groups: see test_delta_staging_is_granted_only_where_it_fits)
                dict(grid=(2, 2), opts=dict(smem_bytes=100000, max_subtile=64, cost_model=-1)),
                dict(grid=(2, 2), opts=dict(smem_bytes=120000, max_subtile=64, cost_model=-1))]
    for v in variants:
        opts = v.pop("opts", {})
        got = run_gpu(wl.with_(**v), x, params, dy=dy, **opts)
        assert np.array_equal(got["y"], base["y"])                   # same arithmetic per output value
        assert rel_err(got["dx"], base["dx"]) <= 1e-5                # sums in another order
        assert rel_err(got["dparams"], base["dparams"]) <= 1e-5


def _crop_check(wl, x, params, y_gpu, n, oy, ox, size):
    """Oracle forward on a crop that contains the receptive field of y[n, :, oy:oy+size, ox:ox+size]."""
    from oracle import spans
    layers = list(wl.layers)
    shapes = synth.map_shapes(layers, wl.C, wl.H, wl.W)
    scale = wl.H // shapes[-1][1]
    def crop_axis(o, extent_out, extent_in):
        a, b = spans.forward_spans(layers, extent_out, (o, o + size - 1))[0]
        a = (a // scale) * scale
        b = min(extent_in, -(-(b + 1) // scale) * scale)
        return a, b
    y0, y1 = crop_axis(oy, shapes[-1][1], wl.H)
    x0, x1 = crop_axis(ox, shapes[-1][2], wl.W)
    sub = wl.with_(H=y1 - y0, W=x1 - x0, N=1)
    from oracle import reference as orc
    maps, _ = orc.forward(list(sub.layers), x[n:n + 1, :, y0:y1, x0:x1].astype(np.float64), params.astype(np.float64))
    ref = maps[-1][0, :, oy - y0 // scale: oy - y0 // scale + size, ox - x0 // scale: ox - x0 // scale + size]
    got = y_gpu[n, :, oy:oy + size, ox:ox + size]
    return float(np.abs(got - ref).max()), float(np.abs(ref).max())


@pytest.mark.parametrize("name", ["C1", "C2", "C3"])
def test_full_size_activations_on_sampled_regions(name):
    """Benchmark launch configuration, paper-like inputs: output regions sampled at the map
    corners, at tile boundaries and in the interior, each recomputed by the oracle from the
    crop of the input that contains its receptive field."""
    wl = synth.workload(name)
    x, params, target = synth.draw(wl)
    plan = ftp.ftp_plan(wl.layers, wl.N, wl.C, wl.H, wl.W, wl.grid, wl.groups)
    ws = plan.new_workspace()
    xd, pd = torch.from_numpy(x).cuda(), torch.from_numpy(params).cuda()
    c, h, w = synth.map_shapes(wl.layers, wl.C, wl.H, wl.W)[-1]
    y = torch.empty((wl.N, c, h, w), dtype=torch.float32, device="cuda")
    ftp.ftp_forward(plan, xd, pd, y, ws)
    torch.cuda.synchronize()
    yh = y.cpu().numpy()
    scale = float(np.abs(yh).max())
    size = 4
    ty = h // wl.grid[0]
    spots = [(0, 0, 0), (wl.N - 1, h - size, w - size), (wl.N // 2, ty - 2, ty - 2), (0, h // 2, w // 3),
             (wl.N - 1, 0, w - size)]
    for n, oy, ox in spots:
        err, _ = _crop_check(wl, x, params, yh, n, oy, ox, size)
        assert err / scale <= FP32_TOL, (n, oy, ox, err / scale)


@pytest.mark.parametrize("name,images", [("C1", None), ("C2", None), ("C3", (0, 15))])
def test_full_size_gradients(name, images):
    """Benchmark launch configuration with dyadic data (forward exact, so both sides take the
    same arg-max and sign decisions).  C1 and C2: the whole batch against the oracle.  C3: the
    loss delta is zero except on two images, so the batch's filter gradient equals the oracle's
    on those two images alone (the gradient is a sum over images)."""
    wl = synth.with_slope(synth.workload(name), 0.5)
    x, params, target = synth.draw_dyadic(wl, nnz=2)
    c, h, w = synth.map_shapes(wl.layers, wl.C, wl.H, wl.W)[-1]
    rng = np.random.default_rng(3)
    dy = rng.standard_normal((wl.N, c, h, w)).astype(np.float32)
    if images is not None:
        mask = np.zeros(wl.N, dtype=bool)
        mask[list(images)] = True
        dy[~mask] = 0.0
    got = run_gpu(wl, x, params, dy=dy)
    sel = slice(None) if images is None else list(images)
    ref = run_oracle(wl.with_(N=len(x[sel])), x[sel], params, dy=dy[sel])
    assert np.array_equal(got["y"][sel].astype(np.float64), ref["y"])
    assert rel_err(got["dx"][sel], ref["dx"]) <= FP32_TOL
    assert rel_err(got["dparams"], ref["dparams"]) <= FP32_TOL
    if images is not None:
        rest = [i for i in range(wl.N) if i not in images]
        assert not got["dx"][rest].any()


@pytest.mark.parametrize("shape", [(1, 16, 8, 8), (3, 5, 7, 9)])
def test_loss_mse_matches_oracle(shape):
    """The loss-delta injection on its own: L = mean((y - t)^2), dy = 2 (y - t) / M."""
    from oracle import reference as orc
    N, C, H, Wd = shape
    wl = W("mse", (conv(2, C, 1),), N, 2, H, Wd, (1, 1), ((1, 1),))
    plan = ftp.ftp_plan(wl.layers, N, wl.C, H, Wd, wl.grid, wl.groups)
    ws = plan.new_workspace()
    rng = np.random.default_rng(5)
    y = rng.standard_normal(shape).astype(np.float32)
    t = rng.standard_normal(shape).astype(np.float32)
    yd, td = torch.from_numpy(y).cuda(), torch.from_numpy(t).cuda()
    dy = torch.empty_like(yd)
    loss = torch.zeros(1, dtype=torch.float32, device="cuda")
    ftp.ftp_loss_mse(plan, yd, td, dy, loss, ws)
    torch.cuda.synchronize()
    ref_loss, ref_dy = orc.mse_loss(y.astype(np.float64), t.astype(np.float64))
    assert loss.item() == pytest.approx(ref_loss, rel=1e-5)
    assert rel_err(dy.cpu().numpy(), ref_dy) <= 1e-6


@pytest.mark.gpu
@pytest.mark.parametrize("precision", [0, 1])
def test_cost_model_estimates_track_measured_pass_times(precision):
    """The planner's time model, fitted on B200, against the kernels it describes: on the 8-layer
    stack at 416 x 416 (batch 4, 3 x 3 tiles) the estimate of every executed group's forward and
    backward pass is within a factor of 2.5 of the measured kernel time, and the whole step within
    a factor of 1.6.  (Median error of the fit is about 5 %; the slack covers other clocks.)"""
    wl = synth.workload("C1")
    x, params, target = synth.draw(wl)
    plan = ftp.ftp_plan(wl.layers, wl.N, wl.C, wl.H, wl.W, wl.grid, wl.groups, precision=precision)
    ws = plan.new_workspace("cuda")
    xd, pd, td = (torch.from_numpy(a).cuda() for a in (x, params.copy(), target))
    loss = torch.zeros(1, device="cuda")
    plan.timing(True)
    best = {}
    for it in range(4):
        ftp.ftp_step(plan, xd, pd, 1e-3, ws, target=td, loss_out=loss)
        torch.cuda.synchronize()
        recs = plan.timing_read()
        if it == 0:
            continue                                                   # first call packs filters and uploads tables
        for g in range(len(plan.exec_groups())):
            f = sum(ms for k, gg, ms in recs if gg == g and k == 1) * 1e3
            b = sum(ms for k, gg, ms in recs if gg == g and k in (3, 4, 6, 7, 8)) * 1e3
            best[g] = (min(f, best.get(g, (f, b))[0]), min(b, best.get(g, (f, b))[1]))
    plan.check(ws)
    tot_meas = tot_est = 0.0
    for g, (a, _) in enumerate(plan.exec_groups()):
        for ps in (0, 1):
            est = plan.cost(ps, g, a > 1)[1]
            assert best[g][ps] / 2.5 <= est <= best[g][ps] * 2.5, (g, ps, est, best[g][ps])
            tot_meas += best[g][ps]; tot_est += est
    assert tot_meas / 1.6 <= tot_est <= tot_meas * 1.6


@pytest.mark.gpu
@pytest.mark.parametrize("precision", [0, 1])
def test_step_can_be_captured_in_a_cuda_graph(precision):
    """ftp_step only launches kernels on the caller's stream once the plan's tables are on the device
    (first call): captured in a CUDA graph and replayed, three steps leave bit for bit the
    parameters and the loss that three direct calls leave."""
    wl = synth.workload("C0").with_(N=2)
    x, params, target = synth.draw(wl, N=2)
    plan = ftp.ftp_plan(wl.layers, 2, wl.C, wl.H, wl.W, wl.grid, wl.groups, precision=precision)
    ws = plan.new_workspace("cuda")
    xd, p0, td = (torch.from_numpy(a).cuda() for a in (x, params, target))
    loss = torch.zeros(1, device="cuda")
    dx = torch.empty_like(xd)
    pd = p0.clone()
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        ftp.ftp_step(plan, xd, pd, 0.05, ws, target=td, loss_out=loss, dx=dx, stream=s)      # uploads the tables
    torch.cuda.synchronize()
    pd.copy_(p0)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=s):
        ftp.ftp_step(plan, xd, pd, 0.05, ws, target=td, loss_out=loss, dx=dx, stream=s)
    launches = plan.launch_count()
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    plan.check(ws)
    assert plan.launch_count() == launches                   # replays do not go through the library
    p_graph, l_graph, dx_graph = pd.clone(), float(loss.item()), dx.clone()
    pd.copy_(p0)
    for _ in range(3):
        ftp.ftp_step(plan, xd, pd, 0.05, ws, target=td, loss_out=loss, dx=dx)
    torch.cuda.synchronize()
    assert torch.equal(p_graph, pd) and l_graph == float(loss.item()) and torch.equal(dx_graph, dx)
    assert not torch.equal(pd, p0)


@pytest.mark.gpu
@pytest.mark.parametrize("precision", [0, 1])
def test_host_batches_with_and_without_prefetch(precision):
    """ftp_step_host on four different host batches in a row: copying each batch inside its step,
    prefetching every batch during the previous step (ftp_prefetch_host), and prefetching on a
    caller's copy stream all leave bit for bit the parameters and losses of ftp_step on device
    copies.  A step given other host pointers than the prefetched ones copies as usual, and the
    prefetched batch is still there for the step after it."""
    wl = synth.workload("C0").with_(N=2)
    batches = [synth.draw(wl.with_(seed=s), N=2) for s in range(4)]
    params = batches[0][1]
    plan = ftp.ftp_plan(wl.layers, 2, wl.C, wl.H, wl.W, wl.grid, wl.groups, precision=precision)
    ws = plan.new_workspace("cuda")
    lr = 0.05

    def run(mode):
        pd = torch.from_numpy(params.copy()).cuda()
        xs = [torch.from_numpy(b[0]).pin_memory() for b in batches]
        ts = [torch.from_numpy(b[2]).pin_memory() for b in batches]
        lh = [torch.zeros(1).pin_memory() for _ in batches]
        copy_stream = torch.cuda.Stream() if mode == "own-stream" else None
        losses = []
        if mode == "device":
            loss = torch.zeros(1, device="cuda")
            for x, t in zip(xs, ts):
                ftp.ftp_step(plan, x.cuda(), pd, lr, ws, target=t.cuda(), loss_out=loss)
                losses.append(float(loss.item()))
        elif mode == "plain":
            for x, t, l in zip(xs, ts, lh):
                ftp.ftp_step_host(plan, x, t, pd, lr, l, ws)
        elif mode == "skipped":
            # batch 1 is prefetched, then batch 0 runs without having been prefetched, then batch 1 finds its copy
            ftp.ftp_prefetch_host(plan, xs[1], ts[1], ws)
            ftp.ftp_step_host(plan, xs[0], ts[0], pd, lr, lh[0], ws)
            ftp.ftp_step_host(plan, xs[1], ts[1], pd, lr, lh[1], ws)
            for i in (2, 3):
                ftp.ftp_step_host(plan, xs[i], ts[i], pd, lr, lh[i], ws)
        elif mode == "side-stream-current":
            # a non-default stream is current: the steps run on it, the default prefetch still goes to the
            # plan's own side stream (NULL at the C-ABI), not behind the step on the current stream
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            seen = []
            real = binding._lib.ftp_prefetch_host

            def spy(h, px, pt, pw, st):
                seen.append(st)
                return real(h, px, pt, pw, st)
            spy.argtypes, spy.restype = real.argtypes, real.restype
            binding._lib.ftp_prefetch_host = spy
            try:
                with torch.cuda.stream(side):
                    ftp.ftp_prefetch_host(plan, xs[0], ts[0], ws)
                    for i in range(4):
                        ftp.ftp_step_host(plan, xs[i], ts[i], pd, lr, lh[i], ws)
                        if i + 1 < 4:
                            ftp.ftp_prefetch_host(plan, xs[i + 1], ts[i + 1], ws)
            finally:
                binding._lib.ftp_prefetch_host = real
            assert seen == [None] * 4
        else:
            ftp.ftp_prefetch_host(plan, xs[0], ts[0], ws, copy_stream)
            for i in range(4):
                ftp.ftp_step_host(plan, xs[i], ts[i], pd, lr, lh[i], ws)
                if i + 1 < 4:
                    ftp.ftp_prefetch_host(plan, xs[i + 1], ts[i + 1], ws, copy_stream)
        torch.cuda.synchronize()
        plan.check(ws)
        if mode != "device":
            losses = [float(l[0]) for l in lh]
        return pd.cpu().numpy(), losses

    ref_p, ref_l = run("device")
    assert len(set(ref_l)) == 4                                  # four different batches
    for mode in ("plain", "prefetch", "own-stream", "skipped", "side-stream-current", "prefetch"):
        p, l = run(mode)
        assert np.array_equal(p, ref_p), mode
        assert l == ref_l, mode


@pytest.mark.parametrize("precision", [0, 1])
def test_step_grad_then_sgd_equals_step(precision):
    """The two halves of the data-parallel step at world size 1: ftp_step_grad followed by ftp_sgd leaves
    the parameters, the loss and the input gradient of ftp_step, bit for bit."""
    wl = Y8
    x, params, target = synth.draw(wl, bias_std=0.1)
    lr = 0.05
    plan = ftp.ftp_plan(wl.layers, wl.N, wl.C, wl.H, wl.W, wl.grid, wl.groups, precision=precision)
    ws = plan.new_workspace()
    xd, td = torch.from_numpy(x).cuda(), torch.from_numpy(target).cuda()
    pa, pb = torch.from_numpy(params.copy()).cuda(), torch.from_numpy(params.copy()).cuda()
    la, lb = torch.zeros(1, device="cuda"), torch.zeros(1, device="cuda")
    dxa, dxb = torch.empty_like(xd), torch.empty_like(xd)
    ftp.ftp_step(plan, xd, pa, lr, ws, target=td, loss_out=la, dx=dxa)
    grad = torch.full_like(pb, float("nan"))
    ftp.ftp_step_grad(plan, xd, pb, grad, ws, target=td, loss_out=lb, dx=dxb)
    torch.cuda.synchronize()
    assert np.array_equal(pb.cpu().numpy(), params)                  # ftp_step_grad leaves the parameters alone
    ftp.ftp_sgd(pb, grad, lr)
    plan.check(ws)
    assert np.array_equal(pa.cpu().numpy(), pb.cpu().numpy())
    assert la.item() == lb.item()
    assert np.array_equal(dxa.cpu().numpy(), dxb.cpu().numpy())
    assert np.isfinite(grad.cpu().numpy()).all() and float(grad.abs().max()) > 0


@pytest.mark.parametrize("precision", [0, 1])
@pytest.mark.parametrize("stationary", [0, -1])
def test_group_by_group_gradient_is_the_same_gradient(precision, stationary):
    """ftp_step_grad_groups reports every executed group's slice of the gradient once, last group first, and
    leaves bit for bit the gradient, loss and input gradient of ftp_step_grad; the slices, handed to the
    overlapped exchange at world size 1, give the update of ftp_step."""
    from paper_2409_09083_b200 import dp
    wl = Y8.with_(groups=((1, 4), (5, 8)))
    x, params, target = synth.draw(wl, bias_std=0.1)
    lr = 0.05
    plan = ftp.ftp_plan(wl.layers, wl.N, wl.C, wl.H, wl.W, wl.grid, wl.groups, precision=precision, stationary=stationary)
    ws = plan.new_workspace()
    xd, td = torch.from_numpy(x).cuda(), torch.from_numpy(target).cuda()
    pd = torch.from_numpy(params.copy()).cuda()
    ga, gb = torch.full_like(pd, float("nan")), torch.full_like(pd, float("nan"))
    la, lb = torch.zeros(1, device="cuda"), torch.zeros(1, device="cuda")
    dxa, dxb = torch.empty_like(xd), torch.empty_like(xd)
    ftp.ftp_step_grad(plan, xd, pd, ga, ws, target=td, loss_out=la, dx=dxa)
    ex = dp.OverlappedExchange(gb, 1, all_reduce=None)
    ftp.ftp_step_grad_groups(plan, xd, pd, gb, ws, ex.ready, target=td, loss_out=lb, dx=dxb)
    plan.check(ws)
    groups = [g for g, _, c in ex.slices]
    assert groups == sorted(groups, reverse=True) and len(set(groups)) == len(groups)
    assert len(groups) == len(plan.exec_groups())                       # every executed group of this stack holds a conv
    assert sum(c for _, _, c in ex.slices) == plan.param_floats
    assert np.array_equal(ga.cpu().numpy(), gb.cpu().numpy())
    assert la.item() == lb.item() and np.array_equal(dxa.cpu().numpy(), dxb.cpu().numpy())
    ex.finish(lr, lambda g, lr_eff: ftp.ftp_sgd(pd, g, lr_eff))
    pa = torch.from_numpy(params.copy()).cuda()
    ftp.ftp_step(plan, xd, pa, lr, ws, target=td)
    torch.cuda.synchronize()
    assert np.array_equal(pa.cpu().numpy(), pd.cpu().numpy())

    def boom(group, begin, count):
        raise KeyError("from the callback")
    with pytest.raises(KeyError):                                        # an exception in the callback surfaces after the call
        ftp.ftp_step_grad_groups(plan, xd, pd, gb, ws, boom, target=td)
    torch.cuda.synchronize()


def test_two_half_batches_reproduce_the_full_batch_update():
    """Data-parallel arithmetic on one GPU: the gradients of the two halves of a batch (ftp_step_grad on
    each, as two ranks would), summed and applied by ftp_sgd with lr / 2, equal the full-batch update
    within 1e-5 (each half's loss is the mean over its own images, so the full-batch gradient is the
    mean of the two)."""
    wl = Y8.with_(N=4)
    x, params, target = synth.draw(wl, bias_std=0.1)
    lr = 0.05
    full = ftp.ftp_plan(wl.layers, 4, wl.C, wl.H, wl.W, wl.grid, wl.groups)
    half = ftp.ftp_plan(wl.layers, 2, wl.C, wl.H, wl.W, wl.grid, wl.groups)
    wsf, wsh = full.new_workspace(), half.new_workspace()
    pf = torch.from_numpy(params.copy()).cuda()
    ftp.ftp_step(full, torch.from_numpy(x).cuda(), pf, lr, wsf, target=torch.from_numpy(target).cuda())
    ph = torch.from_numpy(params.copy()).cuda()
    total = torch.zeros_like(ph)
    for lo in (0, 2):
        g = torch.empty_like(ph)
        ftp.ftp_step_grad(half, torch.from_numpy(x[lo:lo + 2]).cuda(), ph, g, wsh,
                          target=torch.from_numpy(target[lo:lo + 2]).cuda())
        total += g                                                    # what the all-reduce does across ranks
    ftp.ftp_sgd(ph, total, lr / 2)
    torch.cuda.synchronize()
    upd_full = pf.cpu().numpy().astype(np.float64) - params
    upd_half = ph.cpu().numpy().astype(np.float64) - params
    assert np.abs(upd_full).max() > 0
    assert rel_err(upd_half, upd_full) <= 1e-5


def _random_workload(rng):
    """A small random stack of conv (1x1 / 3x3 / 5x5, 1-40 channels) and pool layers with a random
    batch, extent, tile grid and grouping profile."""
    layers, c = [], int(rng.integers(1, 6))
    cin0, h, w = c, int(rng.integers(3, 9)) * 4, int(rng.integers(3, 9)) * 4
    hh, ww = h, w
    for _ in range(int(rng.integers(1, 5))):
        if layers and layers[-1].kind == "conv" and hh % 2 == 0 and ww % 2 == 0 and min(hh, ww) >= 8 and rng.random() < 0.5:
            layers.append(pool()); hh //= 2; ww //= 2
        else:
            co = int(rng.choice([1, 3, 8, 13, 24, 40]))
            layers.append(conv(c, co, int(rng.choice([1, 3, 3, 3, 5])))); c = co
    cuts = sorted(set(int(v) for v in rng.integers(1, len(layers) + 1, size=2)) | {len(layers)})
    groups, a = [], 1
    for b in cuts:
        groups.append((a, b)); a = b + 1
    grid = (int(rng.integers(1, min(4, hh) + 1)), int(rng.integers(1, min(4, ww) + 1)))
    return W("rnd", tuple(layers), int(rng.integers(1, 4)), cin0, h, w, grid, tuple(groups), x_dist="normal")


@pytest.mark.gpu
@pytest.mark.parametrize("seed", range(24))
def test_random_small_stacks_match_oracle(seed):
    """Random layer stacks, shapes, grids and profiles under the planner's defaults (time-model cuts,
    refined backward split, staged filters and deltas) and, every third case, with forced sub-tiling.
    Dyadic values and slope 0.5 as in the mid-size cases: the forward is exact in fp32, so both sides
    take the same leaky-ReLU and arg-max decisions (ties included: first maximum in window order)."""
    rng = np.random.default_rng(1000 + seed)
    wl = synth.with_slope(_random_workload(rng), 0.5)
    opts = dict(max_subtile=int(rng.integers(2, 6))) if seed % 3 == 2 else {}
    x, params, target = synth.draw_dyadic(wl, nnz=3)
    ref = run_oracle(wl, x, params, target=target)
    got = run_gpu(wl, x, params, target=target, **opts)
    assert np.array_equal(got["y"].astype(np.float64), ref["y"]), wl
    assert rel_err(got["dx"], ref["dx"]) <= FP32_TOL, wl
    assert rel_err(got["dparams"], ref["dparams"]) <= FP32_TOL, wl
