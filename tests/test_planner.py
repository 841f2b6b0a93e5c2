"""Host logic: the C-ABI library loads and exports what include/ftp.h declares, the planner
reproduces Eq. (1)/(2) and the hand-derived spans, and bad arguments turn into error codes.
No GPU is touched."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2409_09083_b200 as ftp
from oracle import spans
from paper_2409_09083_b200 import binding, synth
from test_spans_oracle import STACKS, read_golden

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "ftp.h")).read()
    names = set(re.findall(r"\b(ftp_[a-z_]+)\s*\(", header))
    assert {"ftp_plan_create", "ftp_forward", "ftp_backward", "ftp_step"} <= names
    lib = ctypes.CDLL(os.path.join(ROOT, "paper_2409_09083_b200", "libftp.so"))
    for n in sorted(names):
        assert hasattr(lib, n), f"{n} declared in ftp.h but not exported"


def test_binding_has_the_same_names():
    for n in ("ftp_plan", "ftp_forward", "ftp_backward", "ftp_step", "ftp_strerror"):
        assert callable(getattr(ftp, n))


@pytest.mark.parametrize("row", read_golden())
def test_region_matches_hand_derived_spans(row):
    stack, first, last, extent, parts, tile, sp = row
    layers = STACKS[stack]()
    # put the group under test into a valid profile over the whole stack
    groups = []
    if first > 1:
        groups.append((1, first - 1))
    groups.append((first, last))
    if last < len(layers):
        groups.append((last + 1, len(layers)))
    size = {"tiny": 32, "yolo8": 416, "yolo16": 608}[stack]
    plan = ftp.ftp_plan(layers, 1, 3, size, size, (parts, parts), groups)
    gi = groups.index((first, last))
    for m, want in zip(range(last + 1, first - 1, -1), sp):
        x1, y1, x2, y2 = plan.region(0, gi, m, tile, tile)
        assert (x1, x2) == want and (y1, y2) == want
        assert plan.region(1, gi, m, tile, tile) == (x1, y1, x2, y2)


@pytest.mark.parametrize("name", ["C0", "C1", "C2", "C3"])
def test_region_equals_span_recursion_on_all_tiles(name):
    wl = synth.workload(name)
    plan = ftp.ftp_plan(wl.layers, 1, wl.C, wl.H, wl.W, wl.grid, wl.groups)
    shapes = synth.map_shapes(wl.layers, wl.C, wl.H, wl.W)
    for gi, (first, last) in enumerate(wl.groups):
        layers = list(wl.layers[first - 1:last])
        oh, ow = shapes[last][1], shapes[last][2]
        ys = [spans.forward_spans(layers, oh, c) for c in spans.equal_partition(oh, wl.grid[0])]
        xs = [spans.forward_spans(layers, ow, c) for c in spans.equal_partition(ow, wl.grid[1])]
        for ty in range(wl.grid[0]):
            for tx in range(wl.grid[1]):
                for m in range(first, last + 2):
                    x1, y1, x2, y2 = plan.region(0, gi, m, ty, tx)
                    assert (y1, y2) == ys[ty][m - first] and (x1, x2) == xs[tx][m - first]


def test_gather_form_equals_eq2_for_conv_stack():
    layers = [synth.conv(3, 4, 3), synth.conv(4, 4, 5), synth.conv(4, 2, 1)]
    plan = ftp.ftp_plan(layers, 1, 3, 40, 40, (4, 4), [(1, 3)])
    for t in range(4):
        a, b = spans.equal_partition(40, 4)[t]
        for m, l in zip(range(2, 5), layers):
            a, b = spans.eq2_conv(a, b, l.k, 1)
            a, b = spans.clamp(a, b, 40)
            x1, y1, x2, y2 = plan.region(2, 0, m, t, t)
            assert (x1, x2) == (a, b) and (y1, y2) == (a, b)


def test_exec_groups_refine_the_requested_profile():
    for name in ["C0", "C1", "C2", "C3"]:
        wl = synth.workload(name)
        plan = ftp.ftp_plan(wl.layers, wl.N, wl.C, wl.H, wl.W, wl.grid, wl.groups)
        eg = plan.exec_groups()
        assert eg[0][0] == 1 and eg[-1][1] == len(wl.layers)
        for (a, b), (c, d) in zip(eg, eg[1:]):
            assert c == b + 1
        starts = {g[0] for g in eg}
        assert {g[0] for g in wl.groups} <= starts        # every requested boundary is kept
        assert plan.redundancy >= 1.0
        assert plan.param_floats == synth.param_count(wl.layers)
        for gi in range(len(eg)):
            for pass_ in (0, 1):
                st = plan.subtiles(pass_, gi)
                assert st["smem_bytes"] <= 225 * 1024 and st["blocks"] >= 1
                if not plan.group_mode(gi)[0]:                # fused stacks: sub-tiles refine the user tiles
                    assert st["rows"] >= wl.grid[0] and st["cols"] >= wl.grid[1]
    # C2's requested groups fit as they are; by default they are executed as conv(+pool) pairs
    wl = synth.workload("C2")
    mk = lambda **kw: ftp.ftp_plan(wl.layers, wl.N, wl.C, wl.H, wl.W, wl.grid, wl.groups, **kw).exec_groups()
    assert mk(max_group_convs=-1) == list(wl.groups)
    assert mk(max_group_convs=2) == [(1, 2), (3, 4), (5, 6), (7, 8)]
    assert mk(max_group_convs=1) == [(1, 2), (3, 4), (5, 5), (6, 6), (7, 8)]
    assert mk(cost_model=-1) == [(1, 2), (3, 4), (5, 6), (7, 8)]


def _conv_counts(layers, groups):
    return [sum(1 for l in layers[a - 1:b] if l.kind == "conv") for a, b in groups]


def test_cost_model_cuts_are_valid_profiles():
    """The model only moves cuts inside requested groups: executed groups stay contiguous, keep every
    requested boundary, hold one to three convs and never part a conv from the pool after it; an
    explicit max_group_convs or cost_model=-1 leaves the fixed rule alone."""
    for name in ["C1", "C2", "C3"]:
        wl = synth.workload(name)
        for prec in (0, 1):
            mk = lambda **kw: ftp.ftp_plan(wl.layers, wl.N, wl.C, wl.H, wl.W, wl.grid, wl.groups, precision=prec, **kw)
            fixed = mk(cost_model=-1).exec_groups()
            assert mk(max_group_convs=2).exec_groups() == fixed
            for plan in (mk(), mk(cost_model=1)):
                eg = plan.exec_groups()
                assert eg[0][0] == 1 and eg[-1][1] == len(wl.layers)
                assert all(c == b + 1 for (a, b), (c, d) in zip(eg, eg[1:]))
                assert {g[0] for g in wl.groups} <= {g[0] for g in eg}
                assert all(1 <= n <= 3 for n in _conv_counts(wl.layers, eg))
                for a, b in eg[:-1]:
                    assert not (wl.layers[b - 1].kind == "conv" and wl.layers[b].kind == "pool")
                # the model's own estimate of what it chose is never worse than that of the fixed rule's cuts
                est = lambda pl: sum(pl.cost(ps, g, a > 1)[1] for g, (a, b) in enumerate(pl.exec_groups()) for ps in (0, 1))
                assert est(plan) <= est(mk(cost_model=-1)) * (1 + 1e-9)


def test_cost_terms_of_a_single_conv_by_hand():
    """One 3x3 conv 8 -> 16 on a 16 x 16 map, one image, one tile, fp32.  The forward pass cuts the
    map into R x Q stacks that all run side by side, so each term is that of one average stack: at
    most 2 x 4 x 16 = 128 thread tasks of 4 rows x 8 channels, i.e. one round of 512, which counts
    512 x 32 x 8 x 9 multiply-accumulates; the filters, 9 x 8 x 16 floats; the map term, the input
    spans (own rows and columns plus a halo of 1 where the map goes on) plus the 16 x 16 x 16 output."""
    layers = [synth.conv(8, 16, 3)]
    plan = ftp.ftp_plan(layers, 1, 8, 16, 16, (1, 1), ((1, 1),))
    st = plan.subtiles(0, 0)
    R, Q = st["rows"], st["cols"]
    assert 16 % R == 0 and 16 % Q == 0 and R * Q <= 148
    t, est = plan.cost(0, 0, True)
    assert t[0] == pytest.approx(512 * 32 * 8 * 9 / 1e6) and t[1] == 0
    assert t[2] == pytest.approx(9 * 8 * 16 * 4 / 1e6)
    in_floats = 8 * (16 + 2 * (R - 1)) * (16 + 2 * (Q - 1))
    assert t[3] == pytest.approx((in_floats + 16 * 256) * 4 / 1e6 / (R * Q))
    assert t[4] == 1 and t[5] == pytest.approx(16 * 256 / 1e6 / (R * Q)) and t[7] == 1
    assert est > 0
    # backward: the one image's tile is cut into Rb x Qb stacks, one per block, so again every term is
    # that of one stack on the critical path
    sb = plan.subtiles(1, 0)
    Rb, Qb = sb["rows"], sb["cols"]
    assert sb["blocks"] == Rb * Qb <= 148 and 16 % Rb == 0 and 16 % Qb == 0
    tb, estb = plan.cost(1, 0, True)
    assert tb[0] == pytest.approx(256 * 8 * 16 * 9 / 1e6 / (Rb * Qb))   # filter gradient: plain count
    assert tb[1] == pytest.approx(512 * 32 * 16 * 9 / 1e6)           # input delta: at most 1 x 4 x 16 = 64 tasks, one round, 16 delta channels each
    assert tb[4] == pytest.approx((9 * 8 * 16 + 16) * 4 / 1e6)       # the stack's partial set
    assert plan.cost(1, 0, False)[0][1] == 0                         # no input delta asked for
    # twice the batch: twice the stacks on as many blocks, so every term but the launch doubles at most
    plan2 = ftp.ftp_plan(layers, 2, 8, 16, 16, (1, 1), ((1, 1),))
    t2, est2 = plan2.cost(0, 0, True)
    assert est2 >= est and all(b <= 2 * a + 1e-12 for a, b in zip(t[:7], t2[:7]))
    for bad in (dict(pass_=2, group=0), dict(pass_=0, group=1), dict(pass_=0, group=-1)):
        with pytest.raises(binding.FtpError) as e:
            plan.cost(bad["pass_"], bad["group"])
        assert e.value.code == -1


def test_strict_groups_keeps_or_refuses():
    wl = synth.workload("C1")
    plan = ftp.ftp_plan(wl.layers, wl.N, wl.C, wl.H, wl.W, wl.grid, wl.groups, strict_groups=True)
    assert plan.exec_groups() == [(1, 8)]
    wl = synth.workload("C3")
    with pytest.raises(binding.FtpError) as e:
        ftp.ftp_plan(wl.layers, wl.N, wl.C, wl.H, wl.W, wl.grid, wl.groups, strict_groups=True)
    assert e.value.code == -5


def _code(fn):
    with pytest.raises(binding.FtpError) as e:
        fn()
    return e.value.code


def test_argument_errors_are_codes_not_crashes():
    L = synth.stack_tiny()
    ok = dict(N=1, C=3, H=32, W=32)
    mk = lambda layers=L, grid=(2, 2), groups=((1, 3),), **kw: ftp.ftp_plan(
        layers, kw.get("N", 1), kw.get("C", 3), kw.get("H", 32), kw.get("W", 32), grid, groups,
        **{k: v for k, v in kw.items() if k not in ok})
    assert _code(lambda: mk(N=0)) == -1
    assert _code(lambda: mk(grid=(0, 2))) == -1
    assert _code(lambda: mk(C=4)) == -2                                   # channel mismatch
    assert _code(lambda: mk(layers=[synth.Layer("conv", 3, 8, 4, 1, 2, 0.1)], groups=((1, 1),))) == -2   # even kernel
    assert _code(lambda: mk(layers=[synth.Layer("conv", 3, 8, 3, 2, 1, 0.1)], groups=((1, 1),))) == -2   # stride 2
    assert _code(lambda: mk(layers=[synth.Layer("conv", 3, 8, 3, 1, 0, 0.1)], groups=((1, 1),))) == -2   # pad != k/2
    assert _code(lambda: mk(layers=[synth.pool()], groups=((1, 1),), H=31)) == -2                        # odd extent
    assert _code(lambda: mk(groups=((1, 2),))) == -4                      # not covering
    assert _code(lambda: mk(groups=((1, 1), (3, 3)))) == -4               # gap
    assert _code(lambda: mk(groups=((2, 3), (1, 1)))) == -4               # order
    assert _code(lambda: mk(grid=(17, 2))) == -3                          # more tiles than output rows
    assert _code(lambda: mk(precision=5)) == -1
    assert "shared memory" in ftp.ftp_strerror(-5)
    assert ftp.ftp_strerror(0) == "ok"


def test_null_pointers_are_rejected_on_the_host():
    wl = synth.workload("C0")
    plan = ftp.ftp_plan(wl.layers, wl.N, wl.C, wl.H, wl.W, wl.grid, wl.groups)
    lib = binding._lib
    assert lib.ftp_forward(plan._h, None, None, None, None, None) == -1
    assert lib.ftp_backward(plan._h, None, None, None, None, None, None, None) == -1
    assert lib.ftp_step(plan._h, None, None, None, None, 0.0, None, None, None, None) == -1
    assert lib.ftp_forward(None, None, None, None, None, None) == -1
    assert plan.launch_count() == 0


def test_delta_staging_is_granted_only_where_it_fits():
    """fp32 backward: a group with a fused conv+pool gets the 16-channel staging area when the
    sub-tile split leaves room, a half or a quarter of it or none otherwise; groups without such a
    layer report 0.  (Fixed-rule groups and the first split that fits, so that only the shared-memory
    limit varies; the GPU invariance test runs the two reduced settings.)"""
    wl = synth.Workload("y8", tuple(synth.stack_yolo8()), 2, 3, 64, 96, (2, 2), ((1, 8),))
    mk = lambda **kw: ftp.ftp_plan(wl.layers, wl.N, wl.C, wl.H, wl.W, wl.grid, wl.groups, max_subtile=64, cost_model=-1, **kw)
    full, part, none = mk(), mk(smem_bytes=120000), mk(smem_bytes=100000)
    for plan in (full, part, none):
        assert plan.exec_groups() == [(1, 2), (3, 4), (5, 6), (7, 8)]
    staging = lambda plan: [plan.delta_staging(g) for g in range(4)]
    assert staging(full) == [16, 16, 0, 16]
    assert staging(part) == [4, 8, 0, 16]
    assert staging(none) == [0, 0, 0, 16]
    for g in (0, 1):                                                        # refused rather than paid for with smaller sub-tiles
        assert none.subtiles(1, g)["rows"] == full.subtiles(1, g)["rows"] and none.subtiles(1, g)["cols"] == full.subtiles(1, g)["cols"]
    for plan in (full, part, none):
        for gi in range(4):
            assert plan.subtiles(1, gi)["smem_bytes"] <= 225 * 1024
    assert ftp.ftp_plan(wl.layers, wl.N, wl.C, wl.H, wl.W, wl.grid, wl.groups, precision=1).delta_staging(0) == 0   # the bf16 path has no such area
    with pytest.raises(binding.FtpError):
        full.delta_staging(99)


def test_backward_split_is_refined_for_balance():
    """The backward blocks share all sub-tile stacks of the batch evenly; the planner may cut finer
    than the largest sub-tiles that fit when that evens out the stacks per block.  C1, fp32: layer 5
    alone fits as 3 x 2 sub-tiles per tile, i.e. 4 images x 54 = 216 stacks on 148 blocks (two for
    68 of the blocks, one for the rest); 4 x 2 gives 288 smaller stacks, two for nearly every block."""
    wl = synth.workload("C1")
    layers = wl.layers[4:5]
    mk = lambda **kw: ftp.ftp_plan(layers, wl.N, 64, 104, 104, (3, 3), ((1, 1),), stationary=-1, **kw)   # as fused stacks
    first_fit, refined = mk(max_subtile=64).subtiles(1, 0), mk().subtiles(1, 0)
    assert (first_fit["rows"], first_fit["cols"]) == (9, 6)
    assert (refined["rows"], refined["cols"]) == (12, 6)
    assert first_fit["blocks"] == refined["blocks"] == 148
    assert -(-4 * 9 * 6 // 148) == -(-4 * 12 * 6 // 148) == 2        # two stacks on the busiest block either way, smaller ones when refined
    est = lambda **kw: mk(**kw).cost(1, 0, True)[1]
    assert est() < 0.97 * est(max_subtile=64)
    # fewer stacks than blocks: one block per stack
    small = ftp.ftp_plan(layers, 1, 64, 16, 16, (2, 2), ((1, 1),), max_subtile=64, stationary=-1).subtiles(1, 0)
    assert small["blocks"] == small["rows"] * small["cols"]


def test_bf16_plans_run_conv_layers_as_groups_of_their_own():
    """bf16 path: by default every conv layer the banded tensor-core kernels can take (1x1 / 3x3 window; the first
    layer as a 3x3 conv with few channels) is an executed group of its own (with its pool), reported as mode 2 with as
    many partial sets as its filter gradient has pixel shares; `stationary = -1` keeps the fused stacks; a window
    the kernels do not take stays fused."""
    for name in ["C1", "C2", "C3"]:
        wl = synth.workload(name)
        plan = ftp.ftp_plan(wl.layers, wl.N, wl.C, wl.H, wl.W, wl.grid, wl.groups, precision=ftp.FTP_BF16_FP32ACC)
        eg = plan.exec_groups()
        assert _conv_counts(list(wl.layers), eg) == [1] * len(eg)
        assert {g[0] for g in wl.groups} <= {g[0] for g in eg}
        for gi in range(len(eg)):
            mode, sets = plan.group_mode(gi)
            assert mode == 2 and 1 <= sets <= 148
        fused = ftp.ftp_plan(wl.layers, wl.N, wl.C, wl.H, wl.W, wl.grid, wl.groups, precision=ftp.FTP_BF16_FP32ACC, stationary=-1)
        assert all(fused.group_mode(gi)[0] == 0 for gi in range(len(fused.exec_groups())))
        assert plan.workspace_bytes < fused.workspace_bytes or name != "C3"     # no per-sub-tile delta blocks, fewer sets
    # a 5x5 layer stays a fused stack; the layers around it do not
    layers = (synth.conv(3, 16, 3), synth.conv(16, 16, 5), synth.conv(16, 32, 3))
    plan = ftp.ftp_plan(layers, 2, 3, 32, 32, (2, 2), ((1, 3),), precision=ftp.FTP_BF16_FP32ACC)
    modes = {g: plan.group_mode(i)[0] for i, g in enumerate(plan.exec_groups())}
    assert modes[(1, 1)] == 2 and modes[(3, 3)] == 2 and modes[(2, 2)] == 0, modes
    # a first layer with a 1x1 window reads the fp32 input: fused
    layers = (synth.conv(3, 16, 1), synth.conv(16, 16, 3))
    plan = ftp.ftp_plan(layers, 2, 3, 32, 32, (2, 2), ((1, 2),), precision=ftp.FTP_BF16_FP32ACC)
    modes = [plan.group_mode(i)[0] for i in range(len(plan.exec_groups()))]
    assert modes[0] == 0 and modes[-1] == 2, (plan.exec_groups(), modes)


def test_bf16_layers_wider_than_the_tensor_memory_run_banded_or_not_at_all():
    """bf16 path: a conv layer with more than 512 input or output channels (the 512 -> 1024 -> 512 layers behind the
    16-layer stack) is planned as a banded one-conv group; a plan that would put it into a fused stack (fused stacks
    only, a strict profile that fuses it, a 5x5 window) is refused with the layer error, not planned into a kernel
    that cannot hold it; the cost query of such a group answers; the fp32 path plans all of them."""
    conv, pool = synth.conv, synth.pool
    layers = (conv(3, 16, 3), pool(), conv(16, 512, 1), pool(), conv(512, 1024, 3), conv(1024, 512, 1))
    shape = (2, 3, 40, 56, (2, 2))
    bf16 = ftp.FTP_BF16_FP32ACC
    plan = ftp.ftp_plan(layers, *shape, ((1, 6),), precision=bf16)
    assert plan.exec_groups() == [(1, 2), (3, 4), (5, 5), (6, 6)]
    assert [plan.group_mode(i)[0] for i in range(4)] == [2, 2, 2, 2]
    for gi in range(4):
        for pass_ in (0, 1):
            terms, est = plan.cost(pass_, gi, True)
            assert np.isfinite(est) and est > 0 and np.all(np.isfinite(terms))
    assert _code(lambda: ftp.ftp_plan(layers, *shape, ((1, 6),), precision=bf16, stationary=-1)) == -2
    assert _code(lambda: ftp.ftp_plan(layers, *shape, ((1, 4), (5, 6)), precision=bf16, strict_groups=True)) == -2
    five = (conv(3, 16, 3), conv(16, 640, 5))
    assert _code(lambda: ftp.ftp_plan(five, 1, 3, 16, 16, (2, 2), ((1, 2),), precision=bf16)) == -2
    for kw in ({}, dict(stationary=-1), dict(strict_groups=True)):
        ftp.ftp_plan(layers, *shape, ((1, 4), (5, 6)), **kw)


def test_small_launches_of_the_row_convolution_use_half_size_blocks():
    """fp32 one-conv groups: a convolution launch of at most a round and a half of whole (256-thread, 16 row pairs)
    blocks is cut into 128-thread blocks of 8 row pairs (C1, batch 4, layer 5: 4 x 52 row pairs -> 26 tiles instead of
    13); larger launches and `stationary = 1` keep whole blocks."""
    wl = synth.workload("C1")
    plan = ftp.ftp_plan(wl.layers, wl.N, wl.C, wl.H, wl.W, wl.grid, wl.groups)
    gi = plan.exec_groups().index((5, 5))
    st = plan.subtiles(0, gi)
    assert st["rows"] == 26 and st["cols"] == 13 and st["blocks"] == 26 * 13 * 2 and st["smem_bytes"] == 32768
    whole = ftp.ftp_plan(wl.layers, wl.N, wl.C, wl.H, wl.W, wl.grid, wl.groups, stationary=1)
    st = whole.subtiles(0, whole.exec_groups().index((5, 5)))
    assert st["rows"] == 13 and st["blocks"] == 13 * 13 * 2
    big = synth.workload("C3")
    plan = ftp.ftp_plan(big.layers, big.N, big.C, big.H, big.W, big.grid, big.groups)
    st = plan.subtiles(0, plan.exec_groups().index((5, 5)))
    assert st["rows"] == (16 * 76 + 15) // 16
