"""Seeded synthetic workloads: layer stacks, shapes and random tensors.

This module holds no arithmetic of the method.  It describes the YOLOv2-style
early-layer stacks the benchmark and the tests run on and draws their inputs,
targets and initial parameters from NumPy's seeded generator, so the CUDA
library and the CPU oracle can be handed the very same values.  The paper
validates on "the first 16 layers of Yolov2" (Section 5) without listing the
layers, the input resolution, the data or the loss; the stacks below are the
public YOLOv2 early layers without batch-norm, the inputs are U[0,1) or N(0,1)
noise of the stated shapes, and the loss is mean-squared error against an
N(0,1) target.
"""
from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np


@dataclass(frozen=True)
class Layer:
    kind: str            # "conv" or "pool"
    cin: int = 0
    cout: int = 0
    k: int = 2
    stride: int = 2
    pad: int = 0
    leaky: float = 0.0


def conv(cin, cout, k, leaky=0.1) -> Layer:
    return Layer("conv", cin, cout, k, 1, k // 2, leaky)


def pool() -> Layer:
    return Layer("pool", 0, 0, 2, 2, 0, 0.0)


def stack_tiny() -> List[Layer]:
    return [conv(3, 8, 3), pool(), conv(8, 16, 3)]


def stack_yolo8() -> List[Layer]:
    return [conv(3, 32, 3), pool(), conv(32, 64, 3), pool(),
            conv(64, 128, 3), conv(128, 64, 1), conv(64, 128, 3), pool()]


def stack_yolo16() -> List[Layer]:
    return stack_yolo8() + [
        conv(128, 256, 3), conv(256, 128, 1), conv(128, 256, 3), pool(),
        conv(256, 512, 3), conv(512, 256, 1), conv(256, 512, 3), conv(512, 256, 1)]


@dataclass(frozen=True)
class Workload:
    name: str
    layers: Tuple[Layer, ...]
    N: int
    C: int
    H: int
    W: int
    grid: Tuple[int, int]                    # (tiles along y, tiles along x)
    groups: Tuple[Tuple[int, int], ...]      # 1-based inclusive layer ranges
    x_dist: str = "uniform"                  # "uniform" U[0,1) or "normal" N(0,1)
    lr: float = 1e-3
    seed: int = 0

    def with_(self, **kw) -> "Workload":
        d = dict(self.__dict__)
        d.update(kw)
        return Workload(**d)


def workload(name: str) -> Workload:
    """The benchmark configurations: C0 tiny, C1 8-layer one group 3x3 grid,
    C2 8-layer two groups 4x4 grid, C3 16-layer three groups 5x5 grid."""
    if name == "C0":
        return Workload("C0", tuple(stack_tiny()), 1, 3, 32, 32, (2, 2), ((1, 3),),
                        x_dist="normal")
    if name == "C1":
        return Workload("C1", tuple(stack_yolo8()), 4, 3, 416, 416, (3, 3), ((1, 8),))
    if name == "C2":
        return Workload("C2", tuple(stack_yolo8()), 8, 3, 416, 416, (4, 4),
                        ((1, 4), (5, 8)))
    if name == "C3":
        return Workload("C3", tuple(stack_yolo16()), 16, 3, 608, 608, (5, 5),
                        ((1, 4), (5, 8), (9, 16)))
    raise KeyError(name)


def groups_per_maxpool(layers) -> Tuple[Tuple[int, int], ...]:
    """Group profile that closes a group after every pooling layer."""
    out, first = [], 1
    for i, l in enumerate(layers, start=1):
        if l.kind == "pool" or i == len(layers):
            out.append((first, i))
            first = i + 1
    return tuple(out)


def groups_per_layer(layers) -> Tuple[Tuple[int, int], ...]:
    return tuple((i, i) for i in range(1, len(layers) + 1))


def map_shapes(layers, C, H, W):
    """(C, H, W) of X_1 .. X_{L+1}."""
    shapes = [(C, H, W)]
    for l in layers:
        c, h, w = shapes[-1]
        shapes.append((l.cout, h, w) if l.kind == "conv" else (c, h // 2, w // 2))
    return shapes


def param_count(layers) -> int:
    return sum(l.cout * l.cin * l.k * l.k + l.cout for l in layers if l.kind == "conv")


def forward_macs_per_image(layers, C, H, W) -> int:
    """Multiply-accumulates of one untiled forward pass over one image."""
    shapes = map_shapes(layers, C, H, W)
    return sum(l.cout * l.cin * l.k * l.k * shapes[i + 1][1] * shapes[i + 1][2]
               for i, l in enumerate(layers) if l.kind == "conv")


def draw(wl: Workload, bias_std: float = 0.0, N: Optional[int] = None):
    """x, flat params (filter [cout][cin][k][k] then bias [cout] per conv
    layer; He-normal filters, std = sqrt(2 / (cin k^2))), and an N(0,1)
    target of the last map's shape.  All float32, drawn in a fixed order from
    default_rng(seed).  bias_std > 0 gives non-zero biases (used to expose
    padding mistakes); the configurations themselves use zero bias."""
    rng = np.random.default_rng(wl.seed)
    n = wl.N if N is None else N
    shape = (n, wl.C, wl.H, wl.W)
    if wl.x_dist == "normal":
        x = rng.standard_normal(shape, dtype=np.float32)
    else:
        x = rng.random(shape, dtype=np.float32)
    parts = []
    for l in wl.layers:
        if l.kind != "conv":
            continue
        std = np.sqrt(2.0 / (l.cin * l.k * l.k))
        parts.append((rng.standard_normal(l.cout * l.cin * l.k * l.k) * std)
                     .astype(np.float32))
        parts.append((rng.standard_normal(l.cout) * bias_std).astype(np.float32))
    params = np.concatenate(parts)
    c, h, w = map_shapes(wl.layers, wl.C, wl.H, wl.W)[-1]
    target = rng.standard_normal((n, c, h, w), dtype=np.float32)
    return x, params, target


def with_slope(wl: Workload, slope: float) -> Workload:
    """Same workload with another leaky-ReLU slope on every conv layer."""
    layers = tuple(Layer(l.kind, l.cin, l.cout, l.k, l.stride, l.pad, slope if l.kind == "conv" else 0.0)
                   for l in wl.layers)
    return wl.with_(layers=layers)


def draw_dyadic(wl: Workload, nnz: int = 3, N: Optional[int] = None):
    """Inputs whose forward pass is exact in fp32 whatever the summation order:
    integer pixels in [-3, 3], filters with `nnz` non-zero taps of value +-1 per
    output channel, biases in {-0.5, 0, 0.5}.  With a dyadic leaky slope (use
    with_slope(wl, 0.5)) every activation is a small multiple of a power of
    two, so fp32 and fp64 agree bit for bit and every arg-max and sign decision
    is the same on both sides (exact ties included).  The target is N(0,1)."""
    rng = np.random.default_rng(wl.seed + 7919)
    n = wl.N if N is None else N
    x = rng.integers(-3, 4, size=(n, wl.C, wl.H, wl.W)).astype(np.float32)
    parts = []
    for l in wl.layers:
        if l.kind != "conv":
            continue
        fan = l.cin * l.k * l.k
        F = np.zeros((l.cout, fan), dtype=np.float32)
        for co in range(l.cout):
            idx = rng.choice(fan, size=min(nnz, fan), replace=False)
            F[co, idx] = rng.choice(np.array([-1.0, 1.0], dtype=np.float32), size=idx.size)
        parts.append(F.ravel())
        parts.append(rng.integers(-1, 2, size=l.cout).astype(np.float32) * 0.5)
    params = np.concatenate(parts)
    c, h, w = map_shapes(wl.layers, wl.C, wl.H, wl.W)[-1]
    target = rng.standard_normal((n, c, h, w), dtype=np.float32)
    return x, params, target


def draw_integer_relu(wl: Workload, N: Optional[int] = None):
    """Inputs whose forward pass is exact in bfloat16 AND in fp32, for stacks with
    slope 0 on every conv (use with_slope(wl, 0.0)): integer pixels in [0, 3];
    every output channel's filter has exactly one tap of +1 and one of -1;
    biases in {0, 1}.  A conv output is then a - b + bias for two values a, b of
    its input map (or the zero padding), so with M the largest input value every
    activation is an integer in [0, M + 1] after the ReLU: at most 3 + (number of
    conv layers) over a whole stack, far below 256, the largest run of integers
    that 8 significant bits hold.  A path that stores its maps in bf16 and one
    that keeps them in fp64 therefore see identical maps, and every arg-max and
    sign decision (exact ties included) is the same on both sides.  The target
    is N(0,1)."""
    rng = np.random.default_rng(wl.seed + 104729)
    n = wl.N if N is None else N
    x = rng.integers(0, 4, size=(n, wl.C, wl.H, wl.W)).astype(np.float32)
    parts = []
    for l in wl.layers:
        if l.kind != "conv":
            continue
        fan = l.cin * l.k * l.k
        F = np.zeros((l.cout, fan), dtype=np.float32)
        for co in range(l.cout):
            if fan >= 2:
                plus, minus = rng.choice(fan, size=2, replace=False)
                F[co, plus], F[co, minus] = 1.0, -1.0
            else:
                F[co, 0] = 1.0
        parts.append(F.ravel())
        parts.append(rng.integers(0, 2, size=l.cout).astype(np.float32))
    params = np.concatenate(parts)
    c, h, w = map_shapes(wl.layers, wl.C, wl.H, wl.W)[-1]
    target = rng.standard_normal((n, c, h, w), dtype=np.float32)
    return x, params, target
