"""Untiled fp64 training step: the plain definition the tiled method must equal.

TEST INFRASTRUCTURE ONLY.  The paper's tiling, fusing and grouping change where
and when values are computed, never which values (abstract: no loss of
accuracy; Section 4.1: per-tile filter gradients sum to the full gradient).
The oracle is therefore ordinary layer-by-layer training over whole maps.

Notation follows the paper: X_l is the input of layer l and X_{l+1} its output
(Section 4.1); layers are 1-based; maps[l-1] below holds X_l.

A layer is any object with attributes
    kind   "conv" or "pool"
    cin, cout, k, pad, leaky     (conv: stride 1, pad = k // 2)
    (pool: 2x2 window, stride 2, no padding)
Parameters travel as one flat fp64 vector: for each conv layer in order, the
filter [cout][cin][k][k] followed by the bias [cout].
"""
import ctypes

import numpy as np

from .build import build as _build

_lib = None
_D = ctypes.POINTER(ctypes.c_double)
_I = ctypes.POINTER(ctypes.c_int)


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(_build())
        _lib.orc_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    """Threads the C loops actually use (OpenMP max threads)."""
    return int(_load().orc_num_threads())


def _p(a):
    return a.ctypes.data_as(_D)


def _c(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def param_count(layers) -> int:
    return sum(l.cout * l.cin * l.k * l.k + l.cout for l in layers if l.kind == "conv")


def unpack_params(layers, params):
    """Flat vector -> list (per layer) of (F, b) for conv layers, None for pools."""
    params = np.asarray(params)
    out, o = [], 0
    for l in layers:
        if l.kind != "conv":
            out.append(None)
            continue
        nf = l.cout * l.cin * l.k * l.k
        F = params[o:o + nf].reshape(l.cout, l.cin, l.k, l.k)
        b = params[o + nf:o + nf + l.cout]
        o += nf + l.cout
        out.append((F, b))
    assert o == params.size, "parameter vector length does not match the layer list"
    return out


def pack_params(layers, per_layer):
    parts = []
    for l, fb in zip(layers, per_layer):
        if l.kind == "conv":
            parts += [np.asarray(fb[0]).ravel(), np.asarray(fb[1]).ravel()]
    return np.concatenate(parts) if parts else np.zeros(0)


def conv_forward(X, F, b, pad, slope):
    """Conv + bias + leaky ReLU (Section 4.1 forward). Returns (Z, Y)."""
    X, F, b = _c(X), _c(F), _c(b)
    N, Cin, H, W = X.shape
    Cout, Cin2, K, K2 = F.shape
    assert Cin == Cin2 and K == K2 and K % 2 == 1 and pad == K // 2
    Z = np.empty((N, Cout, H, W))
    Y = np.empty((N, Cout, H, W))
    _load().orc_conv_forward(_p(X), _p(F), _p(b), N, Cin, H, W, Cout, K, pad,
                             ctypes.c_double(slope), _p(Z), _p(Y))
    return Z, Y


def conv_backward(X, F, Z, dY, pad, slope):
    """Returns (dX, dF, db) for one conv layer (Section 4.1 backward)."""
    X, F, Z, dY = _c(X), _c(F), _c(Z), _c(dY)
    N, Cin, H, W = X.shape
    Cout, _, K, _ = F.shape
    dZ = np.empty_like(Z)
    dX = np.empty_like(X)
    dF = np.empty_like(F)
    db = np.empty(Cout)
    _load().orc_conv_backward(_p(X), _p(F), _p(Z), _p(dY), N, Cin, H, W, Cout, K,
                              pad, ctypes.c_double(slope), _p(dZ), _p(dX), _p(dF),
                              _p(db))
    return dX, dF, db


def maxpool_forward(X):
    X = _c(X)
    N, C, H, W = X.shape
    assert H % 2 == 0 and W % 2 == 0, "2x2/2 pooling needs even extents"
    Y = np.empty((N, C, H // 2, W // 2))
    arg = np.empty((N, C, H // 2, W // 2), dtype=np.int32)
    _load().orc_maxpool_forward(_p(X), N, C, H, W, _p(Y), arg.ctypes.data_as(_I))
    return Y, arg


def maxpool_backward(dY, arg, in_shape):
    dY = _c(dY)
    N, C, H, W = in_shape
    arg = np.ascontiguousarray(arg, dtype=np.int32)
    dX = np.empty(in_shape)
    _load().orc_maxpool_backward(_p(dY), arg.ctypes.data_as(_I), N, C, H, W, _p(dX))
    return dX


def round_bf16(a):
    """Nearest bfloat16 value (8 significant bits, ties to even) of every entry,
    returned in fp64.  Written from the format's definition: the significand
    m in [0.5, 1) of a = m * 2^e is rounded to a multiple of 2^-8."""
    a = np.asarray(a, dtype=np.float64)
    m, e = np.frexp(a)
    return np.ldexp(np.rint(m * 256.0) / 256.0, e)


def forward(layers, x, params, store=None):
    """Whole-map forward pass. Returns (maps, tape): maps[l-1] = X_l for
    l = 1..L+1, tape[l-1] = what layer l's backward needs.

    store="bf16" models a path that keeps its feature maps in bfloat16: the
    output of every conv layer (after the leaky ReLU) is rounded to bf16 before
    anything else reads it, so pooling and its arg-max act on the stored
    values.  Arithmetic inside a layer stays exact.  The paper does not fix a
    storage precision; None (the default) keeps everything in fp64."""
    assert store in (None, "bf16")
    per = unpack_params(layers, np.asarray(params, dtype=np.float64))
    maps = [_c(x)]
    tape = []
    for l, fb in zip(layers, per):
        if l.kind == "conv":
            Z, Y = conv_forward(maps[-1], fb[0], fb[1], l.pad, l.leaky)
            if store:
                Y = round_bf16(Y)
            tape.append(Z)
            maps.append(Y)
        else:
            Y, arg = maxpool_forward(maps[-1])
            tape.append(arg)
            maps.append(Y)
    return maps, tape


def mse_loss(y, target):
    """L = mean over all elements of (y - t)^2 and dL/dy = 2 (y - t) / M."""
    y, target = _c(y), _c(target)
    diff = y - target
    M = diff.size
    return float(np.sum(diff * diff) / M), 2.0 * diff / M


def backward(layers, maps, tape, params, dy, store=None):
    """Whole-map backward pass from dL/dX_{L+1} = dy.
    Returns (dx, dparams flat, deltas) with deltas[l-1] = dL/dX_l.

    store="bf16" models a path that also keeps the delta in front of every
    conv layer's activation, dL/dZ = dL/dY * leaky'(Z), in bfloat16: it is
    rounded before the filter, bias and input gradients are formed from it."""
    assert store in (None, "bf16")
    per = unpack_params(layers, np.asarray(params, dtype=np.float64))
    L = len(layers)
    deltas = [None] * (L + 1)
    deltas[L] = _c(dy)
    grads = [None] * L
    for i in range(L - 1, -1, -1):
        l = layers[i]
        if l.kind == "conv" and store:
            dZ = round_bf16(deltas[i + 1] * np.where(tape[i] > 0.0, 1.0, l.leaky))
            dX, dF, db = conv_backward(maps[i], per[i][0], np.ones_like(dZ), dZ, l.pad, 1.0)
            grads[i] = (dF, db)
        elif l.kind == "conv":
            dX, dF, db = conv_backward(maps[i], per[i][0], tape[i], deltas[i + 1],
                                       l.pad, l.leaky)
            grads[i] = (dF, db)
        else:
            dX = maxpool_backward(deltas[i + 1], tape[i], maps[i].shape)
        deltas[i] = dX
    return deltas[0], pack_params(layers, grads), deltas


def step(layers, x, params, lr, target=None, dy=None, store=None):
    """One training cycle (forward, back-propagation, filter-gradient sum,
    update; Sections 3 and 4.1): plain SGD, w <- w - lr * dL/dw.

    Give either `target` (MSE loss) or `dy` (the loss delta at the last map).
    `store`: see forward / backward.
    Returns dict(loss, y, dx, dparams, new_params, maps, deltas).
    """
    params = np.asarray(params, dtype=np.float64)
    maps, tape = forward(layers, x, params, store)
    loss = None
    if dy is None:
        loss, dy = mse_loss(maps[-1], target)
    dx, dparams, deltas = backward(layers, maps, tape, params, dy, store)
    return dict(loss=loss, y=maps[-1], dx=dx, dparams=dparams,
                new_params=params - lr * dparams, maps=maps, deltas=deltas)
