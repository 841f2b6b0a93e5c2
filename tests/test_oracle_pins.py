"""Pins for the fp64 CPU oracle: it is checked against things other than itself
-- finite differences of the loss, a library convolution with autograd,
closed forms for constant inputs and hand-evaluated tiny cases -- so that a
dropped term, a flipped kernel, a swapped index or a wrong sign fails here."""
import numpy as np
import pytest
import torch
import torch.nn.functional as tF

from oracle import reference as orc
from paper_2409_09083_b200 import synth


def _tiny_net():
    return [synth.conv(2, 3, 3), synth.pool(), synth.conv(3, 4, 1), synth.conv(4, 2, 3)]


def _draw(layers, N, C, H, W, seed, bias=True):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((N, C, H, W))
    params = rng.standard_normal(orc.param_count(layers)) * 0.5
    if not bias:
        for (F, b) in [p for p in orc.unpack_params(layers, params) if p]:
            b[:] = 0
    shapes = synth.map_shapes(layers, C, H, W)
    target = rng.standard_normal((N,) + shapes[-1])
    return x, params, target


def _loss(layers, x, params, target):
    maps, _ = orc.forward(layers, x, params)
    return orc.mse_loss(maps[-1], target)[0]


def test_hand_evaluated_correlation_is_unflipped():
    # out[y,x] = sum_k F[ky,kx] * X[y+ky-1, x+kx-1], zero outside the map.
    X = np.arange(1.0, 10.0).reshape(1, 1, 3, 3)
    F = np.zeros((1, 1, 3, 3))
    F[0, 0, 0, 0] = 1.0       # reads the upper-left neighbour
    F[0, 0, 2, 2] = 2.0       # reads the lower-right neighbour
    F[0, 0, 1, 2] = -3.0      # reads the right neighbour
    Z, Y = orc.conv_forward(X, F, np.array([0.5]), 1, 0.1)
    # centre (1,1): 1*X[0,0] + 2*X[2,2] - 3*X[1,2] + 0.5 = 1 + 18 - 18 + 0.5
    assert Z[0, 0, 1, 1] == pytest.approx(1.5)
    # corner (0,0): upper-left is padding; 2*X[1,1] - 3*X[0,1] + 0.5 = 10 - 6 + 0.5
    assert Z[0, 0, 0, 0] == pytest.approx(4.5)
    # corner (2,2): 1*X[1,1] + 0.5 (both others are padding)
    assert Z[0, 0, 2, 2] == pytest.approx(5.5)
    # (0,2): right and upper-left are padding; lower-right too -> bias only
    assert Z[0, 0, 0, 2] == pytest.approx(0.5)
    # (2,0): 1*pad + 2*pad - 3*X[2,1] + 0.5 = -24 + 0.5 ; leaky applies
    assert Z[0, 0, 2, 0] == pytest.approx(-23.5)
    assert Y[0, 0, 2, 0] == pytest.approx(-2.35)
    assert Y[0, 0, 1, 1] == pytest.approx(1.5)


def test_brute_force_python_loops_two_channels():
    rng = np.random.default_rng(3)
    X = rng.standard_normal((2, 2, 4, 5))
    F = rng.standard_normal((3, 2, 3, 3))
    b = rng.standard_normal(3)
    Z, _ = orc.conv_forward(X, F, b, 1, 0.1)
    for n in range(2):
        for co in range(3):
            for y in range(4):
                for x in range(5):
                    s = b[co]
                    for ci in range(2):
                        for ky in range(3):
                            for kx in range(3):
                                iy, ix = y + ky - 1, x + kx - 1
                                if 0 <= iy < 4 and 0 <= ix < 5:
                                    s += F[co, ci, ky, kx] * X[n, ci, iy, ix]
                    assert Z[n, co, y, x] == pytest.approx(s, rel=1e-13, abs=1e-13)


def test_closed_form_constant_input_counts_valid_taps():
    Cin, H, W = 3, 5, 6
    X = np.ones((1, Cin, H, W))
    F = np.ones((2, Cin, 3, 3))
    Z, _ = orc.conv_forward(X, F, np.zeros(2), 1, 0.1)
    ny = np.array([2 if y in (0, H - 1) else 3 for y in range(H)])
    nx = np.array([2 if x in (0, W - 1) else 3 for x in range(W)])
    expect = Cin * np.outer(ny, nx)
    assert np.array_equal(Z[0, 0], expect) and np.array_equal(Z[0, 1], expect)
    # filter gradient for all-ones delta: number of valid (pixel, tap) pairs
    dX, dF, db = orc.conv_backward(X, F, Z, np.ones_like(Z), 1, 0.1)
    for ky in range(3):
        for kx in range(3):
            assert dF[0, 0, ky, kx] == (H - abs(ky - 1)) * (W - abs(kx - 1))
    assert db[0] == H * W
    # input delta for all-ones delta and filter: Cout * number of valid taps
    assert np.array_equal(dX[0, 0], 2 * np.outer(ny, nx))


def test_leaky_slope_at_zero_and_negative():
    X = np.array([1.0, -2.0, 0.0, 3.0]).reshape(1, 1, 2, 2)
    F = np.ones((1, 1, 1, 1))
    Z, Y = orc.conv_forward(X, F, np.zeros(1), 0, 0.1)
    assert np.array_equal(Y.ravel(), [1.0, -0.2, 0.0, 3.0])
    dX, dF, db = orc.conv_backward(X, F, Z, np.ones_like(Z), 0, 0.1)
    # derivative 1 for Z > 0, slope for Z <= 0 (including exactly 0)
    assert np.allclose(dX.ravel(), [1.0, 0.1, 0.1, 1.0])
    assert db[0] == pytest.approx(2.2)
    assert dF[0, 0, 0, 0] == pytest.approx(1.0 - 0.2 + 0.0 + 3.0)


def test_maxpool_first_maximum_wins_ties():
    X = np.array([[5.0, 5.0, 1.0, 2.0],
                  [5.0, 5.0, 2.0, 2.0],
                  [0.0, 1.0, -1.0, -1.0],
                  [7.0, 7.0, -1.0, -0.5]]).reshape(1, 1, 4, 4)
    Y, arg = orc.maxpool_forward(X)
    assert np.array_equal(Y[0, 0], [[5.0, 2.0], [7.0, -0.5]])
    assert np.array_equal(arg[0, 0], [[0, 1], [2, 3]])
    dY = np.array([[1.0, 2.0], [3.0, 4.0]]).reshape(1, 1, 2, 2)
    dX = orc.maxpool_backward(dY, arg, X.shape)
    expect = np.zeros((4, 4))
    expect[0, 0], expect[0, 3], expect[3, 0], expect[3, 3] = 1.0, 2.0, 3.0, 4.0
    assert np.array_equal(dX[0, 0], expect)


def test_mse_closed_form():
    y = np.array([[1.0, 2.0], [3.0, 5.0]]).reshape(1, 1, 2, 2)
    t = np.array([[0.0, 2.0], [5.0, 1.0]]).reshape(1, 1, 2, 2)
    loss, d = orc.mse_loss(y, t)
    assert loss == pytest.approx((1 + 0 + 4 + 16) / 4)
    assert np.allclose(d.ravel(), [0.5, 0.0, -1.0, 2.0])


@pytest.mark.parametrize("seed", [0, 1])
def test_gradients_match_central_finite_differences(seed):
    layers = _tiny_net()
    x, params, target = _draw(layers, 2, 2, 6, 8, seed)
    out = orc.step(layers, x, params, lr=0.0, target=target)
    h = 1e-6
    g = np.zeros_like(params)
    for i in range(params.size):
        p1, p2 = params.copy(), params.copy()
        p1[i] += h
        p2[i] -= h
        g[i] = (_loss(layers, x, p1, target) - _loss(layers, x, p2, target)) / (2 * h)
    scale = np.abs(g).max()
    assert np.abs(out["dparams"] - g).max() <= 1e-7 * scale + 1e-9
    rng = np.random.default_rng(seed + 10)
    flat = x.ravel()
    for i in rng.choice(flat.size, size=40, replace=False):
        x1, x2 = flat.copy(), flat.copy()
        x1[i] += h
        x2[i] -= h
        fd = (_loss(layers, x1.reshape(x.shape), params, target)
              - _loss(layers, x2.reshape(x.shape), params, target)) / (2 * h)
        assert out["dx"].ravel()[i] == pytest.approx(fd, rel=1e-6, abs=1e-9)


def _torch_step(layers, x, params, target):
    xt = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    leaves = []
    h = xt
    acts = [xt]
    for l, fb in zip(layers, orc.unpack_params(layers, params)):
        if l.kind == "conv":
            Fw = torch.tensor(fb[0], dtype=torch.float64, requires_grad=True)
            bw = torch.tensor(fb[1], dtype=torch.float64, requires_grad=True)
            leaves += [Fw, bw]
            h = tF.leaky_relu(tF.conv2d(h, Fw, bw, stride=1, padding=l.pad), l.leaky)
        else:
            h = tF.max_pool2d(h, 2, 2)
        acts.append(h)
    loss = torch.mean((h - torch.tensor(target, dtype=torch.float64)) ** 2)
    loss.backward()
    g = torch.cat([t.grad.reshape(-1) for t in leaves]).numpy()
    return loss.item(), [a.detach().numpy() for a in acts], xt.grad.numpy(), g


@pytest.mark.parametrize("name,N,H,W", [("tiny", 2, 12, 16), ("yolo8", 1, 16, 24)])
def test_agrees_with_library_conv_and_autograd_fp64(name, N, H, W):
    layers = synth.stack_tiny() if name == "tiny" else synth.stack_yolo8()
    x, params, target = _draw(layers, N, 3, H, W, 5)
    out = orc.step(layers, x, params, lr=0.01, target=target)
    loss, acts, dx, g = _torch_step(layers, x, params, target)
    assert out["loss"] == pytest.approx(loss, rel=1e-12)
    for a, m in zip(acts, out["maps"]):
        assert np.abs(a - m).max() <= 1e-12 * max(1.0, np.abs(a).max())
    assert np.abs(dx - out["dx"]).max() <= 1e-12 * np.abs(dx).max() + 1e-18
    assert np.abs(g - out["dparams"]).max() <= 1e-12 * np.abs(g).max()
    # plain SGD: w <- w - lr * dL/dw, nothing else
    assert np.array_equal(out["new_params"], params - 0.01 * out["dparams"])
    assert np.abs(out["new_params"] - (params - 0.01 * g)).max() <= 1e-12 * np.abs(g).max()


def test_batch_gradient_is_sum_of_per_image_gradients():
    layers = synth.stack_tiny()
    x, params, _ = _draw(layers, 3, 3, 8, 8, 7)
    rng = np.random.default_rng(8)
    dy = rng.standard_normal((3,) + synth.map_shapes(layers, 3, 8, 8)[-1])
    full = orc.step(layers, x, params, lr=0.0, dy=dy)
    acc = np.zeros_like(params)
    for n in range(3):
        acc += orc.step(layers, x[n:n + 1], params, lr=0.0, dy=dy[n:n + 1])["dparams"]
    assert np.allclose(full["dparams"], acc, rtol=1e-12, atol=1e-14)


_THREAD_SCRIPT = """
import sys
import numpy as np
sys.path.insert(0, sys.argv[1])
from oracle import reference as orc
from paper_2409_09083_b200 import synth
layers = [synth.conv(2, 3, 3), synth.pool(), synth.conv(3, 4, 1), synth.conv(4, 2, 3)]
rng = np.random.default_rng(11)
x = rng.standard_normal((3, 2, 6, 8))
params = rng.standard_normal(orc.param_count(layers)) * 0.5
target = rng.standard_normal((3, 2, 3, 4))
r = orc.step(layers, x, params, lr=0.1, target=target)
np.savez(sys.argv[2], threads=orc.num_threads(), new_params=r["new_params"], dx=r["dx"], y=r["y"], loss=r["loss"])
"""


def test_result_independent_of_thread_count(tmp_path):
    """The same step in fresh processes with 1, 2 and 5 OpenMP threads: the loops are parallel over
    (image, output channel) only, so every sum keeps its order and the results are bit-identical."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    script = tmp_path / "run.py"
    script.write_text(_THREAD_SCRIPT)
    got = {}
    for threads in (1, 2, 5):
        out = tmp_path / f"t{threads}.npz"
        env = dict(os.environ, OMP_NUM_THREADS=str(threads), OMP_DYNAMIC="false")
        subprocess.run([sys.executable, str(script), root, str(out)], check=True, env=env)
        got[threads] = np.load(out)
        assert int(got[threads]["threads"]) == threads          # the setting really reached the C loops
    for threads in (2, 5):
        for key in ("new_params", "dx", "y", "loss"):
            assert np.array_equal(got[1][key], got[threads][key]), (threads, key)


def test_round_bf16_matches_library_conversion_and_ties_go_to_even():
    rng = np.random.default_rng(9)
    a = np.concatenate([rng.standard_normal(5000) * 10.0 ** rng.integers(-6, 6, 5000), [0.0, 1.0, -1.0, 255.0, 256.0]])
    a = a.astype(np.float32).astype(np.float64)          # fp32-representable, as the library routine expects
    want = torch.from_numpy(a.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(orc.round_bf16(a), want)
    # 1 + 2^-8 lies half way between 1 and 1 + 2^-7: ties to even keeps 1; 1 + 3*2^-8 goes up to 1 + 2^-6
    assert orc.round_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    assert orc.round_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6


def test_bf16_storage_only_rounds_stored_maps():
    layers = _tiny_net()
    x, params, target = _draw(layers, 1, 2, 8, 8, 4)
    maps64, _ = orc.forward(layers, x, params)
    maps16, tape = orc.forward(layers, x, params, store="bf16")
    assert np.array_equal(maps16[1], orc.round_bf16(maps64[1]))           # first conv output: rounded once
    for m, l in zip(maps16[1:], layers):
        if l.kind == "conv":
            assert np.array_equal(m, orc.round_bf16(m))                   # every stored conv output is a bf16 value
    # without discrete decisions (slope 1, no pool) storage rounding only perturbs the gradients
    lin = [synth.conv(2, 3, 3, leaky=1.0), synth.conv(3, 2, 3, leaky=1.0)]
    x, params, target = _draw(lin, 1, 2, 8, 8, 4)
    r = orc.step(lin, x, params, 0.0, target=target, store="bf16")
    r64 = orc.step(lin, x, params, 0.0, target=target)
    err = np.abs(r["dparams"] - r64["dparams"]).max() / np.abs(r64["dparams"]).max()
    assert 0.0 < err <= 2e-2


def _integer_case():
    """A small conv / pool stack on data whose maps AND deltas are small integers."""
    layers = [synth.conv(2, 4, 3, leaky=0.0), synth.pool(), synth.conv(4, 3, 1, leaky=0.0), synth.conv(3, 2, 3, leaky=0.0)]
    wl = synth.Workload("int", tuple(layers), 2, 2, 8, 12, (1, 1), ((1, 4),))
    x, params, _ = synth.draw_integer_relu(wl)
    dy = np.random.default_rng(21).integers(-2, 3, size=(2, 2, 4, 6)).astype(np.float64)
    return layers, x.astype(np.float64), params.astype(np.float64), dy


def test_bf16_storage_is_the_identity_on_bf16_exact_data():
    """Pin of the store="bf16" branch against the plain branch (itself pinned by finite differences
    and a library autograd above): where every stored map and every delta in front of an activation
    is exactly representable in bfloat16 (integers of magnitude <= 256), rounding them changes
    nothing, so the two branches must agree BIT FOR BIT in every map, delta and gradient.  A mask
    taken from the wrong tensor, `>=` instead of `>` at Z == 0, or a wrong slope in the store
    branch breaks the equality."""
    layers, x, params, dy = _integer_case()
    plain = orc.step(layers, x, params, 0.25, dy=dy)
    stored = orc.step(layers, x, params, 0.25, dy=dy, store="bf16")
    # the premise, checked on the plain branch: integers that 8 significant bits hold
    tape = orc.forward(layers, x, params)[1]
    zero_preact = 0
    for i, l in enumerate(layers):
        m, d = plain["maps"][i + 1], plain["deltas"][i + 1]
        assert np.array_equal(m, np.rint(m)) and np.abs(m).max() <= 256
        assert np.array_equal(d, np.rint(d)) and np.abs(d).max() <= 256
        if l.kind == "conv":
            zero_preact += int(((tape[i] == 0.0) & (d != 0.0)).sum())
    assert zero_preact > 0          # the Z == 0 rule is exercised with a non-zero delta
    assert np.abs(plain["dparams"]).max() > 0 and np.abs(plain["dx"]).max() > 0
    for a, b in zip(plain["maps"], stored["maps"]):
        assert np.array_equal(a, b)
    for a, b in zip(plain["deltas"], stored["deltas"]):
        assert np.array_equal(a, b)
    for key in ("y", "dx", "dparams", "new_params"):
        assert np.array_equal(plain[key], stored[key]), key


def test_bf16_storage_hand_evaluated_one_conv():
    """One 1x1 conv, one channel, slope 0.1, evaluated by hand.  F = -1, b = 0.25, so Z = 0.25 - X:
        X  = [[1, -2], [0.25, 3]]      Z = [[-0.75, 2.25], [0, -2.75]]
    Derivative of the activation: 1 where Z > 0, else the slope (also at Z == 0):
        mask = [[0.1, 1], [0.1, 0.1]]            (a mask taken from X instead would be [[1, .1], [1, 1]])
        dY   = [[1.01, 1.01], [1.01, 1.3]]       dY * mask = [[0.101, 1.01], [0.101, 0.13]]
    Rounded to 8 significant bits AFTER the mask:
        0.101 = 0.808 * 2^-3 -> 207/256 * 2^-3 = 207/2048 = 0.10107421875
        1.01  = 0.505 * 2^1  -> 129/256 * 2    = 129/128  = 1.0078125
        0.13  = 0.52  * 2^-2 -> 133/256 / 4    = 133/1024 = 0.1298828125
    (rounding dY first would give 1.0078125 * 0.1 = 0.10078125 and 1.296875 * 0.1 = 0.1296875).
    Gradients are formed from the rounded delta:
        db = 2 * 207/2048 + 129/128 + 133/1024                     = 1.33984375
        dF = 1 * 207/2048 - 2 * 129/128 + 0.25 * 207/2048 + 3 * 133/1024 = -1.4996337890625
        dX = F * dZ = -dZ"""
    layers = [synth.conv(1, 1, 1, leaky=0.1)]
    x = np.array([[1.0, -2.0], [0.25, 3.0]]).reshape(1, 1, 2, 2)
    params = np.array([-1.0, 0.25])
    dy = np.array([[1.01, 1.01], [1.01, 1.3]]).reshape(1, 1, 2, 2)
    r = orc.step(layers, x, params, 0.0, dy=dy, store="bf16")
    dz = np.array([[207 / 2048, 129 / 128], [207 / 2048, 133 / 1024]])
    assert np.array_equal(r["dx"][0, 0], -dz)
    assert r["dparams"][1] == 1.33984375
    assert r["dparams"][0] == -1.4996337890625
    # the forward half: Y = leaky(Z) stored in bf16; -0.075 = -0.6 * 2^-3 -> -154/256 / 8 = -0.0751953125,
    # -0.275 = -0.55 * 2^-1 -> -141/256 / 2 = -0.275390625
    assert np.array_equal(r["y"][0, 0], np.array([[-0.0751953125, 2.25], [0.0, -0.275390625]]))
