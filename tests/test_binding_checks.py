"""The Python binding refuses tensors whose sizes do not match the plan BEFORE anything reaches the
library: the kernels index by the plan's shapes, so a wrong-sized tensor would be an out-of-bounds
device access, not an exception.  Everything here runs on the CPU (plans are host objects; the
checks raise before any device pointer is taken)."""
import pytest
import torch

import paper_2409_09083_b200 as ftp
from paper_2409_09083_b200 import synth


@pytest.fixture(scope="module")
def plan():
    wl = synth.workload("C0")
    return ftp.ftp_plan(wl.layers, wl.N, wl.C, wl.H, wl.W, wl.grid, wl.groups)


def _t(n):
    return torch.zeros(n, dtype=torch.float32)


def test_plan_reports_the_sizes_the_checks_use(plan):
    assert plan.in_floats == 1 * 3 * 32 * 32
    assert plan.out_floats == 1 * 16 * 16 * 16
    assert plan.param_floats == 1392
    assert plan.workspace_bytes > 0


def test_forward_rejects_wrong_sizes(plan):
    ws = torch.zeros(plan.workspace_bytes, dtype=torch.uint8)
    with pytest.raises(ValueError, match="x has 10 elements"):
        ftp.ftp_forward(plan, _t(10), _t(plan.param_floats), None, ws)
    with pytest.raises(ValueError, match="params has 7 elements"):
        ftp.ftp_forward(plan, _t(plan.in_floats), _t(7), None, ws)
    with pytest.raises(ValueError, match="y has"):
        ftp.ftp_forward(plan, _t(plan.in_floats), _t(plan.param_floats), _t(plan.out_floats + 1), ws)
    with pytest.raises(ValueError, match="workspace holds"):
        ftp.ftp_forward(plan, _t(plan.in_floats), _t(plan.param_floats), None, ws[:-1])
    # right sizes, but host memory: still refused, by the device check
    with pytest.raises(ValueError, match="CUDA"):
        ftp.ftp_forward(plan, _t(plan.in_floats), _t(plan.param_floats), None, ws)


def test_backward_and_step_reject_wrong_sizes(plan):
    ws = torch.zeros(plan.workspace_bytes, dtype=torch.uint8)
    x, p, dy = _t(plan.in_floats), _t(plan.param_floats), _t(plan.out_floats)
    with pytest.raises(ValueError, match="dy has"):
        ftp.ftp_backward(plan, x, _t(3), p, None, p, ws)
    with pytest.raises(ValueError, match="dparams has"):
        ftp.ftp_backward(plan, x, dy, p, None, _t(plan.param_floats - 1), ws)
    with pytest.raises(ValueError, match="dx has"):
        ftp.ftp_backward(plan, x, dy, p, _t(5), p, ws)
    with pytest.raises(ValueError, match="target has"):
        ftp.ftp_step(plan, x, p, 0.1, ws, target=_t(plan.out_floats * 2))
    with pytest.raises(ValueError, match="loss_out has"):
        ftp.ftp_step(plan, x, p, 0.1, ws, target=dy, loss_out=_t(0))
    with pytest.raises(ValueError, match="dparams has"):
        ftp.ftp_step_grad(plan, x, p, _t(1), ws, target=dy)
    with pytest.raises(ValueError, match="workspace"):
        ftp.ftp_step(plan, x, p, 0.1, None, target=dy)


def test_loss_and_sgd_reject_wrong_sizes(plan):
    ws = torch.zeros(plan.workspace_bytes, dtype=torch.uint8)
    y = _t(plan.out_floats)
    with pytest.raises(ValueError, match="dy has"):
        ftp.ftp_loss_mse(plan, y, y, _t(4), _t(1), ws)
    with pytest.raises(ValueError, match="loss_out has"):
        ftp.ftp_loss_mse(plan, y, y, None, _t(2), ws)
    with pytest.raises(ValueError, match="target has"):
        ftp.ftp_loss_mse_static(_t(8), _t(9), None, _t(1))
    with pytest.raises(ValueError, match="dy has"):
        ftp.ftp_loss_mse_static(_t(8), _t(8), _t(7), _t(1))
    with pytest.raises(ValueError, match="loss_out has"):
        ftp.ftp_loss_mse_static(_t(8), _t(8), None, _t(3))
    with pytest.raises(ValueError, match="grad has"):
        ftp.ftp_sgd(_t(8), _t(9), 0.1)


def test_host_batch_calls_reject_wrong_sizes(plan):
    ws = torch.zeros(plan.workspace_bytes, dtype=torch.uint8)
    x, t = _t(plan.in_floats), _t(plan.out_floats)
    with pytest.raises(ValueError, match="x_host has"):
        ftp.ftp_prefetch_host(plan, _t(3), t, ws)
    with pytest.raises(ValueError, match="target_host has"):
        ftp.ftp_prefetch_host(plan, x, _t(3), ws)
    with pytest.raises(ValueError, match="loss_host has"):
        ftp.ftp_step_host(plan, x, t, _t(plan.param_floats), 0.1, _t(2), ws)
    with pytest.raises(ValueError, match="params has"):
        ftp.ftp_step_host(plan, x, t, _t(2), 0.1, _t(1), ws)
