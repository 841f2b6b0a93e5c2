"""ftp_loss_mse_static: the loss and its delta for callers that may not allocate device memory
(stream capture in progress, an allocator that owns the whole device, a fixed memory budget).
It keeps its partial sums in an array inside the library image instead of a workspace, so every
call on a GPU shares that array.  Checked here against ftp_loss_mse through the C-ABI on two calls
in a row -- the second smaller than the first, so anything it wrongly picked up from the array's
earlier contents would show -- plus the capacity check.  This file sorts last on purpose."""
import numpy as np
import pytest
import torch

import paper_2409_09083_b200 as ftp
from paper_2409_09083_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _both(shape, seed):
    N, C, H, Wd = shape
    wl = synth.Workload("mse", (synth.conv(2, C, 1),), N, 2, H, Wd, (1, 1), ((1, 1),))
    plan = ftp.ftp_plan(wl.layers, N, wl.C, H, Wd, wl.grid, wl.groups)
    ws = plan.new_workspace()
    rng = np.random.default_rng(seed)
    y = torch.from_numpy(rng.standard_normal(shape).astype(np.float32)).cuda()
    t = torch.from_numpy(rng.standard_normal(shape).astype(np.float32)).cuda()
    dy_a, dy_b = torch.empty_like(y), torch.empty_like(y)
    loss_a = torch.zeros(1, dtype=torch.float32, device="cuda")
    loss_b = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
    ftp.ftp_loss_mse(plan, y, t, dy_a, loss_a, ws)
    # The first call on a device resolves the array's address and loads the kernels' module, which the
    # driver may account as device memory; the library asks for that call to come before any region
    # that must not allocate.  Free memory is therefore sampled around a LATER call.
    ftp.ftp_loss_mse_static(y, t, None, loss_b)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    ftp.ftp_loss_mse_static(y, t, dy_b, loss_b)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before     # the device's free memory did not move
    return dy_a.cpu().numpy(), loss_a.item(), dy_b.cpu().numpy(), loss_b.item()


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    # 3 x 40 x 64 x 72 = 552 960 elements = 34 blocks; then 2 x 5 x 7 x 9 = 630 elements = 1 block
    for shape, seed in (((3, 40, 64, 72), 11), ((2, 5, 7, 9), 12)):
        dy_a, loss_a, dy_b, loss_b = _both(shape, seed)
        assert np.array_equal(dy_a, dy_b)                  # same expression per element
        assert loss_b == pytest.approx(loss_a, rel=1e-5)   # sums in another fixed order
        assert 1.5 < loss_b < 2.5                          # mean of (a - b)^2 for unit normals is 2


def test_loss_only_and_delta_only():
    y = torch.randn(1000, device="cuda")
    t = torch.randn(1000, device="cuda")
    loss = torch.zeros(1, device="cuda")
    dy = torch.empty_like(y)
    ftp.ftp_loss_mse_static(y, t, None, loss)
    ftp.ftp_loss_mse_static(y, t, dy, None)
    torch.cuda.synchronize()
    assert loss.item() == pytest.approx(((y - t) ** 2).mean().item(), rel=1e-5)
    assert torch.allclose(dy, 2 * (y - t) / 1000, rtol=1e-6, atol=0)


def test_capacity_is_enforced_before_anything_is_launched():
    y = torch.zeros(8, device="cuda")
    loss = torch.full((1,), 7.0, device="cuda")
    rc = binding._lib.ftp_loss_mse_static(y.data_ptr(), y.data_ptr(), None, loss.data_ptr(), (1 << 26) + 1, None)
    assert rc == -9 and "capacity" in ftp.ftp_strerror(rc)
    rc = binding._lib.ftp_loss_mse_static(y.data_ptr(), y.data_ptr(), None, None, 8, None)
    assert rc == -1
    torch.cuda.synchronize()
    assert loss.item() == 7.0
