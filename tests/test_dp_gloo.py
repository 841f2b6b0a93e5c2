"""The multi-GPU exchange step on CPU: two gloo ranks, each holding half of the batch, must arrive
at the update of the whole batch.  The per-rank gradient comes from the oracle here (the CUDA path
needs a GPU); what is tested is the sharding, the all-reduce and the learning-rate scaling that
`bench.py --gpus N` uses."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import reference as orc
from paper_2409_09083_b200 import dp, synth


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = synth.workload("C0").with_(N=4)
    x, params, target = synth.draw(wl, bias_std=0.3)
    lo, hi = dp.shard_range(wl.N, rank, world)
    local = orc.step(list(wl.layers), x[lo:hi], params, 0.0, target=target[lo:hi])
    grad = torch.from_numpy(local["dparams"].copy())
    new = torch.from_numpy(params.astype(np.float64))

    def sgd(g, lr_eff):
        new.sub_(lr_eff * g)

    dp.allreduce_and_update(grad, 0.05, world, dist.all_reduce, sgd)
    np.save(os.path.join(out_dir, f"rank{rank}.npy"), new.numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reproduce_the_full_batch_update(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    wl = synth.workload("C0").with_(N=4)
    x, params, target = synth.draw(wl, bias_std=0.3)
    ref = orc.step(list(wl.layers), x, params, 0.05, target=target)
    a = np.load(tmp_path / "rank0.npy")
    b = np.load(tmp_path / "rank1.npy")
    assert np.array_equal(a, b)
    assert np.abs(a - ref["new_params"]).max() <= 1e-12 * np.abs(ref["new_params"]).max()


def _worker_overlapped(rank, world, port, out_dir):
    """Each rank hands the gradient to the exchange slice by slice, last executed group first, as
    ftp_step_grad_groups does; the slices come from the plan (a host object), the numbers from the oracle."""
    import paper_2409_09083_b200 as ftp
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = synth.Workload("y8", tuple(synth.stack_yolo8()), 4, 3, 32, 32, (2, 2), ((1, 4), (5, 8)))
    x, params, target = synth.draw(wl, bias_std=0.3)
    lo, hi = dp.shard_range(wl.N, rank, world)
    local = orc.step(list(wl.layers), x[lo:hi], params, 0.0, target=target[lo:hi])
    grad = torch.zeros(params.size, dtype=torch.float64)
    new = torch.from_numpy(params.astype(np.float64))
    plan = ftp.ftp_plan(wl.layers, hi - lo, wl.C, wl.H, wl.W, wl.grid, wl.groups)
    # parameter range of every executed group: its conv layers' filters and biases, in layer order
    starts, off = {}, 0
    for i, l in enumerate(wl.layers, start=1):
        starts[i] = off
        if l.kind == "conv":
            off += l.cout * l.cin * l.k * l.k + l.cout
    starts[len(wl.layers) + 1] = off
    ex = dp.OverlappedExchange(grad, world, lambda view: dist.all_reduce(view, async_op=True))
    for gi, (a, b) in reversed(list(enumerate(plan.exec_groups()))):
        begin, end = starts[a], starts[b + 1]
        grad[begin:end] = torch.from_numpy(local["dparams"][begin:end])       # "the group's backward pass has run"
        ex.ready(gi, begin, end - begin)
    ex.finish(0.05, lambda g, lr_eff: new.sub_(lr_eff * g))
    np.save(os.path.join(out_dir, f"ov{rank}.npy"), new.numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_overlapped_exchange_reproduces_the_full_batch_update(tmp_path):
    world = 2
    mp.spawn(_worker_overlapped, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    wl = synth.Workload("y8", tuple(synth.stack_yolo8()), 4, 3, 32, 32, (2, 2), ((1, 4), (5, 8)))
    x, params, target = synth.draw(wl, bias_std=0.3)
    ref = orc.step(list(wl.layers), x, params, 0.05, target=target)
    a, b = np.load(tmp_path / "ov0.npy"), np.load(tmp_path / "ov1.npy")
    assert np.array_equal(a, b)
    assert np.abs(a - ref["new_params"]).max() <= 1e-12 * np.abs(ref["new_params"]).max()


def test_exchange_refuses_slices_that_do_not_tile_the_gradient():
    import pytest
    grad = torch.zeros(10, dtype=torch.float64)
    ex = dp.OverlappedExchange(grad, 1, all_reduce=None)
    ex.ready(1, 4, 6)
    ex.ready(0, 0, 3)                                   # parameter 3 is never reported
    with pytest.raises(RuntimeError, match="gap or overlap"):
        ex.finish(0.1, lambda g, lr: None)
    ex = dp.OverlappedExchange(grad, 1, all_reduce=None)
    ex.ready(0, 0, 4)
    with pytest.raises(RuntimeError, match="cover 4 of 10"):
        ex.finish(0.1, lambda g, lr: None)


def test_shard_ranges_partition_the_batch():
    for total, world in [(16, 8), (4, 2), (7, 3), (1, 1)]:
        r = [dp.shard_range(total, k, world) for k in range(world)]
        assert r[0][0] == 0 and r[-1][1] == total
        assert all(a[1] == b[0] for a, b in zip(r, r[1:]))
