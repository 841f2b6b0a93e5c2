"""Spatial sharding on CPU: two and three gloo ranks split every map by rows (rank r = user tile (r, 0) of a
(world x 1) grid), exchange boundary rows at the group inputs as the planner's spans say, and must
arrive at the untiled oracle's activations, input gradient and update.  Each rank computes with the oracle's
own layer routines on its slab; what is tested is the tables (`dp.row_shard_tables`, built on
ftp_plan_region), the forward exchange, the adjoint backward exchange (overlapping input deltas are summed at
their owner) and the gradient all-reduce -- the host logic of a row-sharded multi-GPU step."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import paper_2409_09083_b200 as ftp
from oracle import reference as orc
from paper_2409_09083_b200 import dp, synth

WL = synth.Workload("y8", tuple(synth.stack_yolo8()), 2, 3, 48, 32, (1, 1), ((1, 2), (3, 4), (5, 8)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _exchange(world, rank, full_rows, table, have, add):
    """Moves rows between ranks.  have[r] = (lo, array of rows lo..): what this rank holds of the map.
    Forward (add=False): every rank receives the rows of table['recv'][rank] from their owners.
    Backward (add=True): the same rows travel the other way and are added at the owner."""
    reqs, bufs = [], []
    for dst in range(world):
        for src, a, b in table["recv"][dst]:
            sender, receiver = (dst, src) if add else (src, dst)
            if rank == sender:
                lo, arr = have
                t = torch.from_numpy(np.ascontiguousarray(arr[:, :, a - lo:b - lo + 1, :]))
                reqs.append(dist.isend(t, receiver))
            if rank == receiver:
                t = torch.empty((full_rows[0], full_rows[1], b - a + 1, full_rows[2]), dtype=torch.float64)
                reqs.append(dist.irecv(t, sender))
                bufs.append((a, b, t))
    for q in reqs:
        q.wait()
    return bufs


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = WL
    layers = list(wl.layers)
    x, params, target = synth.draw(wl, bias_std=0.3)
    x, params, target = x.astype(np.float64), params.astype(np.float64), target.astype(np.float64)
    shapes = synth.map_shapes(layers, wl.C, wl.H, wl.W)
    rows = [s[1] for s in shapes]
    plan = ftp.ftp_plan(wl.layers, wl.N, wl.C, wl.H, wl.W, (world, 1), wl.groups)
    tables = dp.row_shard_tables(plan, rows, world)
    per = orc.unpack_params(layers, params)

    # ---- forward, group by group ----
    owned = None            # (lo, rows lo..hi of the current group-input map) this rank owns
    saved = []
    for g, t in enumerate(tables):
        first, last = t["first"], t["last"]
        glayers = layers[first - 1:last]
        gparams = orc.pack_params(glayers, per[first - 1:last])
        lo, hi = t["needed_in"][rank]
        C, W = shapes[first - 1][0], shapes[first - 1][2]
        slab = np.zeros((wl.N, C, hi - lo + 1, W))
        if g == 0:
            slab[:] = x[:, :, lo:hi + 1, :]                 # the host scatters the input: each rank gets what it needs
        else:
            olo, oarr = owned
            a, b = max(olo, lo), min(olo + oarr.shape[2] - 1, hi)
            slab[:, :, a - lo:b - lo + 1, :] = oarr[:, :, a - olo:b - olo + 1, :]
            for a, b, buf in _exchange(world, rank, (wl.N, C, W), t, owned, add=False):
                slab[:, :, a - lo:b - lo + 1, :] = buf.numpy()
        # align the slab to the group's total stride with zero rows (they only reach rows nobody owns here)
        scale = rows[first - 1] // rows[last]
        top = lo % scale
        bottom = (-(hi + 1)) % scale
        padded = np.concatenate([np.zeros((wl.N, C, top, W)), slab, np.zeros((wl.N, C, bottom, W))], axis=2)
        maps, tape = orc.forward(glayers, padded, gparams)
        olo_out, ohi_out = t["owned_out"][rank]
        base = (lo - top) // scale                           # map row of the slab output's row 0
        y_owned = maps[-1][:, :, olo_out - base:ohi_out - base + 1, :]
        saved.append(dict(maps=maps, tape=tape, glayers=glayers, gparams=gparams, top=top, lo=lo, hi=hi, base=base))
        owned = (olo_out, y_owned)

    # ---- loss delta on the owned rows of the last map ----
    M = target.size
    olo, y_owned = owned
    dy_owned = 2.0 * (y_owned - target[:, :, olo:olo + y_owned.shape[2], :]) / M
    loss_part = float(((y_owned - target[:, :, olo:olo + y_owned.shape[2], :]) ** 2).sum() / M)

    # ---- backward, adjoint form: every rank back-propagates the delta of ITS output rows through its own slab ----
    grad = np.zeros_like(params)
    goff = [0]
    for l in layers:
        goff.append(goff[-1] + (l.cout * l.cin * l.k * l.k + l.cout if l.kind == "conv" else 0))
    d_owned = (olo, dy_owned)
    dx_owned = None
    for g in range(len(tables) - 1, -1, -1):
        t, sv = tables[g], saved[g]
        first, last = t["first"], t["last"]
        out_map = sv["maps"][-1]
        dslab = np.zeros_like(out_map)
        dlo, darr = d_owned
        dslab[:, :, dlo - sv["base"]:dlo - sv["base"] + darr.shape[2], :] = darr
        dxs, dpar, _ = orc.backward(sv["glayers"], sv["maps"], sv["tape"], sv["gparams"], dslab)
        grad[goff[first - 1]:goff[last]] += dpar
        dxs = dxs[:, :, sv["top"]:sv["top"] + sv["hi"] - sv["lo"] + 1, :]          # the needed rows lo..hi
        ilo, ihi = t["owned_in"][rank] if g > 0 else (sv["lo"], sv["hi"])
        C, W = shapes[first - 1][0], shapes[first - 1][2]
        if g > 0:
            mine = np.zeros((wl.N, C, ihi - ilo + 1, W))
            a, b = max(ilo, sv["lo"]), min(ihi, sv["hi"])
            mine[:, :, a - ilo:b - ilo + 1, :] = dxs[:, :, a - sv["lo"]:b - sv["lo"] + 1, :]
            for a, b, buf in _exchange(world, rank, (wl.N, C, W), t, (sv["lo"], dxs), add=True):
                mine[:, :, a - ilo:b - ilo + 1, :] += buf.numpy()
            d_owned = (ilo, mine)
        else:
            dx_owned = (sv["lo"], dxs)                       # network input: overlapping rows are summed by the host below

    gt = torch.from_numpy(grad)
    dist.all_reduce(gt)                                       # the sum of the ranks' partial gradient sets
    lt = torch.tensor([loss_part], dtype=torch.float64)
    dist.all_reduce(lt)
    np.savez(os.path.join(out_dir, f"r{rank}.npz"), grad=gt.numpy(), loss=lt.numpy(), y_lo=owned[0], y=owned[1],
             dx_lo=dx_owned[0], dx=dx_owned[1])
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_row_sharded_step_matches_the_untiled_oracle(tmp_path, world):
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    wl = WL
    x, params, target = synth.draw(wl, bias_std=0.3)
    ref = orc.step(list(wl.layers), x.astype(np.float64), params.astype(np.float64), 0.0, target=target.astype(np.float64))
    parts = [np.load(tmp_path / f"r{r}.npz") for r in range(world)]
    y = np.zeros_like(ref["y"])
    dx = np.zeros_like(ref["dx"])
    for p in parts:
        y[:, :, int(p["y_lo"]):int(p["y_lo"]) + p["y"].shape[2], :] = p["y"]
        dx[:, :, int(p["dx_lo"]):int(p["dx_lo"]) + p["dx"].shape[2], :] += p["dx"]       # overlapping input rows add up
    assert np.abs(y - ref["y"]).max() <= 1e-12 * np.abs(ref["y"]).max()
    assert parts[0]["loss"][0] == pytest.approx(ref["loss"], rel=1e-12)
    for p in parts:
        assert np.abs(p["grad"] - ref["dparams"]).max() <= 1e-12 * np.abs(ref["dparams"]).max()
    assert np.abs(dx - ref["dx"]).max() <= 1e-12 * np.abs(ref["dx"]).max()


def test_tables_partition_the_maps_and_name_the_owners():
    wl = WL
    rows = [s[1] for s in synth.map_shapes(wl.layers, wl.C, wl.H, wl.W)]
    for world in (2, 3, 4):
        plan = ftp.ftp_plan(wl.layers, wl.N, wl.C, wl.H, wl.W, (world, 1), wl.groups)
        tables = dp.row_shard_tables(plan, rows, world)
        assert [(t["first"], t["last"]) for t in tables] == list(wl.groups)
        for g, t in enumerate(tables):
            covered = []
            for r in range(world):
                covered += list(range(t["owned_out"][r][0], t["owned_out"][r][1] + 1))
                lo, hi = t["needed_in"][r]
                olo, ohi = t["owned_in"][r]
                got = set(range(max(lo, olo), min(hi, ohi) + 1)) if g > 0 else set(range(lo, hi + 1))
                for src, a, b in t["recv"][r]:
                    assert src != r and t["owned_in"][src][0] <= a <= b <= t["owned_in"][src][1]
                    got |= set(range(a, b + 1))
                assert got == set(range(lo, hi + 1))          # own rows + received rows = needed rows
            assert covered == list(range(rows[t["last"]]))    # owned output rows partition the map
        assert tables[0]["recv"] == [[] for _ in range(world)]


# ---------------------------------------------------------------------------------------------
# The same step as the library runs it on GPUs (`shard.RowShardedStep` over `shard.DistTransport`), here with two
# and three gloo ranks on the CPU and the oracle's layer routines in the place of the CUDA library.
# ---------------------------------------------------------------------------------------------
class OracleGroup:
    """Stand-in for shard.LibraryGroup: a requested group on a slab, computed by the oracle (fp64, CPU)."""

    def __init__(self, glayers, N, c_in, hs, w_in, out_shape, device, **_):
        self.glayers = list(glayers)

    def forward(self, slab, pg):
        self.maps, self.tape = orc.forward(self.glayers, slab.numpy(), pg.numpy())
        return torch.from_numpy(self.maps[-1])

    def backward(self, slab, dslab, pg, grad_out):
        dxs, dpar, _ = orc.backward(self.glayers, self.maps, self.tape, pg.numpy(), dslab.numpy())
        grad_out += torch.from_numpy(dpar)
        return torch.from_numpy(dxs)

    @staticmethod
    def sgd(params, grad, lr):
        params -= lr * grad


def _shard_worker(rank, world, port, out_dir):
    from paper_2409_09083_b200 import shard
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = WL
    x, params, target = synth.draw(wl, bias_std=0.3)
    xd, pd, td = (torch.from_numpy(a.astype(np.float64)) for a in (x, params, target))
    st = shard.RowShardedStep(wl.layers, wl.N, wl.C, wl.H, wl.W, wl.groups, shard.DistTransport(dist), device="cpu",
                              group_cls=OracleGroup, dtype=torch.float64)
    loss = st.step(xd, td, pd, 0.05)
    np.savez(os.path.join(out_dir, f"s{rank}.npz"), loss=loss, y_lo=st.y_lo, y=st.y_owned.numpy(), dx_lo=st.dx_lo,
             dx=st.dx_needed.numpy(), grad=st.grad.numpy(), params=pd.numpy())
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_row_sharded_step_class_over_gloo_matches_the_oracle(world, tmp_path):
    mp.spawn(_shard_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    wl = WL
    x, params, target = synth.draw(wl, bias_std=0.3)
    ref = orc.step(list(wl.layers), x.astype(np.float64), params.astype(np.float64), 0.05, target=target.astype(np.float64))
    outs = [np.load(os.path.join(str(tmp_path), f"s{r}.npz")) for r in range(world)]
    y = np.zeros_like(ref["y"]); dx = np.zeros_like(ref["dx"])
    for o in outs:
        y[:, :, int(o["y_lo"]):int(o["y_lo"]) + o["y"].shape[2], :] = o["y"]
        dx[:, :, int(o["dx_lo"]):int(o["dx_lo"]) + o["dx"].shape[2], :] += o["dx"]
        assert float(o["loss"]) == pytest.approx(ref["loss"], rel=1e-12)
        assert np.abs(o["grad"] - ref["dparams"]).max() <= 1e-12 * max(1.0, np.abs(ref["dparams"]).max())
        assert np.abs(o["params"] - ref["new_params"]).max() <= 1e-12 * max(1.0, np.abs(ref["new_params"]).max())
    assert np.abs(y - ref["y"]).max() <= 1e-12 * np.abs(ref["y"]).max()
    assert np.abs(dx - ref["dx"]).max() <= 1e-12 * max(1.0, np.abs(ref["dx"]).max())
