"""Spatial sharding: one training step with every map split by rows over `world` ranks, one GPU per rank.

This is the paper's own partitioning with a GPU in the place of a device (Sections 3 and 4.2): rank r is user
tile (r, 0) of a (world x 1) grid.  Between two requested groups the ranks exchange the boundary rows the
planner's spans call for (`dp.row_shard_tables`, Eq. (1) through the whole group); inside a group nothing is
exchanged.  Per group every rank runs the one-GPU library on ITS slab of the group's input map:

  forward   rows it owns + rows received from their owners -> `ftp_forward` on the slab -> it keeps the rows
            of the output map it owns.  The slab is handled as an image of its own: its zero padding at an
            interior edge only reaches output rows that belong to the neighbour, which are dropped.
  backward  adjoint form: the delta of the OWNED output rows (zero elsewhere) goes through `ftp_backward` on the
            same slab; the input-delta rows outside the owned range travel back to their owners, who ADD them
            (the overlapping input deltas of Section 4.1); the partial filter gradients of all ranks are summed
            (one all-reduce), and every rank applies the same update.

No kernel reads another GPU's memory: rows are received into local tensors first (point-to-point copies of the
transport), and the library only ever sees local pointers.

Transports: `DistTransport` (torch.distributed: NCCL between GPUs, gloo on the CPU) and `ThreadTransport`, which
runs the ranks as threads of one process with queues in between (all ranks on ONE device; their launches are
serialised by the stream and no kernel waits for another, only host threads wait for rows).  The latter is how
the step is tested where one GPU is all there is.
"""
import queue
import threading

import numpy as np
import torch

from . import binding as ftp
from . import dp, synth


class ThreadTransport:
    """Ranks as threads of one process.  Make one with ThreadTransport.group(world)."""

    def __init__(self, rank, world, boxes, barrier):
        self.rank, self.world, self._boxes, self._barrier = rank, world, boxes, barrier

    @staticmethod
    def group(world):
        boxes = {(s, d): queue.Queue() for s in range(world) for d in range(world)}
        barrier = threading.Barrier(world)
        return [ThreadTransport(r, world, boxes, barrier) for r in range(world)]

    def send(self, dst, tensor):
        t = tensor.clone()
        if t.is_cuda:
            torch.cuda.current_stream().synchronize()                # the rows are complete before they are handed over
        self._boxes[(self.rank, dst)].put(t)

    def recv(self, src, like):
        t = self._boxes[(src, self.rank)].get(timeout=120)
        assert t.shape == like.shape, (t.shape, like.shape)
        return t

    def all_reduce(self, tensor):
        """Sum over the ranks, in rank order on every rank (so all ranks hold the same bits)."""
        if tensor.is_cuda:
            torch.cuda.current_stream().synchronize()
        for d in range(self.world):
            if d != self.rank:
                self._boxes[(self.rank, d)].put(tensor.clone())
        parts = {self.rank: tensor.clone()}
        for s in range(self.world):
            if s != self.rank:
                parts[s] = self._boxes[(s, self.rank)].get(timeout=120)
        tensor.zero_()
        for s in range(self.world):
            tensor += parts[s]
        self._barrier.wait(timeout=120)


class DistTransport:
    """Ranks as processes of a torch.distributed group (NCCL for CUDA tensors, gloo for CPU tensors)."""

    def __init__(self, dist):
        self._dist, self.rank, self.world = dist, dist.get_rank(), dist.get_world_size()

    def send(self, dst, tensor):
        self._dist.send(tensor.contiguous(), dst)

    def recv(self, src, like):
        t = torch.empty_like(like)
        self._dist.recv(t, src)
        return t

    def all_reduce(self, tensor):
        self._dist.all_reduce(tensor)


def _exchange(tr, table, have_lo, have, add):
    """Rows of one map between the ranks.  have = this rank's rows have_lo.. of the map (N, C, rows, W).
    Forward (add=False): receive the rows of table['recv'][rank] from their owners; backward (add=True): the same
    rows travel the other way.  Sends first (they do not block on the queues; over torch.distributed the pairs
    are ordered by rank so that matching send/recv calls meet), returns [(lo, hi, tensor)] of what arrived."""
    got = []
    pairs = [(dst, src, a, b) for dst in range(tr.world) for src, a, b in table["recv"][dst]]
    for dst, src, a, b in pairs:
        sender, receiver = (dst, src) if add else (src, dst)
        if tr.rank == sender:
            tr.send(receiver, have[:, :, a - have_lo:b - have_lo + 1, :].contiguous())
        elif tr.rank == receiver:
            like = torch.empty((have.shape[0], have.shape[1], b - a + 1, have.shape[3]), dtype=have.dtype, device=have.device)
            got.append((a, b, tr.recv(sender, like)))
    return got


class LibraryGroup:
    """One requested group on one rank's slab, computed by the CUDA library (fp32 path)."""

    def __init__(self, glayers, N, c_in, hs, w_in, out_shape, device, **plan_opts):
        self.plan = ftp.ftp_plan(glayers, N, c_in, hs, w_in, (1, 1), ((1, len(glayers)),), **plan_opts)
        self.ws = self.plan.new_workspace(device)
        self.y = torch.empty(out_shape, device=device)

    def forward(self, slab, pg):
        ftp.ftp_forward(self.plan, slab, pg, self.y, self.ws)
        return self.y

    def backward(self, slab, dslab, pg, grad_out):
        dxs = torch.empty_like(slab)
        ftp.ftp_backward(self.plan, slab, dslab, pg, dxs, grad_out, self.ws)
        return dxs

    @staticmethod
    def sgd(params, grad, lr):
        ftp.ftp_sgd(params, grad, lr)


class RowShardedStep:
    """One rank of a row-sharded training step (see the module text).  `group_cls` computes a group on a slab:
    LibraryGroup (the CUDA library, fp32 path) unless a test puts another implementation with the same three methods
    in its place to drive the exchange logic on the CPU.

    layers, N, C, H, W, groups: the network and the requested grouping profile; x and target are the FULL batch
    tensors on every rank in this form (a loader would hand each rank its rows only); params is the full
    parameter vector, replicated.  `step` returns the loss of the global batch and leaves the updated parameters in
    `params`; `y_owned`, `dx_needed` and `grad` hold the rank's rows of the last map, its rows of the input
    gradient and the summed gradient afterwards.
    """

    def __init__(self, layers, N, C, H, W, groups, transport, device="cuda", group_cls=LibraryGroup, dtype=torch.float32,
                 **plan_opts):
        self.tr, self.device, self.group_cls = transport, device, group_cls
        self.layers, self.N = list(layers), N
        world, rank = transport.world, transport.rank
        self.shapes = synth.map_shapes(self.layers, C, H, W)
        rows = [s[1] for s in self.shapes]
        full = ftp.ftp_plan(layers, N, C, H, W, (world, 1), groups)          # spans only: never executed
        self.tables = dp.row_shard_tables(full, rows, world)
        self.goff = [0]
        for l in self.layers:
            self.goff.append(self.goff[-1] + (l.cout * l.cin * l.k * l.k + l.cout if l.kind == "conv" else 0))
        self.g = []
        for t in self.tables:
            first, last = t["first"], t["last"]
            lo, hi = t["needed_in"][rank]
            scale = rows[first - 1] // rows[last]
            top, bottom = lo % scale, (-(hi + 1)) % scale            # zero rows that align the slab to the group's stride
            c_in, w_in = self.shapes[first - 1][0], self.shapes[first - 1][2]
            c_out, h_out_full, w_out = self.shapes[last]
            hs = top + (hi - lo + 1) + bottom
            glayers = self.layers[first - 1:last]
            comp = group_cls(glayers, N, c_in, hs, w_in, (N, c_out, hs // scale, w_out), device, **plan_opts)
            self.g.append(dict(t=t, first=first, last=last, lo=lo, hi=hi, top=top, base=(lo - top) // scale, comp=comp,
                               slab=torch.zeros((N, c_in, hs, w_in), device=device, dtype=dtype)))
        self.grad = torch.zeros(self.goff[-1], device=device, dtype=dtype)

    def forward(self, x, params):
        rank, owned = self.tr.rank, None
        for gi, G in enumerate(self.g):
            t, lo, hi, top = G["t"], G["lo"], G["hi"], G["top"]
            slab = G["slab"]
            slab.zero_()
            if gi == 0:
                slab[:, :, top:top + hi - lo + 1, :] = x[:, :, lo:hi + 1, :]
            else:
                olo, oarr = owned
                a, b = max(olo, lo), min(olo + oarr.shape[2] - 1, hi)
                slab[:, :, top + a - lo:top + b - lo + 1, :] = oarr[:, :, a - olo:b - olo + 1, :]
                for a, b, buf in _exchange(self.tr, t, olo, oarr, add=False):
                    slab[:, :, top + a - lo:top + b - lo + 1, :] = buf
            pg = params[self.goff[G["first"] - 1]:self.goff[G["last"]]]
            G["y"] = G["comp"].forward(slab, pg)
            o1, o2 = t["owned_out"][rank]
            owned = (o1, G["y"][:, :, o1 - G["base"]:o2 - G["base"] + 1, :].contiguous())
        self.y_lo, self.y_owned = owned
        return owned

    def backward(self, params, dy_owned):
        """dy_owned: delta of the owned rows of the last map.  Fills self.grad (summed over the ranks) and
        self.dx_lo / self.dx_needed (this rank's contribution to the input gradient over its needed rows: rows
        that two ranks need are the sum of both contributions)."""
        rank = self.tr.rank
        self.grad.zero_()
        d_lo, d = self.y_lo, dy_owned
        for gi in range(len(self.g) - 1, -1, -1):
            G = self.g[gi]
            t, lo, hi, top = G["t"], G["lo"], G["hi"], G["top"]
            dslab = torch.zeros_like(G["y"])
            dslab[:, :, d_lo - G["base"]:d_lo - G["base"] + d.shape[2], :] = d
            pg = params[self.goff[G["first"] - 1]:self.goff[G["last"]]]
            gp = self.grad[self.goff[G["first"] - 1]:self.goff[G["last"]]]
            dxs = G["comp"].backward(G["slab"], dslab, pg, gp)
            dxs = dxs[:, :, top:top + hi - lo + 1, :]                    # the needed rows lo..hi
            if gi == 0:
                self.dx_lo, self.dx_needed = lo, dxs
                break
            i1, i2 = t["owned_in"][rank]
            mine = torch.zeros((dxs.shape[0], dxs.shape[1], i2 - i1 + 1, dxs.shape[3]), device=dxs.device, dtype=dxs.dtype)
            a, b = max(i1, lo), min(i2, hi)
            mine[:, :, a - i1:b - i1 + 1, :] = dxs[:, :, a - lo:b - lo + 1, :]
            for a, b, buf in _exchange(self.tr, t, lo, dxs, add=True):
                mine[:, :, a - i1:b - i1 + 1, :] += buf
            d_lo, d = i1, mine
        self.tr.all_reduce(self.grad)

    def step(self, x, target, params, lr):
        y_lo, y = self.forward(x, params)
        tgt = target[:, :, y_lo:y_lo + y.shape[2], :]
        m = float(target.numel())
        loss = ((y - tgt) ** 2).sum().reshape(1) / m
        self.tr.all_reduce(loss)
        self.backward(params, 2.0 * (y - tgt) / m)
        self.group_cls.sgd(params, self.grad, lr)
        return float(loss.item())


def run_threads(world, fn):
    """Runs fn(transport) for the ranks of a ThreadTransport group, one thread each; returns their results in rank
    order and re-raises the first exception."""
    trs = ThreadTransport.group(world)
    out, err = [None] * world, []

    def body(r):
        try:
            out[r] = fn(trs[r])
        except BaseException as e:      # noqa: BLE001 - surfaced below
            err.append(e)
            try:
                trs[r]._barrier.abort()
            except Exception:
                pass

    ts = [threading.Thread(target=body, args=(r,)) for r in range(world)]
    for t in ts:
        t.start()
    for t in ts:
        t.join()
    if err:
        raise err[0]
    return out


def gather_rows(parts, rows, add=False):
    """Assembles a full map (numpy) from per-rank (lo, tensor) row pieces; overlapping rows are summed if `add`
    (the input gradient), else they must not overlap (owned rows)."""
    n, c, _, w = parts[0][1].shape
    full = np.zeros((n, c, rows, w), dtype=np.float64)
    for lo, t in parts:
        a = t.detach().cpu().numpy().astype(np.float64)
        if add:
            full[:, :, lo:lo + a.shape[2], :] += a
        else:
            full[:, :, lo:lo + a.shape[2], :] = a
    return full
