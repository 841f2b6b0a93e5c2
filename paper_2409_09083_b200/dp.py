"""Data-parallel replicas: the one exchange step of the path across GPUs.

Every rank runs the one-GPU path on its own share of the batch and obtains the fixed-order sum of
its partial filter-gradient sets.  The paper sums the sets of all tiles one time per batch on a common
device (Section 4.1); across GPUs that sum is an all-reduce.  Each rank's loss is the mean over ITS
images, so the gradient of the mean over the global batch is the all-reduced sum divided by the
number of ranks, which is folded into the learning rate.

Two forms.  `allreduce_and_update`: the whole gradient after the step (`ftp_step_grad`).
`OverlappedExchange`: the gradient slice of every executed group is all-reduced as soon as the library
reports it complete (`ftp_step_grad_groups`; groups finish last layer first), on a communication
stream, while the groups before it are still being back-propagated on the compute stream.
"""


def shard_range(total: int, rank: int, world: int):
    """Images [lo, hi) of a global batch that `rank` of `world` processes (equal partition)."""
    return total * rank // world, total * (rank + 1) // world


def allreduce_and_update(grad, lr, world, all_reduce, sgd):
    """`all_reduce(grad)` sums in place over ranks; `sgd(grad, lr_eff)` applies w -= lr_eff * grad."""
    if world > 1:
        all_reduce(grad)
    sgd(grad, lr / world)


class OverlappedExchange:
    """The exchange of one training step, slice by slice.

    grad        flat gradient tensor the step writes (device or host)
    all_reduce  all_reduce(tensor_view) -> handle with .wait() or None; sums in place over the ranks
    order_after called before a slice's all-reduce is started: makes the communication side wait for the
                compute work queued so far (CUDA: record an event on the compute stream and let the
                communication stream wait for it; CPU tensors: nothing to do)
    `ready` is the callback for ftp_step_grad_groups; `finish` waits for all slices and applies the update.
    """

    def __init__(self, grad, world, all_reduce, order_after=None):
        self.grad, self.world, self.all_reduce, self.order_after = grad, world, all_reduce, order_after
        self.handles, self.slices = [], []

    def ready(self, group, begin, count):
        self.slices.append((group, begin, count))
        if self.world > 1 and count > 0:
            if self.order_after is not None:
                self.order_after()
            h = self.all_reduce(self.grad[begin:begin + count])
            if h is not None:
                self.handles.append(h)

    def finish(self, lr, sgd, join=None):
        """Waits for the slices in flight (`join()`: make the compute side wait for the communication side),
        checks that the reported slices cover the gradient exactly once, and applies w -= (lr / world) * grad."""
        for h in self.handles:
            h.wait()
        if join is not None:
            join()
        covered = sorted((b, b + c) for _, b, c in self.slices if c > 0)
        pos = 0
        for b, e in covered:
            if b != pos:
                raise RuntimeError(f"gradient slices do not tile the parameters: gap or overlap at {pos} (next slice starts at {b})")
            pos = e
        if pos != self.grad.numel():
            raise RuntimeError(f"gradient slices cover {pos} of {self.grad.numel()} parameters")
        sgd(self.grad, lr / self.world)
        self.handles, self.slices = [], []


def cuda_overlap(torch, dist, grad, world):
    """An OverlappedExchange over NCCL: all-reduces run on a communication stream of their own."""
    compute = torch.cuda.current_stream()
    comm = torch.cuda.Stream()

    def order_after():
        ev = torch.cuda.Event()
        ev.record(compute)
        comm.wait_event(ev)

    def all_reduce(view):
        with torch.cuda.stream(comm):
            return dist.all_reduce(view, async_op=True)

    ex = OverlappedExchange(grad, world, all_reduce, order_after)
    ex.join = lambda: compute.wait_stream(comm)
    return ex


# ---------------------------------------------------------------------------------------------
# Spatial sharding: tile rows across ranks (the paper's own partitioning, with a rank in the place
# of a device: Sections 3 and 4.2).  Host-side tables only; they come from the planner's spans.
# ---------------------------------------------------------------------------------------------
def equal_rows(extent: int, rank: int, world: int):
    """Rows [lo, hi] (inclusive) of a map of `extent` rows that `rank` owns: the equal partition of Section 4.2."""
    return extent * rank // world, extent * (rank + 1) // world - 1


def row_shard_tables(plan, map_rows, world):
    """Exchange tables of a row split over `world` ranks, rank r taking user tile (r, 0) of a plan created
    with tile grid (world, 1).

    map_rows[l - 1] = rows of map X_l (l = 1 .. L + 1).  Returns, per requested group g, a dict with
      first, last            the group's layers
      owned_out[r]           rows of the group's output map rank r owns (equal partition)
      owned_in[r]            rows of the group's input map it owns (the previous group's partition)
      needed_in[r]           rows of the input map its stack reads (Eq. (1) through the whole group, clamped)
      recv[r]                [(source rank, lo, hi)]: rows of needed_in[r] that other ranks own -- the forward
                             boundary exchange at the group input; in the backward pass the same rows travel
                             the other way and are ADDED at their owner (overlapping input deltas)
    The first group's input is the network input, which the host scatters: every rank is handed its
    needed rows, recv is empty.
    """
    out = []
    for g, (first, last) in enumerate(plan.groups):
        h_in, h_out = map_rows[first - 1], map_rows[last]
        entry = dict(first=first, last=last, owned_out=[], owned_in=[], needed_in=[], recv=[])
        for r in range(world):
            x1, y1, x2, y2 = plan.region(0, g, first, r, 0)
            entry["owned_out"].append(equal_rows(h_out, r, world))
            entry["owned_in"].append(equal_rows(h_in, r, world))
            entry["needed_in"].append((y1, y2))
        for r in range(world):
            lo, hi = entry["needed_in"][r]
            recv = []
            if g > 0:
                for src in range(world):
                    if src == r:
                        continue
                    a, b = entry["owned_in"][src]
                    a, b = max(a, lo), min(b, hi)
                    if a <= b:
                        recv.append((src, a, b))
            entry["recv"].append(recv)
        out.append(entry)
    return out
