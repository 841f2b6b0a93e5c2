"""Data-parallel replicas: the one exchange step of the path across GPUs.

Every rank runs the one-GPU path on its own share of the batch and obtains the fixed-order sum of
its partial filter-gradient sets (`ftp_step_grad`).  The paper sums the sets of all tiles once per
batch on a common device (Section 4.1); across GPUs that sum is an all-reduce.  Each rank's loss
is the mean over ITS images, so the gradient of the mean over the global batch is the all-reduced
sum divided by the number of ranks, which is folded into the learning rate.
"""


def shard_range(total: int, rank: int, world: int):
    """Images [lo, hi) of a global batch that `rank` of `world` processes (equal partition)."""
    return total * rank // world, total * (rank + 1) // world


def allreduce_and_update(grad, lr, world, all_reduce, sgd):
    """`all_reduce(grad)` sums in place over ranks; `sgd(grad, lr_eff)` applies w -= lr_eff * grad."""
    if world > 1:
        all_reduce(grad)
    sgd(grad, lr / world)
