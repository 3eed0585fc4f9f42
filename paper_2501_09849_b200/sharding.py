"""Data-parallel sharding of a CDL layer step: which rows a rank owns and what the ranks exchange.

The quantizer passes and the forward / dX products act on each batch row independently; the weight-side
results (dW, the level histograms, the summed scalar gradients) are sums over the global batch.  A rank
therefore runs the unchanged kernels on its contiguous block of rows and the ranks all-reduce those sums -
integers for the histogram and the dW accumulators, so the result does not depend on the rank count.
Only plumbing lives here (index arithmetic and torch.distributed calls); no arithmetic of the method.
"""
from __future__ import annotations


def row_range(n_rows: int, rank: int, world: int):
    """Contiguous block [start, stop) of rank `rank`; the first n_rows % world ranks get one extra row."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    base, extra = divmod(n_rows, world)
    start = rank * base + min(rank, extra)
    return start, start + base + (1 if rank < extra else 0)


def exchange(dist, world: int, *tensors):
    """Sum every tensor over the ranks in place (no-op for a single rank)."""
    if world <= 1:
        return
    for t in tensors:
        if t is not None:
            dist.all_reduce(t, op=dist.ReduceOp.SUM)
