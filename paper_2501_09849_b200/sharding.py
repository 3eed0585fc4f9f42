"""Data-parallel sharding of a CDL layer step: which rows a rank owns and what the ranks exchange, and when.

The quantizer passes and the forward / dX products act on each batch row independently, and the weights are
replicated, so everything computed from the weights alone (their indices, histogram, entropy, dL/dq, dL/dalpha)
is identical on every rank and is never exchanged.  Three results are sums over the global batch, and each is
exchanged at the point of the step where the global value is first needed:

  1. the level histogram of the activations - all-reduced (uint64 counts, exact) BEFORE cdl_index_entropy, so
     that every rank gets H(x) and the level probabilities of the whole batch and its quantizer backward pass
     differentiates through those (entropies themselves are never summed);
  2. the int32 accumulators of the weight-gradient product - all-reduced as integers (widened to int64 when the
     sum over all ranks could leave int32) BEFORE the single conversion to float (cdl_rescale_acc), so that dW has
     the bits of one product over the whole batch whatever the number of ranks;
  3. the two scalar gradients of the activation quantizer (dL/ds, dL/dbeta) - fp64 sums, all-reduced at the end.

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


def acc_bits_for(rows_global: int, absmax_a: int, absmax_g: int) -> int:
    """Width the weight-gradient accumulators need for the all-reduce: 32 while the sum over the global batch is
    bounded below 2^31 for the declared index ranges, else 64."""
    return 32 if rows_global * absmax_a * absmax_g < (1 << 31) else 64


class StepExchange:
    """The exchange points of a data-parallel layer step (see the module text).  `dist` is torch.distributed (or
    anything with all_reduce / ReduceOp); every method sums in place over the ranks and is a no-op for one rank."""

    def __init__(self, dist, world: int):
        self.dist, self.world = dist, int(world)
        self.calls = []          # (name, dtype, numel) of every exchange, for tests and launch counting

    def _sum(self, name, t, dtypes):
        if str(t.dtype).replace("torch.", "") not in dtypes:
            raise TypeError(f"{name}: exchanged as {t.dtype}, expected one of {dtypes}")
        self.calls.append((name, str(t.dtype).replace("torch.", ""), int(t.numel())))
        if self.world > 1:
            self.dist.all_reduce(t, op=self.dist.ReduceOp.SUM)
        return t

    def histogram(self, hist):
        """uint64 level counts (held as int64 tensors): before the entropy / level probabilities are taken."""
        return self._sum("histogram", hist, ("int64",))

    def accumulators(self, acc):
        """Integer accumulators of dW: before the one conversion to float."""
        return self._sum("accumulators", acc, ("int32", "int64"))

    def batch_scalars(self, scal):
        """fp64 sums over the batch (dL/ds, dL/dbeta of the activation quantizer) - and nothing else: entropies
        and the weight quantizer's dL/dq, dL/dalpha are the same on every rank."""
        return self._sum("batch_scalars", scal, ("float64",))
