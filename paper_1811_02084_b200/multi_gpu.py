"""Host-side plumbing for running one mesh dimension across several GPUs (one process per GPU).

The paper's data-parallel layout (Section 8.1, Algorithm 1) splits `batch` over a mesh dimension; when
that mesh dimension is mapped onto physical GPUs every rank holds the processors whose coordinate on
it is the rank, i.e. one contiguous block of the batch (Section 5), runs the block on its shard, and
the parameter gradients - einsums that reduce out `batch` - are summed across ranks (Algorithm 1,
line 2).  Nothing else is exchanged.  These helpers carry no arithmetic of the method and work with
any torch.distributed backend (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations


def rank_block(extent: int, world: int, rank: int):
    """Contiguous block [start, stop) of a dimension of size ``extent`` owned by ``rank`` of ``world``."""
    if extent % world != 0:
        raise ValueError(f"dimension of size {extent} is not divisible by {world} ranks")
    t = extent // world
    return rank * t, (rank + 1) * t


def allreduce_gradients(dist, grads) -> None:
    """Sum every tensor of ``grads`` over all ranks, in place (Algorithm 1, line 2)."""
    if dist is None:
        return
    for g in grads:
        dist.all_reduce(g)


class GradientSync:
    """Sums gradients over the ranks while later kernels of the backward pass still run: ``start`` is
    called right after the launch that produces a gradient and enqueues its all-reduce without
    blocking (the collective waits for that launch on its own stream), ``finish`` makes the calling
    stream wait for every all-reduce started since.  With one rank (``dist`` None) both do nothing."""

    def __init__(self, dist):
        self.dist = dist
        self.pending = []

    def start(self, tensor) -> None:
        if self.dist is not None:
            self.pending.append(self.dist.all_reduce(tensor, async_op=True))

    def finish(self) -> None:
        for work in self.pending:
            work.wait()
        self.pending = []


def max_over_ranks(dist, value: float, device="cpu") -> float:
    """The slowest rank's value (timings of a multi-rank step are reported as the maximum)."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
