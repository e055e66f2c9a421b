"""Host-side plumbing for running one mesh dimension across several GPUs (one process per GPU).

The library decides WHAT has to be summed across ranks (mtf_layout_bind_ranks: every einsum or
reduction that sums out a dimension split over the rank-spanning mesh dimension - Algorithm 1 line 2
for a batch split, the Allreduce of y and dx of Section 8.2 for a split of the hidden dimension) and
calls two hooks: "start a sum over all ranks of these values, behind what is queued on this stream"
and "make this stream wait for the sums started so far".  This module provides those hooks over
torch.distributed (NCCL on GPUs, gloo in the CPU tests).  It holds no arithmetic of the method.
"""
from __future__ import annotations

import ctypes

from .binding import MTF_BF16, RANK_ALLREDUCE_FN, RANK_WAIT_FN


class _CudaView:
    """Wraps a raw device pointer so that torch.as_tensor can view it (no copy, no ownership)."""

    def __init__(self, ptr: int, count: int, typestr: str):
        self.__cuda_array_interface__ = {"shape": (count,), "typestr": typestr, "data": (ptr, False), "version": 2}


def tensor_from_pointer(ptr: int, count: int, dtype_code: int, device: str):
    """A 1-d torch tensor over ``count`` values at ``ptr`` (bf16 or f32), on ``device`` ("cuda" / "cpu")."""
    import numpy as np
    import torch
    if device == "cpu":
        ctype = ctypes.c_uint16 if dtype_code == MTF_BF16 else ctypes.c_float
        arr = np.ctypeslib.as_array((ctype * count).from_address(ptr))
        t = torch.from_numpy(arr.view(np.int16) if dtype_code == MTF_BF16 else arr)
    else:
        t = torch.as_tensor(_CudaView(ptr, count, "<i2" if dtype_code == MTF_BF16 else "<f4"), device=device)
    return t.view(torch.bfloat16) if dtype_code == MTF_BF16 else t


class RankCollective:
    """The two hooks of mtf_layout_bind_ranks over a torch.distributed process group.

    ``start`` enqueues an in-place all-reduce (sum) without blocking the host: with NCCL the collective
    runs on the group's own stream after the launches already queued on the caller's stream, so it
    overlaps whatever the caller launches next; ``wait`` makes the caller's stream wait for every
    all-reduce started since the last wait.  ``log`` records (count, dtype) of every sum started."""

    def __init__(self, dist, device: str = "cuda", group=None):
        self.dist, self.device, self.group = dist, device, group
        self.pending = []
        self.log = []
        self.error = None
        self.start_cb = RANK_ALLREDUCE_FN(self._start)
        self.wait_cb = RANK_WAIT_FN(self._wait)

    def _start(self, user, data, count, dtype, stream):
        try:
            t = tensor_from_pointer(int(data), int(count), int(dtype), self.device)
            self.log.append((int(count), int(dtype)))
            self.pending.append(self.dist.all_reduce(t, group=self.group, async_op=True))
            return 0
        except Exception as e:      # nothing may propagate through the C frames
            self.error = e
            return 9

    def _wait(self, user, stream):
        try:
            for work in self.pending:
                work.wait()
            self.pending = []
            return 0
        except Exception as e:
            self.error = e
            return 9


def rank_block(extent: int, world: int, rank: int):
    """Contiguous block [start, stop) of a dimension of size ``extent`` owned by ``rank`` of ``world``."""
    if extent % world != 0:
        raise ValueError(f"dimension of size {extent} is not divisible by {world} ranks")
    t = extent // world
    return rank * t, (rank + 1) * t


def max_over_ranks(dist, value: float, device="cpu") -> float:
    """The slowest rank's value (timings of a multi-rank step are reported as the maximum)."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
