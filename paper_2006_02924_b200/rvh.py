"""Recursive vector-halving Adasum across ranks: one gradient per GPU (Algorithm 1, Section 4.2.1).

Every rank starts with its own full gradient.  Level by level (neighbour distance 1, 2, 4, ...)
a rank swaps half of what it holds with its neighbour, computes the per-tensor
[a.b, a.a, b.b] of the two halves it now has, adds those over the 2 x distance ranks that
together hold the whole of the two operands, applies the operator to its half, and recurses on
the result; an all-gather phase (the same exchanges backwards) rebuilds the full vector on every
rank.  The tree is the bottom-up one of the single-GPU reduce with N = number of ranks: ranks
2 i and 2 i + 1 are combined first.

Layers of this module:

* ``rvh_schedule``  host arithmetic only: who talks to whom about which element range.
* ``rvh_steps``     the algorithm for one rank, written as a generator that yields its
                    communication steps (``Exchange``, ``AllReduce``) and leaves the arithmetic to a
                    ``kernels`` object.  Nothing in it touches torch.distributed, so the same code
                    runs under a real process group and under a test's in-process lock-step driver.
* ``CudaKernels``   the arithmetic: ``adasum_sharded_gram`` / ``adasum_sharded_apply`` of the C
                    ABI with the two halves as operands.  There is no CPU implementation here.
* ``AdasumRVH``     the user-facing object: runs ``rvh_steps`` over a torch.distributed group
                    (NCCL on GPUs): send/recv pairs for the exchanges, one all-reduce per level
                    over the sub-group of 2 x distance ranks.
"""
from __future__ import annotations

import dataclasses
from typing import Iterator, Sequence

import numpy as np
import torch

_ALIGN = 64          # elements; split points sit on this grid when the range is long enough


@dataclasses.dataclass(frozen=True)
class RvhLevel:
    distance: int
    neighbor: int
    left: bool                  # floor(rank / distance) is even: keeps the lower half
    lo: int
    mid: int
    hi: int                     # [lo, hi) is held on entry; split at mid
    group: tuple[int, ...]      # the 2 x distance ranks that share the two operands

    @property
    def keep(self) -> tuple[int, int]:
        return (self.lo, self.mid) if self.left else (self.mid, self.hi)

    @property
    def give(self) -> tuple[int, int]:
        return (self.mid, self.hi) if self.left else (self.lo, self.mid)


def rvh_schedule(rank: int, size: int, total: int) -> list[RvhLevel]:
    """The levels of Algorithm 1 for ``rank`` of ``size`` ranks reducing ``total`` elements."""
    if size < 1 or size & (size - 1):
        raise ValueError(f"the number of ranks must be a power of two (Algorithm 1), got {size}")
    if not 0 <= rank < size:
        raise ValueError(f"rank {rank} outside 0..{size - 1}")
    if total < size:
        raise ValueError(f"{total} elements cannot be halved over {size} ranks")
    levels = []
    lo, hi, d = 0, int(total), 1
    while d < size:
        mid = lo + (hi - lo) // 2
        if hi - lo >= 4 * _ALIGN:
            mid = mid // _ALIGN * _ALIGN
        left = (rank // d) % 2 == 0
        base = rank // (2 * d) * (2 * d)
        lv = RvhLevel(distance=d, neighbor=rank + d if left else rank - d, left=left, lo=lo, mid=mid, hi=hi,
                      group=tuple(range(base, base + 2 * d)))
        levels.append(lv)
        lo, hi = lv.keep
        d *= 2
    return levels


def clip_offsets(tensor_offsets: Sequence[int], lo: int, hi: int) -> np.ndarray:
    """Tensor boundaries of the slice [lo, hi) of the fused buffer, relative to lo.  Every tensor
    keeps its index; tensors outside the slice become empty."""
    offs = np.asarray(tensor_offsets, dtype=np.int64)
    return np.clip(offs, lo, hi) - lo


@dataclasses.dataclass
class Exchange:
    """Send ``send`` to ``peer`` and receive the same number of elements from it into ``recv``."""
    peer: int
    send: torch.Tensor
    recv: torch.Tensor


@dataclasses.dataclass
class AllReduce:
    """Add ``tensor`` (fp64) over ``ranks`` in place."""
    ranks: tuple[int, ...]
    tensor: torch.Tensor


def rvh_steps(rank: int, size: int, x: torch.Tensor, tensor_offsets: Sequence[int], kernels) -> Iterator:
    """Algorithm 1 on one rank.  Yields ``Exchange`` / ``AllReduce`` steps; the caller performs each
    before resuming the generator.  The generator's return value (StopIteration.value) is the
    full reduced vector, fp32.

    ``kernels`` supplies the arithmetic and the memory:
      empty(n, dtype, like)                 -> uninitialised 1-D scratch tensor beside ``like``
      result(n, like)                       -> uninitialised fp32 tensor for the final vector
      gram(a, b, offsets, level)            -> fp64 tensor of per-tensor [a.a, a.b, b.b] sums of
                                               this rank's slices, to be added over the group in place
      apply(a, b, offsets, level)           -> fp32 tensor, the operator applied with the summed values
    """
    total = x.numel()
    offsets = np.asarray(tensor_offsets, dtype=np.int64)
    if offsets[0] != 0 or offsets[-1] != total:
        raise ValueError("tensor_offsets must start at 0 and end at the number of elements")
    schedule = rvh_schedule(rank, size, total)
    cur, cur_lo = x, 0
    for level, lv in enumerate(schedule):
        keep_lo, keep_hi = lv.keep
        give_lo, give_hi = lv.give
        mine = cur[keep_lo - cur_lo:keep_hi - cur_lo]
        recv = kernels.empty(keep_hi - keep_lo, cur.dtype, cur)
        yield Exchange(lv.neighbor, cur[give_lo - cur_lo:give_hi - cur_lo], recv)
        # a is the left neighbour's data, b the right neighbour's
        a, b = (mine, recv) if lv.left else (recv, mine)
        local = clip_offsets(offsets, keep_lo, keep_hi)
        sums = kernels.gram(a, b, local, level)
        yield AllReduce(lv.group, sums)
        cur, cur_lo = kernels.apply(a, b, local, level), keep_lo
    result = kernels.result(total, x)
    if schedule:
        lo, hi = schedule[-1].keep
        result[lo:hi].copy_(cur)
    else:
        result.copy_(x)
    for lv in reversed(schedule):
        keep_lo, keep_hi = lv.keep
        give_lo, give_hi = lv.give
        yield Exchange(lv.neighbor, result[keep_lo:keep_hi], result[give_lo:give_hi])
    return result


class CudaKernels:
    """The arithmetic of ``rvh_steps`` on this rank's GPU, through the C ABI.  Scratch tensors and
    workspaces are kept between reduces (the k-th request of a reduce gets the k-th buffer of its
    size again); the result is a fresh tensor every time."""

    def __init__(self, flags: int = 0):
        from . import binding

        self._lib = binding
        self._flags = flags
        self._workspaces: dict = {}
        self._buffers: dict = {}
        self._requests: dict = {}

    def begin(self) -> None:
        """Start of a reduce: scratch requests count from zero again."""
        self._requests = {}

    @staticmethod
    def _check(like) -> None:
        if not like.is_cuda:
            raise RuntimeError(f"AdasumRVH computes on the GPU only; got a tensor on {like.device}")

    def empty(self, n, dtype, like):
        self._check(like)
        kind = (int(n), dtype, like.device)
        slot = self._requests.get(kind, 0)
        self._requests[kind] = slot + 1
        buf = self._buffers.get(kind + (slot,))
        if buf is None:
            buf = self._buffers[kind + (slot,)] = torch.empty(int(n), dtype=dtype, device=like.device)
        return buf

    def result(self, n, like):
        self._check(like)
        return torch.empty(int(n), dtype=torch.float32, device=like.device)

    def _workspace(self, a, offsets, level):
        key = (level, a.numel(), a.dtype, a.device)
        ws = self._workspaces.get(key)
        if ws is None:
            need = self._lib.adasum_workspace_bytes(a.numel(), len(offsets) - 1, 2, a.dtype, self._flags)
            ws = self._workspaces[key] = torch.empty(max(need, 256), dtype=torch.uint8, device=a.device)
        return ws

    def gram(self, a, b, offsets, level):
        return self._lib.adasum_sharded_gram([a, b], offsets, self._workspace(a, offsets, level), 0,
                                             flags=self._flags)

    def apply(self, a, b, offsets, level):
        out = self.empty(a.numel(), torch.float32, a)
        self._lib.adasum_sharded_apply([a, b], offsets, out, self._workspace(a, offsets, level), 0,
                                       flags=self._flags)
        return out


class AdasumRVH:
    """``y = AdasumRVH(group)(x, tensor_offsets)``: every rank passes its own gradient ``x`` (fp32,
    fp16 or bf16, the whole fused buffer) and gets the Adasum of all ranks' gradients, fp32.  All
    ranks of ``group`` must call it together.  The number of ranks must be a power of two."""

    def __init__(self, group=None, kernels=None):
        import torch.distributed as dist

        self._dist = dist
        self._group = group
        self._rank = dist.get_rank(group)
        self._size = dist.get_world_size(group)
        self._kernels = kernels if kernels is not None else CudaKernels()
        self._subgroups: dict = {}

    def _subgroup(self, ranks: tuple[int, ...]):
        """The process group of ``ranks`` (indices within ``self._group``).  Creating a group is a
        collective over the parent, so all of them are made on first use, in one fixed order."""
        if len(ranks) == self._size:
            return self._group
        if not self._subgroups:
            dist = self._dist
            width = 2
            while width < self._size:
                for base in range(0, self._size, width):
                    members = tuple(range(base, base + width))
                    global_ranks = [self._global(r) for r in members]
                    self._subgroups[members] = dist.new_group(global_ranks)
                width *= 2
        return self._subgroups[ranks]

    def _global(self, r: int) -> int:
        return r if self._group is None else self._dist.get_global_rank(self._group, r)

    def __call__(self, x: torch.Tensor, tensor_offsets=None) -> torch.Tensor:
        dist = self._dist
        if tensor_offsets is None:
            tensor_offsets = [0, x.numel()]
        if hasattr(self._kernels, "begin"):
            self._kernels.begin()
        steps = rvh_steps(self._rank, self._size, x, tensor_offsets, self._kernels)
        try:
            step = next(steps)
            while True:
                if isinstance(step, Exchange):
                    peer = self._global(step.peer)
                    ops = [dist.P2POp(dist.isend, step.send, peer, self._group),
                           dist.P2POp(dist.irecv, step.recv, peer, self._group)]
                    for req in dist.batch_isend_irecv(ops):
                        req.wait()
                else:
                    if step.tensor.numel() > 0:
                        dist.all_reduce(step.tensor, op=dist.ReduceOp.SUM, group=self._subgroup(step.ranks))
                step = next(steps)
        except StopIteration as done:
            return done.value
