"""Coordinate-sharded EFCP state: host-side orchestration only.

One optimizer state is split over several GPUs by ranges of coordinates (efcp_create_shard in
include/efcp.h).  A step is six phases; after each of the first five a small buffer (three
histograms of the Top-k threshold search, the tie counts, the m scalar products) is summed
over the shards.  This module calls the phases in order and performs those sums: with
torch.distributed (one shard per process, NCCL on GPUs) or, for several shards held by one
process on one device, by adding the buffers up directly.  Every step of the method itself
runs in the CUDA library.
"""
from typing import Callable, List, Optional, Sequence

import torch

N_PHASES = 6


def even_ranges(d: int, n: int, align: int = 2048) -> List[tuple]:
    """[lo, hi) of n shards of d coordinates: equal sizes rounded to `align`, ascending."""
    per = -(-d // n)
    per = -(-per // align) * align
    out = []
    for r in range(n):
        lo, hi = min(d, r * per), min(d, (r + 1) * per)
        out.append((lo, hi))
    assert all(hi > lo for lo, hi in out), "more shards than aligned pieces"
    return out


def sum_over_processes(group=None) -> Callable[[Sequence[torch.Tensor]], None]:
    """Exchange for one shard per process: an all-reduce (sum) of each buffer."""
    import torch.distributed as dist

    def reduce(buffers):
        for b in buffers:
            dist.all_reduce(b, op=dist.ReduceOp.SUM, group=group)
    return reduce


def sum_in_process(buffers: Sequence[torch.Tensor]) -> None:
    """Exchange for several shards in one process on one device: every buffer becomes the
    sum of all of them (in shard order, so every shard sees the same bits)."""
    total = buffers[0].clone()
    for b in buffers[1:]:
        total += b
    for b in buffers:
        b.copy_(total)


class ShardedStep:
    """Runs the phases of a step on the shards this process holds and exchanges the buffers.

    shards: objects with shard_phase(phase, grad=None, update=None, stream=None) and
    shard_buffer(phase) -> tensor (binding.Efcp handles made with shard=...).
    reduce: called after each of the phases 0..4 with the list of this process's buffers of
    that phase; must leave in every buffer the sum over all shards of the state."""

    def __init__(self, shards: Sequence, reduce: Callable[[Sequence[torch.Tensor]], None]):
        self.shards = list(shards)
        self.reduce = reduce

    def step(self, grads: Sequence[torch.Tensor], updates: Sequence[torch.Tensor],
             stream: Optional[torch.cuda.Stream] = None) -> None:
        assert len(grads) == len(updates) == len(self.shards)
        for phase in range(N_PHASES):
            for s, g, u in zip(self.shards, grads, updates):
                s.shard_phase(phase, grad=g if phase == 0 else None,
                              update=u if phase == N_PHASES - 1 else None, stream=stream)
            if phase < N_PHASES - 1:
                self.reduce([s.shard_buffer(phase) for s in self.shards])


def create_local_shards(binding, d: int, m: int, k: int, lam: float, n: int, flags: int = 0,
                        ranges: Optional[Sequence[tuple]] = None, row_cap: int = 0):
    """n shards of one state, all on the current device of this process."""
    ranges = list(ranges) if ranges is not None else even_ranges(d, n)
    assert len(ranges) == n
    return [binding.Efcp(hi - lo, m, row_cap, lam, flags, shard=(d, lo, hi, k, r, n))
            for r, (lo, hi) in enumerate(ranges)], ranges


def create_rank_shard(binding, d: int, m: int, k: int, lam: float, flags: int = 0,
                      group=None, row_cap: int = 0):
    """This process's shard of a state split over the processes of `group`."""
    import torch.distributed as dist
    n, r = dist.get_world_size(group), dist.get_rank(group)
    lo, hi = even_ranges(d, n)[r]
    return binding.Efcp(hi - lo, m, row_cap, lam, flags, shard=(d, lo, hi, k, r, n)), (lo, hi)
