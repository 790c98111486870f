"""Host-side plumbing for running the pruned VAR step on several GPUs of one node.

Selection, KV cache, sublayer caches and attention are all per image (the per-image mean of Eq. 4, the
per-image top-k of Algorithm 1), so images shard across ranks with NO data-path collective: every rank
is a replica holding the weights and its own images.  What is shared is only the measurement: the
slowest rank's device time and the total of forwarded tokens.  Backend-agnostic (nccl on GPUs, gloo in
the CPU tests)."""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


def world() -> Tuple[int, int]:
    """(rank, world_size); (0, 1) when no process group is up."""
    if dist.is_available() and dist.is_initialized():
        return dist.get_rank(), dist.get_world_size()
    return 0, 1


def image_shard(n_images: int, rank: int, world_size: int) -> range:
    """Images [lo, hi) of a global batch owned by `rank`: contiguous, disjoint, covering, sizes differing
    by at most one (the first n_images % world_size ranks take one more)."""
    if n_images < 0 or world_size <= 0 or not (0 <= rank < world_size):
        raise ValueError("bad shard request")
    base, extra = divmod(n_images, world_size)
    lo = rank * base + min(rank, extra)
    return range(lo, lo + base + (1 if rank < extra else 0))


def rank_seed(base_seed: int, rank: int) -> int:
    """Replicas draw their own token maps (weak scaling: per-GPU work fixed) from distinct seeds."""
    return base_seed + 7919 * rank


def max_over_ranks(value: float, device=None) -> float:
    """Slowest rank's time: the only number that crosses ranks."""
    r, w = world()
    if w == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device=None) -> float:
    r, w = world()
    if w == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def aggregate_throughput(units_local: float, seconds_local: float, device=None) -> float:
    """Whole-job throughput: units processed by all ranks / the slowest rank's time."""
    return sum_over_ranks(units_local, device) / max_over_ranks(seconds_local, device)


def barrier() -> None:
    if world()[1] > 1:
        dist.barrier()
