"""Lloyd iterations over rows of X that are spread over the ranks of a torch.distributed group.

One process per GPU.  Every rank holds a contiguous share of the rows and all K centroids.  Per iteration
each rank assigns its rows and adds them up per cluster with this library's kernels, the sums and counts are
all-reduced over the group (NCCL on GPUs; the only exchange step of the method: K*D + K numbers per
iteration, whatever N is), and every rank divides, so all ranks hold the same centroids without a
broadcast; the inertia is all-reduced once at the end.  The paper describes the single-device iteration (Section 5, "Flash-KMeans clean-start
workload"); fp32 sums of different ranks are added in the order the all-reduce chooses.

Nothing here computes on tensors by itself: calls of the library and collectives only.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import binding
from .binding import LloydOutput


def shard_rows(N: int, rank: int, world: int) -> tuple[int, int]:
    """[first, last) rows of `rank` when N rows are dealt to `world` ranks in contiguous shares that differ by
    at most one row (the first N % world ranks get the longer ones)."""
    if world < 1 or not 0 <= rank < world or N < 0:
        raise ValueError("need 0 <= rank < world and N >= 0")
    q, r = divmod(N, world)
    first = rank * q + min(rank, r)
    return first, first + q + (1 if rank < r else 0)


def cake_kmeans_lloyd_sharded(X_local: torch.Tensor, C0: torch.Tensor, iters: int, group=None, flags: int = 0,
                              out: LloydOutput | None = None, ws: torch.Tensor | None = None) -> LloydOutput:
    """iters Lloyd iterations; X_local bf16 [N_local, D] are this rank's rows, C0 bf16 [K, D] the same on all ranks.

    Returns this rank's idx / dist (for its own rows) and the global C, counts and inertia.  Without an
    initialised process group (or with a group of one rank) it is the single-device iteration.
    The loop itself runs inside the library (cake_kmeans_lloyd_sharded of the C ABI); this function supplies the
    exchange: one all-reduce of the sums and one of the counts per iteration, and one of the inertia at the end.
    """
    if X_local.dim() != 2 or C0.dim() != 2 or X_local.shape[1] != C0.shape[1]:
        raise ValueError("X_local must be [N_local, D] and C0 [K, D]")
    N, D = X_local.shape
    K = C0.shape[0]
    dev = X_local.device
    exchange = dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1
    if iters == 0:
        return binding.cake_kmeans_lloyd(X_local, C0, 0)
    if ws is None:
        ws = binding.alloc_workspace(1, N, D, K, dev)
    if out is None:
        out = binding.alloc_lloyd_outputs(X_local, C0, iters)

    def reduce(sums, counts):
        dist.all_reduce(sums, group=group)
        dist.all_reduce(counts, group=group)

    binding.cake_kmeans_lloyd_sharded_call(X_local, C0, iters, out, ws, reduce if exchange else None, flags=flags)
    if exchange:
        dist.all_reduce(out.inertia, group=group)
    return out
