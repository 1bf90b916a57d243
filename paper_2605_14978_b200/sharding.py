"""Window sharding across GPUs: one process per GPU, windows partitioned contiguously.

Windows are independent through the row reduction and the window scan, so each rank scores its own
slice with no communication.  Only ADAW's ranking is global (Sec. 4.2: the windows with the largest
``s_j`` over the whole batch are kept): the ``[N_r]`` score shards are all-gathered (a few KB) and
every rank runs the same deterministic selection over the global score array, so all ranks agree on
the kept set without a broadcast.  No logit ever leaves the GPU that holds it.

This module is host-side plumbing only: index arithmetic and one ``torch.distributed`` collective.
The selection itself is the CUDA library's (``binding.select_windows``); a different callable can be
injected for process groups that have no GPU.
"""
from __future__ import annotations

from typing import Callable, List, Optional, Tuple

import torch


def window_range(n_total: int, world: int, rank: int) -> Tuple[int, int]:
    """Half-open range of global window indices owned by ``rank``: contiguous, sizes differ by at most one,
    the first ``n_total % world`` ranks take the extra window."""
    if world < 1 or not (0 <= rank < world) or n_total < 0:
        raise ValueError("bad partition request: n_total=%d world=%d rank=%d" % (n_total, world, rank))
    base, extra = divmod(n_total, world)
    start = rank * base + min(rank, extra)
    return start, start + base + (1 if rank < extra else 0)


def shard_sizes(n_total: int, world: int) -> List[int]:
    return [window_range(n_total, world, r)[1] - window_range(n_total, world, r)[0] for r in range(world)]


def owner_of(window: int, n_total: int, world: int) -> Tuple[int, int]:
    """(rank, local index) of a global window index under ``window_range``."""
    if not (0 <= window < n_total):
        raise ValueError("window %d outside [0, %d)" % (window, n_total))
    base, extra = divmod(n_total, world)
    split = extra * (base + 1)
    if window < split:
        r = window // (base + 1)
        return r, window - r * (base + 1)
    r = extra + (window - split) // base
    return r, window - split - (r - extra) * base


def gather_scores(local_score: torch.Tensor, n_total: int, group=None) -> torch.Tensor:
    """All-gather the per-rank score shards into the global ``[n_total]`` score array (same on every rank).

    The one exchange step of the path.  CUDA shards take one ``all_gather_into_tensor`` (NCCL, on the current
    stream), ragged shards padded to the largest shard and trimmed afterwards; host tensors (gloo) use
    ``all_gather``."""
    import torch.distributed as dist
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    sizes = shard_sizes(n_total, world)
    if local_score.numel() != sizes[rank]:
        raise ValueError("rank %d holds %d scores, its shard of %d windows has %d"
                         % (rank, local_score.numel(), n_total, sizes[rank]))
    local_score = local_score.contiguous()
    width = max(sizes)
    if local_score.is_cuda:
        # one code path for equal and ragged shards (so that a one-rank group exercises all of it): every rank
        # contributes `width` scores, its own shard padded with zeros, in one NCCL all-gather on the current stream
        if sizes[rank] == width:
            padded = local_score
        else:
            padded = torch.zeros((width,), dtype=local_score.dtype, device=local_score.device)
            padded[: sizes[rank]].copy_(local_score)
        flat = torch.empty((world * width,), dtype=local_score.dtype, device=local_score.device)
        dist.all_gather_into_tensor(flat, padded, group=group)
        if len(set(sizes)) == 1:
            return flat
        return torch.cat([p[:s] for p, s in zip(flat.split(width), sizes)])
    if len(set(sizes)) == 1:
        out = torch.empty((n_total,), dtype=local_score.dtype, device=local_score.device)
        dist.all_gather(list(out.split(sizes[0])), local_score, group=group)
        return out
    padded = torch.zeros((width,), dtype=local_score.dtype, device=local_score.device)
    padded[: sizes[rank]].copy_(local_score)
    parts = [torch.empty_like(padded) for _ in range(world)]
    dist.all_gather(parts, padded, group=group)
    return torch.cat([p[:s] for p, s in zip(parts, sizes)])


def local_part(selected_global: torch.Tensor, n_total: int, world: int, rank: int) -> torch.Tensor:
    """Local indices (order of ``selected_global`` kept) of the selected windows this rank owns."""
    start, end = window_range(n_total, world, rank)
    mine = (selected_global >= start) & (selected_global < end)
    return selected_global[mine] - start


def sharded_select(local_score: torch.Tensor, n_total: int, n_keep: int, group=None,
                   select_fn: Optional[Callable] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Global ADAW selection from per-rank score shards.

    Returns ``(selected_global [n_keep], selected_local)``: the global indices of the kept windows in
    (score descending, index ascending) order, identical on every rank, and the local indices of those
    this rank owns.  ``select_fn(scores, n_keep)`` defaults to the CUDA library's selection."""
    import torch.distributed as dist
    if select_fn is None:
        from . import binding
        select_fn = binding.select_windows
    scores = gather_scores(local_score, n_total, group)
    selected = select_fn(scores, n_keep)
    return selected, local_part(selected, n_total, dist.get_world_size(group), dist.get_rank(group))
