"""Key-range sharded recall: one rank per GPU, each holding a contiguous range of the context's
keys at the retrieval layer and the whole query.

Eq. 4's softmax runs over all keys, so the ranks exchange twice: the per-row softmax statistics
of their shards (2 floats per query row), then the scores of their positions (one float per
position).  Algorithm 1 then runs replicated on every rank from the gathered scores, so every
rank ends with the same index list and no third exchange is needed.  All arithmetic is in the
library's kernels; this module only moves the two tensors with ``torch.distributed``.
"""
from __future__ import annotations

from typing import Optional, Sequence, Tuple

import torch
import torch.distributed as dist


def shard_bounds(L: int, world: int, rank: int, align: int = 128) -> Tuple[int, int]:
    """[begin, end) of rank's key range: ranges are contiguous, in rank order, cover [0, L),
    and every boundary except L itself is a multiple of ``align`` (one key tile), so that no
    rank gets a ragged first tile.  Late ranks may be empty when L is small."""
    assert L >= 0 and world >= 1 and 0 <= rank < world and align >= 1
    tiles = (L + align - 1) // align
    lo = (tiles * rank // world) * align
    hi = (tiles * (rank + 1) // world) * align
    return min(lo, L), min(hi, L)


def sharded_recall(engine, K_shard: torch.Tensor, Q: torch.Tensor, L: int, budget: int,
                   max_sizes: Sequence[int], win_sizes: Sequence[int], win_op: int = 0,
                   n_sink: int = 0, group: Optional[dist.ProcessGroup] = None,
                   want_scores: bool = False):
    """One recall over keys sharded by ``shard_bounds(L, world, rank)``.

    ``engine`` provides ``shard_stats``, ``shard_scores`` and ``allocate`` (an ``IlreRecall``
    whose ``max_L`` covers the whole context: the allocation step sees all L scores).
    K_shard: this rank's rows [begin, end) of the key cache; Q: the full query on every rank.
    Returns the ascending indices (identical on every rank) and, if asked, the scores [L].
    """
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    lo, hi = shard_bounds(L, world, rank)
    assert K_shard.shape[0] == hi - lo, "K_shard does not match this rank's key range"
    bounds = [shard_bounds(L, world, r) for r in range(world)]
    n_rows = Q.shape[0] * Q.shape[1]
    dev = Q.device

    # exchange 1: per-row (max, sum) of every shard.  An empty shard contributes (-inf, 0),
    # the identity of the merge.
    if hi > lo:
        mine = engine.shard_stats(K_shard, Q)
    else:
        mine = torch.empty(n_rows, 2, dtype=torch.float32, device=dev)
        mine[:, 0] = float("-inf")
        mine[:, 1] = 0.0
    flat = torch.empty(world * n_rows, 2, dtype=torch.float32, device=dev)
    dist.all_gather_into_tensor(flat, mine.contiguous(), group=group)
    stats_all = flat.view(world, n_rows, 2)

    # exchange 2: the scores of every position.  Shards differ in length by at most one
    # tile; pad to the longest so that one fixed-size all-gather serves.
    longest = max(b - a for a, b in bounds)
    padded = torch.zeros(longest, dtype=torch.float32, device=dev)
    if hi > lo:
        engine.shard_scores(K_shard, Q, stats_all, out=padded[:hi - lo])
    flat = torch.empty(world * longest, dtype=torch.float32, device=dev)
    dist.all_gather_into_tensor(flat, padded, group=group)
    all_padded = flat.view(world, longest)
    scores = torch.cat([all_padded[r, :b - a] for r, (a, b) in enumerate(bounds)])

    idx = engine.allocate(scores, budget, max_sizes, win_sizes, win_op, n_sink)
    return (idx, scores) if want_scores else (idx, None)
