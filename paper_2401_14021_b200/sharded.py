"""Row-sharded retrieval: the corpus is split by rows over ranks (one process per GPU), every
rank searches its own rows, the per-rank answers are all-gathered and merged on every rank.

Only plumbing lives here (the partition arithmetic and the collective); scoring, selection and
the merge run in the CUDA library (ralm_search, ralm_merge_lists). The one exchange of the path
is an all-gather of s * k (id, score) pairs per rank, 12 bytes each; gathered data lands in
local memory before the merge kernel reads it.
"""
from typing import Optional, Tuple

import torch

from . import binding


def shard_rows(N: int, world: int, rank: int, align: int = 256) -> Tuple[int, int]:
    """Rows [lo, hi) of `rank` when N rows are split contiguously over `world` ranks: equal
    shares rounded up to a multiple of `align` rows, the last ranks taking what is left."""
    if world < 1 or not 0 <= rank < world or N < 0:
        raise ValueError("bad partition")
    share = -(-N // world)
    share = -(-share // align) * align
    lo = min(N, rank * share)
    return lo, min(N, lo + share)


def gather_lists(ids: torch.Tensor, scores: torch.Tensor, row_lo: int, group=None):
    """All-gather of one rank's answer ([s][k] ids and scores) and of its first global row id.
    Returns (ids [G][s][k], scores [G][s][k], row_offset [G]), the same on every rank. Without an
    initialised process group this is the single-rank case."""
    import torch.distributed as dist
    offset = torch.tensor([row_lo], dtype=torch.int64, device=ids.device)
    if not (dist.is_available() and dist.is_initialized()):
        return ids.unsqueeze(0).contiguous(), scores.unsqueeze(0).contiguous(), offset
    G = dist.get_world_size(group)
    def gather(t: torch.Tensor) -> torch.Tensor:
        parts = [torch.empty_like(t) for _ in range(G)]
        dist.all_gather(parts, t.contiguous(), group=group)
        return torch.stack(parts)

    all_ids, all_scores, all_offsets = gather(ids), gather(scores), gather(offset).reshape(G)
    return all_ids, all_scores, all_offsets


class ShardedIndex:
    """This rank's shard of a row-sharded corpus. `local_rows` are rows [row_lo, row_lo + n) of
    the whole corpus, resident on this rank's GPU."""

    def __init__(self, local_rows: torch.Tensor, row_lo: int, metric: int, max_s: int = 8, max_k: int = 32,
                 group=None):
        self.index = binding.Index(local_rows, metric, max_s, max_k)
        self.row_lo = int(row_lo)
        self.metric = metric
        self.group = group

    def search(self, queries: torch.Tensor, k: int, stream: Optional[torch.cuda.Stream] = None):
        """Every rank passes the same queries; every rank gets the answer over the whole corpus."""
        ids, scores = binding.search(self.index, queries, k, stream=stream)
        all_ids, all_scores, offsets = gather_lists(ids, scores, self.row_lo, self.group)
        return binding.merge_lists(all_ids, all_scores, offsets, self.metric, stream=stream)

    def close(self):
        self.index.close()
