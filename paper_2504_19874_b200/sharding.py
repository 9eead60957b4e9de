"""Host-side plumbing for a search sharded over ranks (one process per GPU).

Database vectors are independent and the quantiser is data-oblivious, so a sharded index needs no
exchange while quantising: every rank holds the same plan (Pi, S, codebook) and the codes of its own
contiguous range of vectors.  A query is answered by every rank on its shard (tq_topk); the local
best lists, with ids made global, are all-gathered (nq * k * 8 bytes per rank) and reduced to the
global best list (tq_select_topk on a GPU).  Nothing here computes scores.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_bounds(n_total: int, rank: int, world: int) -> tuple[int, int]:
    """(first id, count) of the contiguous shard of `rank`; the remainder goes to the first ranks."""
    if not 0 <= rank < world:
        raise ValueError("rank outside the world")
    base, rem = divmod(n_total, world)
    count = base + (1 if rank < rem else 0)
    start = rank * base + min(rank, rem)
    return start, count


def gather_candidates(top_scores: torch.Tensor, top_ids: torch.Tensor, id_offset: int, group=None):
    """All-gathers the local best lists.  Returns (scores, ids), both [nq, world * k]; ids are global
    (local id + the shard's first id), empty slots (id < 0) stay negative."""
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    ids = torch.where(top_ids >= 0, top_ids + id_offset, top_ids).to(torch.int32)
    if world == 1:
        return top_scores.contiguous(), ids.contiguous()
    s_list = [torch.empty_like(top_scores) for _ in range(world)]
    i_list = [torch.empty_like(ids) for _ in range(world)]
    dist.all_gather(s_list, top_scores.contiguous(), group=group)
    dist.all_gather(i_list, ids.contiguous(), group=group)
    return torch.cat(s_list, dim=1).contiguous(), torch.cat(i_list, dim=1).contiguous()
