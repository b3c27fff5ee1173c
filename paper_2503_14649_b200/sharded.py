"""Database-sharded search: one process per GPU, each holding the index of its own shard.

The paper's retrieval model (Sec. 4) splits a large database over servers that index their shards
independently; a query goes to every shard and the shards' results are aggregated.  Here a rank
searches its shard with `rago_search`, the ranks exchange their [nq, k] answers with one all-gather
(12 bytes per result) and every rank aggregates them with `rago_merge_results`.  The query batch
must be the same on every rank; ids should be unique across shards.

torch.distributed is the plumbing (NCCL between GPUs); the search and the aggregation run in the
library's kernels.
"""

from typing import Optional, Tuple

import torch
import torch.distributed as dist

from . import binding


def gather_parts(ids: torch.Tensor, dists: torch.Tensor, group=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """All-gather the ranks' [nq, k] answers into [world, nq, k] tensors, rank r's answer at index r."""
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    if world == 1:
        return ids.unsqueeze(0).contiguous(), dists.unsqueeze(0).contiguous()
    nq, k = ids.shape
    # the ranks' blocks end to end along the first dimension, then viewed as [world, nq, k]
    all_ids = torch.empty((world * nq, k), dtype=ids.dtype, device=ids.device)
    all_dists = torch.empty((world * nq, k), dtype=dists.dtype, device=dists.device)
    dist.all_gather_into_tensor(all_ids, ids.contiguous(), group=group)
    dist.all_gather_into_tensor(all_dists, dists.contiguous(), group=group)
    return all_ids.view(world, nq, k), all_dists.view(world, nq, k)


def rago_search_sharded(index: "binding.Index", queries: torch.Tensor, nprobe: int, k: int, group=None,
                        workspace: Optional[torch.Tensor] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Search this rank's shard, exchange, aggregate: every rank returns the global [nq, k] answer."""
    ids, dists = index.rago_search(queries, nprobe, k, workspace=workspace)
    all_ids, all_dists = gather_parts(ids, dists, group)
    return binding.rago_merge_results(all_ids, all_dists, k, index.metric)
