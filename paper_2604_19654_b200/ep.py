"""Host side of expert parallelism over R real ranks (paper Section 2.2, Phases 1 and 2; Section 2.3:
every device derives the same plan by itself).  One process per rank over ``torch.distributed``.

What is here is the control plane only: the all-gather of the per-expert counts and, from it, each
rank's plan, its send / receive row counts for the dispatch all-to-all-v, for the rows of migrated
pieces and for the combine, and the list of peer weight copies into receive slots
(``feplb_ep_schedule``, C++).  The data plane -- the row exchange over NCCL or peer stores and the
copy-engine transfers of weights -- is not part of this library yet.
"""
from __future__ import annotations

import numpy as np

from . import feplb as F


def exchange_counts(local_counts, group=None) -> np.ndarray:
    """All-gathers every rank's per-expert counts (int32 [E]) -> int32 [R, E], identical on all ranks.

    This is the one collective the balancer needs: E int32 values per rank."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    mine = torch.from_numpy(np.ascontiguousarray(local_counts, np.int32))
    parts = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(parts, mine, group=group)
    return np.stack([p.numpy() for p in parts]).astype(np.int32)


def schedule(cfg: F.Config, counts_by_src: np.ndarray, rank: int, dyn_mask=None) -> dict:
    """This rank's share of the micro-batch's exchanges (see ``feplb.ep_schedule``).  With
    ``dyn_mask`` None the dynamic experts are the ``cfg.dyn`` busiest of every rank's block by the
    global counts, the same rule the single-GPU path applies."""
    counts = np.asarray(counts_by_src, np.int64).sum(0)
    if dyn_mask is None:
        dyn_mask = F.select_dynamic(counts, cfg.E, cfg.R, cfg.dyn)
    return F.ep_schedule(cfg, counts_by_src, dyn_mask, rank)
