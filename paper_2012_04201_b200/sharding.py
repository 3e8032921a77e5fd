"""Splitting one ``params_list`` over several ranks (one process per GPU).

Every (configuration, fold) fit is independent and its random streams are keyed by the
configuration's position in the full list, so a rank that evaluates a contiguous slice with
``config_index_base`` = the slice's first position gets exactly the scores of the unsplit
call.  No data-path collective is involved; the scores are gathered at the end.  (The paper
runs independent jobs per GPU in round-robin order, sec. 5.)
"""
from __future__ import annotations

import numpy as np


def shard_bounds(n_configs: int, rank: int, world: int):
    """Contiguous slice [begin, end) of the list for ``rank``; the first ranks get one more."""
    if not (0 <= rank < world) or n_configs < 0:
        raise ValueError("bad rank/world/n_configs")
    base, rem = divmod(n_configs, world)
    begin = rank * base + min(rank, rem)
    return begin, begin + base + (1 if rank < rem else 0)


def gather_scores(local_scores, n_configs: int, rank: int, world: int, dist=None):
    """All ranks' slices of scores, concatenated in list order.  ``dist``: torch.distributed
    (initialised), or None when world == 1.  Works with CPU (gloo) or CUDA (nccl) tensors."""
    import torch

    local = torch.as_tensor(local_scores, dtype=torch.float32)
    if world == 1:
        return local.clone()
    sizes = [shard_bounds(n_configs, r, world) for r in range(world)]
    longest = max(e - b for b, e in sizes)
    padded = torch.zeros(longest, dtype=torch.float32, device=local.device)
    padded[: local.numel()] = local
    parts = [torch.zeros_like(padded) for _ in range(world)]
    dist.all_gather(parts, padded)
    return torch.cat([parts[r][: e - b] for r, (b, e) in enumerate(sizes)])
