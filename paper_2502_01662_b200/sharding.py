"""Row sharding of a verification batch over ranks (one process per GPU).

Rows are independent in the verification step, so a batch shards by contiguous row blocks with no
collective on the data path.  The only thing a shard must know about the whole batch is the global
index of its first row (`row_base`), which enters the random-number counter; results are then
identical for any number of ranks.  Gathering the small per-row outputs is a plain all_gather.
"""
from __future__ import annotations

from typing import Dict, Tuple

import torch


def shard_rows(batch: int, world: int, rank: int) -> Tuple[int, int]:
    """(first_row, row_count) of `rank`: contiguous blocks, the first `batch % world` ranks one row longer."""
    if world < 1 or not (0 <= rank < world) or batch < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(batch, world)
    count = base + (1 if rank < extra else 0)
    first = rank * base + min(rank, extra)
    return first, count


def gather_rows(local: Dict[str, torch.Tensor], batch: int, group=None) -> Dict[str, torch.Tensor]:
    """all_gather of per-row outputs (first dimension = this rank's rows) into full-batch tensors.

    Works on any backend (NCCL over NVLink on GPUs, gloo on CPU).  Uneven shards are padded to the
    longest shard for the collective and trimmed afterwards."""
    import torch.distributed as dist
    world = dist.get_world_size(group)
    longest = (batch + world - 1) // world
    out = {}
    for name, t in local.items():
        pad = torch.zeros((longest,) + tuple(t.shape[1:]), dtype=t.dtype, device=t.device)
        pad[: t.shape[0]] = t
        parts = [torch.empty_like(pad) for _ in range(world)]
        dist.all_gather(parts, pad, group=group)
        rows = [parts[r][: shard_rows(batch, world, r)[1]] for r in range(world)]
        out[name] = torch.cat(rows, dim=0)
    return out
