"""A cache whose rows are partitioned over the GPUs of one node: one process and one SisoCache per GPU.

FindClosestCentroid over the whole cache is the best of the shards' best, so a lookup is: every rank scores the full
query batch against its own rows (siso_lookup_keys), ONE all-gather moves k packed 64-bit keys per query and rank
(8192 queries x top-4 = 256 KiB per rank), and every rank combines the lists (siso_combine_keys).  The keys order by
(similarity, then lower GLOBAL slot), so the result does not depend on the number of ranks.  torch.distributed (NCCL
over NVLink on GPUs) is the plumbing; there is no other exchange on the lookup path.

Global slot g lives on rank g // rows_per_rank at local slot g % rows_per_rank.
"""
from __future__ import annotations

from typing import Optional, Tuple

import torch
import torch.distributed as dist


def shard_rows(total_rows: int, world: int) -> int:
    """Rows per rank: equal shards, the last one possibly short."""
    return (int(total_rows) + world - 1) // world


def owner_of(global_slot: int, rows_per_rank: int) -> Tuple[int, int]:
    """(rank, local slot) of a global slot."""
    return int(global_slot) // rows_per_rank, int(global_slot) % rows_per_rank


def local_range(rank: int, total_rows: int, rows_per_rank: int) -> Tuple[int, int]:
    """[lo, hi) of the global rows that `rank` holds."""
    lo = min(total_rows, rank * rows_per_rank)
    return lo, min(total_rows, lo + rows_per_rank)


def gather_keys(keys: torch.Tensor, group=None) -> torch.Tensor:
    """keys [n, k] of this rank -> [n, world, k] with list r = rank r's keys (the layout siso_combine_keys reads).
    Works on any backend (NCCL for CUDA tensors, gloo for CPU tensors); without an initialised process group the
    world is this process alone."""
    if not (dist.is_available() and dist.is_initialized()):
        return keys.unsqueeze(1).contiguous()
    world = dist.get_world_size(group)
    n, k = keys.shape
    out = torch.empty((world * n, k), dtype=keys.dtype, device=keys.device)      # rank r's rows at [r n, (r + 1) n)
    dist.all_gather_into_tensor(out, keys.contiguous(), group=group)
    return out.view(world, n, k).permute(1, 0, 2).contiguous()


class ShardedCache:
    """This rank's shard of a cache of `total_rows` rows, plus the sharded lookup."""

    def __init__(self, total_rows: int, dim: int, dtype: str = "bf16", rank: Optional[int] = None,
                 world: Optional[int] = None, device: Optional[int] = None, group=None):
        from .binding import SisoCache
        inited = dist.is_available() and dist.is_initialized()
        self.rank = (dist.get_rank(group) if inited else 0) if rank is None else int(rank)
        self.world = (dist.get_world_size(group) if inited else 1) if world is None else int(world)
        self.group = group
        self.total_rows = int(total_rows)
        self.rows_per_rank = shard_rows(total_rows, self.world)
        self.lo, self.hi = local_range(self.rank, self.total_rows, self.rows_per_rank)
        dev = torch.cuda.current_device() if device is None else device
        self.local = SisoCache(max(1, self.rows_per_rank), dim, dtype, device=dev)

    def fill(self, all_rows: torch.Tensor) -> None:
        """Every rank passes the same [total_rows, dim] tensor (or at least its own rows' range) and keeps its part:
        global row g goes to local slot g - lo."""
        part = all_rows[self.lo:self.hi]
        if part.shape[0] > 0:
            slots = self.local.insert(part.to(self.local._dev))
            assert int(slots[0]) == 0, "fill expects an empty shard"

    def lookup(self, queries: torch.Tensor, theta, k: int = 1, stream=None):
        """The same batch on every rank -> (idx [n, k] int64 GLOBAL slots, sim [n, k], hit [n]), identical on all ranks."""
        from .binding import combine_keys
        keys = self.local.lookup_keys(queries, k, slot_offset=self.lo, stream=stream)
        return combine_keys(gather_keys(keys, self.group), theta, stream=stream)

    def close(self) -> None:
        self.local.close()
