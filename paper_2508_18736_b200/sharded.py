"""A cache whose rows are partitioned over the GPUs of one node: one process and one SisoCache per GPU.

FindClosestCentroid over the whole cache is the best of the shards' best, so a lookup is: every rank scores the full
query batch against its own rows (siso_lookup_keys), ONE all-gather moves k packed 64-bit keys per query and rank
(8192 queries x top-4 = 256 KiB per rank), and every rank combines the lists (siso_combine_keys).  The keys order by
(similarity, then lower GLOBAL slot), so the result does not depend on the number of ranks.  torch.distributed (NCCL
over NVLink on GPUs) is the plumbing; there is no other exchange on the lookup path.

Maintenance keeps the whole equal to ONE cache over the global slots: a hit updates the row on its owner (every rank
calls the update once per batch, so the clocks agree), FilteringCentroids becomes "every rank reports its m lowest keys,
the m lowest of all reported keys go" (one all-gather of 24 bytes per key), and the misses of a batch, in ascending row
order, take the free slots of the whole cache in ascending global order (one all-gather of the free counts, one
all-reduce(max) of the slots).  Each of these operations is written once, as a generator that yields its exchanges
(`("gather", tensor)` -> [world, ...], `("max", tensor)` -> elementwise maximum over ranks) and is driven either by
torch.distributed (`run`) or, on one GPU, by `run_lockstep` over several shards of the same process.

Global slot g lives on rank g // rows_per_rank at local slot g % rows_per_rank.
"""
from __future__ import annotations

from typing import Generator, List, Optional, Sequence, Tuple

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


def exchange(kind: str, t: torch.Tensor, group=None) -> torch.Tensor:
    """One exchange of a sharded operation over torch.distributed: "gather" -> [world, *t.shape], "max" -> t's shape."""
    inited = dist.is_available() and dist.is_initialized()
    if kind == "gather":
        if not inited:
            return t.unsqueeze(0).contiguous()
        world = dist.get_world_size(group)
        flat = t.contiguous().reshape(1, -1)
        out = torch.empty((world, flat.shape[1]), dtype=t.dtype, device=t.device)
        dist.all_gather_into_tensor(out, flat, group=group)
        return out.view((world,) + tuple(t.shape))
    if kind == "max":
        out = t.clone()
        if inited:
            dist.all_reduce(out, op=dist.ReduceOp.MAX, group=group)
        return out
    raise ValueError(kind)


def run(steps: Generator, group=None):
    """Drives one sharded operation of THIS rank, doing its exchanges with torch.distributed."""
    try:
        req = next(steps)
        while True:
            req = steps.send(exchange(req[0], req[1], group))
    except StopIteration as done:
        return done.value


def run_lockstep(all_steps: Sequence[Generator]) -> List:
    """Drives the same sharded operation of several shards held by ONE process (all on one device): the shards advance
    from exchange to exchange together, and an exchange is a stack or an elementwise maximum of what they yielded."""
    results, reqs = [None] * len(all_steps), {}

    def advance(r, value, first):
        try:
            reqs[r] = next(all_steps[r]) if first else all_steps[r].send(value)
        except StopIteration as done:
            reqs.pop(r, None)
            results[r] = done.value

    for r in range(len(all_steps)):
        advance(r, None, True)
    while reqs:
        assert len(reqs) == len(all_steps), "shards finished at different exchanges"
        kinds = {q[0] for q in reqs.values()}
        assert len(kinds) == 1, "shards disagree on the next exchange"
        stacked = torch.stack([reqs[r][1] for r in range(len(all_steps))])
        answer = stacked if kinds == {"gather"} else stacked.max(dim=0).values
        for r in range(len(all_steps)):
            advance(r, answer.clone(), False)
    return results


class ShardedCache:
    """This rank's shard of a cache of `total_rows` rows: the sharded lookup and the owner-routed maintenance."""

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
        self.local = SisoCache(max(1, self.hi - self.lo), dim, dtype, device=dev)     # a rank beyond the rows holds one unused slot

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

    # ---- maintenance: generators that yield their exchanges; drive them with run() or run_lockstep() ----
    def _free(self) -> int:
        return (self.hi - self.lo) - int(self.local.stats()["occupancy"])

    def evict_steps(self, n_evict: int, flags: int = 0):
        """FilteringCentroids over the whole cache: -> victims [n_evict] int64 global slots in eviction order (-1 padding),
        the same on every rank."""
        from .binding import select_evict
        n_evict = int(n_evict)
        if n_evict <= 0:
            if flags:
                self.local.evict_slots(torch.empty((0,), dtype=torch.int64, device=self.local._dev), self.lo, flags)
            return torch.empty((0,), dtype=torch.int64, device=self.local._dev)
        keys = self.local.evict_keys(n_evict, slot_offset=self.lo)
        if self.hi == self.lo:
            keys.fill_(-1)                                    # a rank without rows reports nothing
        all_keys = yield ("gather", keys)                     # [world, n_evict, 3]
        victims = select_evict(all_keys, n_evict)
        if self.hi > self.lo:
            self.local.evict_slots(victims, self.lo, flags)
        return victims

    def stream_steps(self, queries: torch.Tensor, theta):
        """One micro-batch of the streaming step over the whole cache (lookup, running-mean update of the hits, room for
        the misses, insertion): -> (idx [n] int64 global slot, sim [n], hit [n], victims int64 [#evicted], slots [n] int64
        global slot of each stored miss or -1), the same on every rank and equal to one unsharded cache's step."""
        from .binding import combine_keys, route
        q = self.local._vec(queries, "queries")
        n = q.shape[0]
        dev = q.device
        keys = self.local.lookup_keys(q, 1, slot_offset=self.lo)
        if self.hi == self.lo:
            keys.zero_()
        all_keys = yield ("gather", keys)                     # [world, n, 1]
        idx, sim, hit = combine_keys(all_keys.permute(1, 0, 2).contiguous(), theta)
        idx, sim = idx[:, 0].contiguous(), sim[:, 0].contiguous()
        # hits: the owner updates; every rank calls the update so that every clock advances
        idx_local, upd_hit, _ = route(idx, hit, self.lo, self.hi, 0, 0)
        self.local.update(q, idx_local, upd_hit)
        # room: the misses need free slots somewhere in the cache
        n_miss = n - int(hit.sum().item())
        free = yield ("gather", torch.tensor([self._free()], dtype=torch.int64, device=dev))       # [world, 1]
        lack = n_miss - int(free.sum().item())
        victims = torch.empty((0,), dtype=torch.int64, device=dev)
        if lack > 0:
            victims = yield from self.evict_steps(lack)
            free = yield ("gather", torch.tensor([self._free()], dtype=torch.int64, device=dev))
        # insertion: misses in row order take the free slots in global order
        skip = int(free[:self.rank].sum().item())
        take = int(free[self.rank].item())
        _, _, ins_hit = route(idx, hit, self.lo, self.hi, skip, take)
        slots = self.local.insert_misses(q, ins_hit).to(torch.int64)
        slots = torch.where(slots >= 0, slots + self.lo, slots)
        if self.hi == self.lo:
            slots.fill_(-1)
        slots = yield ("max", slots)
        return idx, sim, hit, victims, slots

    def evict(self, n_evict: int, flags: int = 0) -> torch.Tensor:
        return run(self.evict_steps(n_evict, flags), self.group)

    def stream_step(self, queries: torch.Tensor, theta):
        return run(self.stream_steps(queries, theta), self.group)

    def close(self) -> None:
        self.local.close()
