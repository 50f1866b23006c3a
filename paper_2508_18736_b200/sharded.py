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
(`("gather", tensor)` -> [world, ...], `("max", tensor)` -> elementwise maximum over ranks, `("ring", tensor, shift)` ->
the tensor of the rank `shift` places back, copied into this rank's memory) and is driven either by torch.distributed
(`run`) or, on one GPU, by `run_lockstep` over several shards of the same process.  MergeCentroids over the partitioned
cache (`merge_steps`) cuts its pairwise sweep into block products along such a ring.

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


def exchange(kind: str, t: torch.Tensor, group=None, shift: int = 0) -> torch.Tensor:
    """One exchange of a sharded operation over torch.distributed: "gather" -> [world, *t.shape], "max" -> t's shape,
    "ring" -> the tensor that rank (own rank - shift) mod world passed, received into this rank's own memory (every
    rank passes the same shape)."""
    inited = dist.is_available() and dist.is_initialized()
    if kind == "ring":
        world = dist.get_world_size(group) if inited else 1
        shift %= world
        if shift == 0:
            return t.clone()
        rank = dist.get_rank(group)
        src, dst = (rank - shift) % world, (rank + shift) % world
        if group is not None:
            src, dst = dist.get_global_rank(group, src), dist.get_global_rank(group, dst)
        t = t.contiguous()
        out = torch.empty_like(t)
        for req in dist.batch_isend_irecv([dist.P2POp(dist.isend, t, dst, group), dist.P2POp(dist.irecv, out, src, group)]):
            req.wait()
        return out
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
            req = steps.send(exchange(req[0], req[1], group, *req[2:]))
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
        if kinds == {"ring"}:
            shifts = {q[2] for q in reqs.values()}
            assert len(shifts) == 1, "shards disagree on the ring step"
            shift = shifts.pop() % len(all_steps)
            answers = [stacked[(r - shift) % len(all_steps)].clone() for r in range(len(all_steps))]
        else:
            answer = stacked if kinds == {"gather"} else stacked.max(dim=0).values
            answers = [answer.clone() for _ in range(len(all_steps))]
        for r in range(len(all_steps)):
            advance(r, answers[r], False)
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

    def _free_dev(self) -> torch.Tensor:
        """[1] int64 on the device: this shard's free slots (0 for a rank without rows)."""
        if self.hi == self.lo:
            return torch.zeros((1,), dtype=torch.int64, device=self.local._dev)
        return self.local.free_slots()

    def stream_steps(self, queries: torch.Tensor, theta):
        """One micro-batch of the streaming step over the whole cache (lookup, running-mean update of the hits, room for
        the misses, insertion): -> (idx [n] int64 global slot, sim [n], hit [n], victims int64 [n]: the evicted global
        slots in eviction order, then -1, slots [n] int64 global slot of each stored miss or -1), the same on every rank
        and equal to one unsharded cache's step.  Every count the step depends on (misses, free slots, entries to evict)
        stays on the device, so the host issues the same launches and exchanges for every batch and never waits."""
        from .binding import combine_keys, route, select_evict_planned, shard_plan
        q = self.local._vec(queries, "queries")
        n = q.shape[0]
        if n > self.total_rows:          # its misses could outnumber the slots of the whole cache (SISO_ERR_CAPACITY on one cache)
            raise ValueError(f"a micro-batch of {n} rows does not fit a cache of {self.total_rows} entries")
        empty = self.hi == self.lo
        keys = self.local.lookup_keys(q, 1, slot_offset=self.lo)
        if empty:
            keys.zero_()
        all_keys = yield ("gather", keys)                     # [world, n, 1]
        idx, sim, hit = combine_keys(all_keys.permute(1, 0, 2).contiguous(), theta)
        idx, sim = idx[:, 0].contiguous(), sim[:, 0].contiguous()
        # hits: the owner updates; every rank calls the update so that every clock advances
        idx_local, upd_hit, _ = route(idx, hit, self.lo, self.hi, 0, 0)
        self.local.update(q, idx_local, upd_hit)
        # room: the misses that find no free slot anywhere in the cache evict (plan[1] of them, possibly none)
        free = yield ("gather", self._free_dev())             # [world, 1]
        plan = shard_plan(hit, free, self.rank)
        ekeys = self.local.evict_keys(n, slot_offset=self.lo)
        if empty:
            ekeys.fill_(-1)                                   # a rank without rows reports nothing
        all_ekeys = yield ("gather", ekeys)                   # [world, n, 3]
        victims = select_evict_planned(all_ekeys, plan)
        if not empty:
            self.local.evict_slots(victims, self.lo, 0)
        # insertion: misses in row order take the free slots in global order
        free = yield ("gather", self._free_dev())
        plan = shard_plan(hit, free, self.rank)
        _, _, ins_hit = route(idx, hit, self.lo, self.hi, plan=plan)
        slots = self.local.insert_misses(q, ins_hit).to(torch.int64)
        slots = torch.where(slots >= 0, slots + self.lo, slots)
        if empty:
            slots.fill_(-1)
        slots = yield ("max", slots)
        return idx, sim, hit, victims, slots

    def merge_steps(self, theta_c: float, flags: int, cand_capacity: Optional[int] = None):
        """MergeCentroids over the whole cache (one pass, like siso_merge with no repository): -> (merge_map int32
        [total_rows] over the global slots, number of entries merged away), the same on every rank and equal to one
        unsharded cache's pass.  The pairwise sweep is cut into block products: every rank sweeps its own block, and
        every unordered pair of blocks is swept once, on one of its owners, after the other block has travelled round
        the ring into that rank's own memory (about world / 2 ring steps).  Candidates, live flags and the merged rows
        are then gathered; the resolution runs identically on every rank."""
        from .binding import MERGE_WEIGHTED_MEAN
        G, r, rpr = self.world, self.rank, self.rows_per_rank
        dev, D = self.local._dev, self.local.dim
        n_own = self.hi - self.lo
        st = self.local.export()
        block = torch.zeros((rpr, D), dtype=torch.float32, device=dev)
        valid = torch.zeros((rpr,), dtype=torch.uint8, device=dev)
        if n_own:
            block[:n_own] = st["master"][:n_own]
            valid[:n_own] = st["valid"][:n_own]
        del st
        cap = int(cand_capacity) if cand_capacity else 32 * rpr + 65536
        cand = torch.full((cap, 3), -1, dtype=torch.int32, device=dev)
        n_cand = torch.zeros((1,), dtype=torch.int64, device=dev)
        if n_own:
            self.local.pair_sweep_block(self.lo, theta_c, cand, n_cand)
        for t in range(1, G // 2 + 1):
            peer_block = yield ("ring", block, t)
            peer_valid = yield ("ring", valid, t)
            s = (r - t) % G
            s_lo, s_hi = local_range(s, self.total_rows, rpr)
            mine = (2 * t < G) or (2 * t == G and r < s)          # each unordered pair of blocks on exactly one owner
            if mine and n_own and s_hi > s_lo:
                self.local.pair_sweep_block(self.lo, theta_c, cand, n_cand, peer_block[:s_hi - s_lo], peer_valid[:s_hi - s_lo], s_lo)
        self.local.check_status()
        counts = yield ("gather", n_cand)                        # [world, 1]
        pad = max(1, int(counts.max().item()))
        all_cand = yield ("gather", cand[:pad].contiguous())     # [world, pad, 3]; places beyond a rank's count hold i = -1
        all_valid = yield ("gather", valid)                      # [world, rows_per_rank] = live flags by global slot
        mm, n_merged = self.local.merge_resolve(all_cand.reshape(-1, 3), all_valid.reshape(-1))
        weighted = bool(flags & MERGE_WEIGHTED_MEAN)
        own_map = mm[self.lo:self.lo + max(n_own, 1)]
        n_gone = 0
        if n_own:
            slots = torch.arange(self.lo, self.hi, dtype=torch.int32, device=dev)
            n_gone = int(((own_map[:n_own] >= 0) & (own_map[:n_own] != slots) & (valid[:n_own] != 0)).sum().item())
        gone = yield ("gather", torch.tensor([n_gone], dtype=torch.int64, device=dev))
        P = max(1, int(gone.max().item()))
        meta, sizes, rows, _ = self.local.merge_pack(mm, self.lo, P, weighted)
        if not n_own:
            meta.fill_(-1)
        all_meta = yield ("gather", meta)                        # [world, P, 2]: rank order = ascending global slot
        all_sizes = yield ("gather", sizes)
        all_rows = (yield ("gather", rows)) if weighted else None
        self.local.merge_apply_shard(mm, self.lo, all_meta.reshape(-1, 2), all_sizes.reshape(-1),
                                     None if all_rows is None else all_rows.reshape(-1, D), flags)
        self.local.check_status()
        return mm[:self.total_rows], int(n_merged.item())

    def merge(self, theta_c: float, flags: int):
        return run(self.merge_steps(theta_c, flags), self.group)

    def evict(self, n_evict: int, flags: int = 0) -> torch.Tensor:
        return run(self.evict_steps(n_evict, flags), self.group)

    def stream_step(self, queries: torch.Tensor, theta):
        return run(self.stream_steps(queries, theta), self.group)

    def close(self) -> None:
        self.local.close()
