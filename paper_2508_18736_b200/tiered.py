"""Locality-ordered exact search over a cache held as two tiers (the exact-search counterpart of the paper's Sec. 4.3
placement of strongly local centroids where a search reaches them first).

The HOT tier holds the entries FilteringCentroids would evict last (largest cluster_size, then access count, then
recency); the COLD tier holds the rest.  A lookup scores the whole batch against the hot tier, lets every query whose
best hot similarity exceeds the exit similarity stop there (no cold entry can beat it, see siso_tier_exit_sim), packs
the remaining queries into a dense batch and scores only those against the cold tier.  The answer is the top-1 over the
whole cache, with the slots of the cache the tiers were built from.

The tiers are a snapshot: build them after maintenance (MergeCentroids at theta_C makes every pair of entries at most
theta_C similar, which is the separation bound the exit needs) and rebuild after the next one.
"""
from __future__ import annotations

from typing import Optional

import torch

from .binding import SisoCache, tier_exit_sim, tier_finish, tier_select


class TieredCache:
    def __init__(self, cache: SisoCache, hot_rows: int, sep_sim: float, norm_slack: float = 0.0):
        """cache: the cache to split (left untouched).  hot_rows: size of the hot tier.  sep_sim: an upper bound on the
        similarity of any hot entry to any cold entry (e.g. theta_C right after a merge).  norm_slack: how far the norms
        of entries and queries may be from 1 (bf16 rounding of unit vectors: about 1e-3)."""
        occ = int(cache.stats()["occupancy"])
        hot_rows = max(0, min(int(hot_rows), occ))
        dev = cache._dev
        # the cold tier = what FilteringCentroids would evict to leave hot_rows entries: run it on a copy
        tmp = SisoCache(cache.capacity, cache.dim, cache.dtype, device=dev.index)
        tmp.copy_from(cache)
        victims = tmp.evict(occ - hot_rows) if occ > hot_rows else torch.empty((0,), dtype=torch.int32, device=dev)
        st = cache.export()
        torch.cuda.synchronize(dev)
        tmp.close()
        cold_slots = torch.sort(victims.to(torch.int64)).values
        keep = st["valid"].to(torch.bool).clone()
        keep[cold_slots] = False
        hot_slots = torch.nonzero(keep).reshape(-1)
        clock = int(cache.stats()["clock"])
        self.hot, self.hot_slot = self._tier(cache, st, hot_slots, clock)
        self.cold, self.cold_slot = self._tier(cache, st, cold_slots, clock)
        self.n_hot, self.n_cold = int(hot_slots.numel()), int(cold_slots.numel())
        self.exit_sim = tier_exit_sim(sep_sim, norm_slack)
        self.settled = 0            # queries of the last lookup that ended in the hot tier

    @staticmethod
    def _tier(cache: SisoCache, st: dict, slots: torch.Tensor, clock: int):
        n = int(slots.numel())
        t = SisoCache(max(1, n), cache.dim, cache.dtype, device=cache._dev.index)
        if n:
            t.import_(st["master"][slots], st["size"][slots], st["access"][slots], st["last"][slots],
                      torch.ones(n, dtype=torch.uint8, device=slots.device), clock)
        return t, slots.to(torch.int32).contiguous()

    def lookup(self, queries: torch.Tensor, theta, stream=None):
        """-> (idx [n] int32 slots of the original cache, sim [n], hit [n]); equal to cache.lookup(queries, theta, 1)."""
        q = self.hot._vec(queries, "queries")
        hk = self.hot.lookup_keys(q, 1, stream=stream)
        rows, packed, count = tier_select(hk, q, self.exit_sim, stream=stream)
        n_go = int(count.item())                             # one 8-byte read: sizes the cold lookup
        self.settled = q.shape[0] - n_go
        ck = self.cold.lookup_keys(packed[:n_go], 1, stream=stream) if n_go else None
        return tier_finish(hk, self.exit_sim, ck, rows, n_go, self.hot_slot, self.cold_slot, theta, stream=stream)

    def close(self) -> None:
        self.hot.close()
        self.cold.close()
