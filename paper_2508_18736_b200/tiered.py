"""Locality-ordered exact search over a cache held as two tiers (the exact-search counterpart of the paper's Sec. 4.3
placement of strongly local centroids where a search reaches them first).

The HOT tier holds the entries FilteringCentroids would evict last (largest cluster_size, then access count, then
recency); the COLD tier holds the rest.  A lookup scores the whole batch against the hot tier, lets every query whose
best hot similarity exceeds the exit similarity stop there (no cold entry can beat it, see siso_tier_exit_sim), packs
the remaining queries into a dense batch and scores only those against the cold tier.  The answer is the top-1 over the
whole cache, with the slots of the cache the tiers were built from.

The tiers are a snapshot: build them after maintenance and rebuild after the next one.  Both the split and the lookup's
control flow are entry points of the library (siso_tier_build, siso_tier_lookup); this class only marshals.
"""
from __future__ import annotations

import ctypes
import math
from typing import Optional

import torch

from .binding import SisoCache, SisoError, _ptr, _stream, tier_exit_sim


class TieredCache:
    def __init__(self, cache: SisoCache, hot_rows: int, sep_sim: float, norm_slack: float = 0.0, certify: bool = True):
        """cache: the cache to split (left untouched).  hot_rows: size of the hot tier.  sep_sim: an upper bound on the
        similarity of any hot entry to any cold entry; norm_slack: how far the norms of entries and queries may be from 1
        (bf16 rounding of unit vectors: about 1e-3).  The exit rule is only exact if the bound holds, and nothing in the
        cache's history guarantees it for good (a weighted merge recentres survivors, a two-set merge never compares
        the old entries with each other, later inserts and updates move vectors), so by default the build CHECKS it:
        every hot/cold pair is swept (tensor cores + exact fp64 check) and a pair above sep_sim raises ValueError, and so
        does an entry whose norm is further from 1 than norm_slack (the queries' norms stay the caller's promise).
        certify=False skips the check for a caller that has just established the bound some other way."""
        if certify:
            dev = cache.norm_deviation()
            if not dev <= norm_slack:
                raise ValueError(f"entries deviate from unit norm by up to {dev:.3g}, more than norm_slack = {norm_slack}: "
                                 "the early exit would not be exact")
        occ = int(cache.stats()["occupancy"])
        hot_rows = max(0, min(int(hot_rows), occ))
        dev = cache._dev.index
        self.hot = SisoCache(max(1, hot_rows), cache.dim, cache.dtype, device=dev)
        self.cold = SisoCache(max(1, occ - hot_rows), cache.dim, cache.dtype, device=dev)
        self.hot_slot = torch.full((self.hot.capacity,), -1, dtype=torch.int32, device=cache._dev)
        self.cold_slot = torch.full((self.cold.capacity,), -1, dtype=torch.int32, device=cache._dev)
        counts = (ctypes.c_int64 * 3)()
        st = cache._lib.siso_tier_build(cache._h, hot_rows, float(sep_sim) if certify else math.nan, self.hot._h, self.cold._h,
                                        _ptr(self.hot_slot), _ptr(self.cold_slot), counts, _stream(None))
        if st != 0:
            raise SisoError(st, "siso_tier_build")
        self.n_hot, self.n_cold, self.pairs_above_sep = int(counts[0]), int(counts[1]), int(counts[2])
        if self.pairs_above_sep > 0:
            self.close()
            raise ValueError(f"{self.pairs_above_sep} hot/cold pairs are more similar than sep_sim = {sep_sim}: "
                             "the early exit would not be exact")
        self.exit_sim = tier_exit_sim(sep_sim, norm_slack)
        self.settled = 0            # queries of the last lookup that ended in the hot tier
        self._work = None

    def lookup(self, queries: torch.Tensor, theta, stream=None):
        """-> (idx [n] int32 slots of the original cache, sim [n], hit [n]); equal to cache.lookup(queries, theta, 1)."""
        q = self.hot._vec(queries, "queries")
        n = q.shape[0]
        lib, dev = self.hot._lib, q.device
        need = int(lib.siso_tier_work_bytes(n, self.hot.dim, 0 if self.hot.dtype == "f32" else 1))
        if self._work is None or self._work.numel() < need:
            self._work = torch.empty(need, dtype=torch.uint8, device=dev)
        th_t, th_s = (theta.to(device=dev, dtype=torch.float32).contiguous(), 0.0) if isinstance(theta, torch.Tensor) else (None, float(theta))
        idx = torch.empty((n,), dtype=torch.int32, device=dev)
        sim = torch.empty((n,), dtype=torch.float32, device=dev)
        hit = torch.empty((n,), dtype=torch.uint8, device=dev)
        settled = ctypes.c_int64(0)
        st = lib.siso_tier_lookup(self.hot._h, self.cold._h, _ptr(self.hot_slot), _ptr(self.cold_slot), _ptr(q), n, float(self.exit_sim),
                                  _ptr(th_t), th_s, _ptr(self._work), _ptr(idx), _ptr(sim), _ptr(hit), ctypes.byref(settled),
                                  _stream(stream))
        if st != 0:
            raise SisoError(st, "siso_tier_lookup")
        self.settled = int(settled.value)
        return idx, sim, hit

    def close(self) -> None:
        self.hot.close()
        self.cold.close()
