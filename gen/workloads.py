"""Seeded synthetic workloads shaped like a semantic cache's traffic.

This module only *draws inputs*: unit-norm embedding vectors grouped around
cluster means, popularity-skewed query streams, per-query thresholds.  It holds
none of the cache's arithmetic (no similarity search, no centroid update, no
merge, no eviction).  Both the CPU oracle's tests and the CUDA tests take their
inputs from here, so that both sides see the same bits.

Recipe (all draws in fp32 from ``numpy.random.default_rng`` keyed by
``[seed, tag, chunk]`` so that the result does not depend on how many threads
generate it):

* cluster means   mu_k = normalise(g),           g ~ N(0, I_D)
* a cluster member x  = normalise(mu_k + s * g / sqrt(D)),  g ~ N(0, I_D)
  so the perturbation has length about ``s`` and cos(x, mu_k) ~ 1/sqrt(1+s^2)
* out-of-distribution queries: uniform on the sphere (normalised Gaussians)
* Zipf(s) popularity: p_r ~ r^-s assigned to a seeded random permutation of
  the clusters
* per-query thresholds: uniform fp32 in a stated interval

Three readings of a stated "sigma":
  T  s = sigma                (sigma is the length of the whole perturbation)
  L  s = sigma * sqrt(D)      (sigma per coordinate)
  P  s_k ~ U[0.05, 0.60] per cluster (pair cosines straddle usual thresholds)
"""
from __future__ import annotations

import dataclasses
from concurrent.futures import ThreadPoolExecutor
from typing import Dict, Iterator, Optional, Tuple

import numpy as np

ROWS_PER_CHUNK = 8192

# tags that separate the random streams of one seed
_TAG_MEANS, _TAG_CENT, _TAG_QUERY, _TAG_LABEL, _TAG_POP, _TAG_THETA, _TAG_SPREAD, _TAG_OOD, _TAG_STREAM = range(9)


# ----------------------------------------------------------------------------
# number formats (input formatting only)
# ----------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bfloat16 (round-to-nearest-even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns (uint16) to fp32, exactly."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _normalise_rows(x: np.ndarray) -> np.ndarray:
    n = np.sqrt(np.einsum("ij,ij->i", x, x, dtype=np.float64)).astype(np.float32)
    x /= n[:, None]
    return x


def _rng(seed: int, tag: int, chunk: int = 0) -> np.random.Generator:
    return np.random.default_rng([int(seed), int(tag), int(chunk)])


def _chunks(n: int):
    return [(c, lo, min(n, lo + ROWS_PER_CHUNK)) for c, lo in enumerate(range(0, n, ROWS_PER_CHUNK))]


def _parallel(fn, jobs, threads: int):
    if threads <= 1 or len(jobs) <= 1:
        for j in jobs:
            fn(*j)
        return
    with ThreadPoolExecutor(max_workers=threads) as ex:
        list(ex.map(lambda j: fn(*j), jobs))


# ----------------------------------------------------------------------------
# building blocks
# ----------------------------------------------------------------------------
def unit_gaussian_rows(n: int, dim: int, seed: int, tag: int, threads: int = 1) -> np.ndarray:
    """n points uniform on the unit sphere of R^dim (fp32)."""
    out = np.empty((n, dim), dtype=np.float32)

    def job(c, lo, hi):
        g = _rng(seed, tag, c).standard_normal((hi - lo, dim), dtype=np.float32)
        out[lo:hi] = _normalise_rows(g)

    _parallel(job, _chunks(n), threads)
    return out


def cluster_members(means: np.ndarray, labels: np.ndarray, spread: np.ndarray, seed: int, tag: int,
                    threads: int = 1) -> np.ndarray:
    """One member per label: normalise(mu + s*g/sqrt(D)); ``spread`` holds s per cluster."""
    n, dim = labels.shape[0], means.shape[1]
    out = np.empty((n, dim), dtype=np.float32)
    inv = np.float32(1.0 / np.sqrt(dim))

    def job(c, lo, hi):
        g = _rng(seed, tag, c).standard_normal((hi - lo, dim), dtype=np.float32)
        lab = labels[lo:hi]
        g *= (spread[lab] * inv)[:, None]
        g += means[lab]
        out[lo:hi] = _normalise_rows(g)

    _parallel(job, _chunks(n), threads)
    return out


def zipf_probs(n_clusters: int, s: float, seed: int, tag: int = _TAG_POP, epoch: int = 0) -> np.ndarray:
    """p_r ~ r^-s, ranks assigned to a seeded random permutation of clusters (fp64, sums to 1)."""
    w = np.arange(1, n_clusters + 1, dtype=np.float64) ** (-float(s))
    w /= w.sum()
    perm = _rng(seed, tag, epoch).permutation(n_clusters)
    p = np.empty(n_clusters, dtype=np.float64)
    p[perm] = w
    return p


def spread_for_mode(mode: str, sigma: float, n_clusters: int, dim: int, seed: int) -> np.ndarray:
    mode = mode.upper()
    if mode == "T":
        return np.full(n_clusters, sigma, dtype=np.float32)
    if mode == "L":
        return np.full(n_clusters, sigma * np.sqrt(dim), dtype=np.float32)
    if mode == "P":
        return _rng(seed, _TAG_SPREAD).uniform(0.05, 0.60, n_clusters).astype(np.float32)
    raise ValueError("mode must be T, L or P")


def thresholds(n: int, lo: float, hi: float, seed: int) -> np.ndarray:
    return _rng(seed, _TAG_THETA).uniform(lo, hi, n).astype(np.float32)


# ----------------------------------------------------------------------------
# the five workloads
# ----------------------------------------------------------------------------
@dataclasses.dataclass
class Workload:
    name: str
    dtype: str                      # "f32" or "bf16": storage type of centroids and queries
    dim: int
    centroids: np.ndarray           # fp32 [N, D] if f32, uint16 bf16 bits [N, D] if bf16
    queries: Optional[np.ndarray]   # same convention, [B, D]
    theta: Optional[np.ndarray]     # fp32 [B]
    k: int
    centroid_labels: np.ndarray     # int32 [N] generating cluster of each centroid
    query_labels: Optional[np.ndarray]  # int32 [B], -1 = out-of-distribution
    params: Dict

    def centroids_f32(self) -> np.ndarray:
        return bf16_bits_to_f32(self.centroids) if self.dtype == "bf16" else self.centroids

    def queries_f32(self) -> np.ndarray:
        return bf16_bits_to_f32(self.queries) if self.dtype == "bf16" else self.queries


def _store(x: np.ndarray, dtype: str) -> np.ndarray:
    return f32_to_bf16_bits(x) if dtype == "bf16" else x


def clustered_lookup_workload(name: str, *, n_centroids: int, n_queries: int, dim: int, n_clusters: int,
                              sigma: float, dtype: str, seed: int = 0, mode: str = "T",
                              zipf_s: Optional[float] = None, ood_fraction: float = 0.0,
                              theta: Tuple[float, float] = (0.85, 0.85), k: int = 1,
                              threads: int = 1, query_seed: Optional[int] = None) -> Workload:
    """Centroids and queries drawn around shared cluster means (configs 1, 2, 3, 4).

    ``query_seed`` (default: ``seed``) keys the draws of the query batch only, so that several
    batches can be drawn against one centroid set."""
    qseed = seed if query_seed is None else query_seed
    means = unit_gaussian_rows(n_clusters, dim, seed, _TAG_MEANS, threads)
    spread = spread_for_mode(mode, sigma, n_clusters, dim, seed)
    c_lab = _rng(seed, _TAG_LABEL, 0).integers(0, n_clusters, n_centroids).astype(np.int32)
    cent = cluster_members(means, c_lab, spread, seed, _TAG_CENT, threads)
    q = q_lab = th = None
    if n_queries > 0:
        if zipf_s is None:
            q_lab = _rng(qseed, _TAG_LABEL, 1).integers(0, n_clusters, n_queries).astype(np.int32)
        else:
            p = zipf_probs(n_clusters, zipf_s, seed)
            q_lab = _rng(qseed, _TAG_LABEL, 1).choice(n_clusters, size=n_queries, p=p).astype(np.int32)
        q = cluster_members(means, q_lab, spread, qseed, _TAG_QUERY, threads)
        if ood_fraction > 0.0:
            is_ood = _rng(qseed, _TAG_OOD, 0).random(n_queries) < ood_fraction
            n_ood = int(is_ood.sum())
            q[is_ood] = unit_gaussian_rows(n_ood, dim, qseed, _TAG_OOD + 100, threads)
            q_lab = q_lab.copy()
            q_lab[is_ood] = -1
        if theta[0] == theta[1]:
            th = np.full(n_queries, theta[0], dtype=np.float32)
        else:
            th = thresholds(n_queries, theta[0], theta[1], qseed)
        q = _store(q, dtype)
    params = dict(n_centroids=n_centroids, n_queries=n_queries, dim=dim, n_clusters=n_clusters, sigma=sigma,
                  mode=mode, seed=seed, zipf_s=zipf_s, ood_fraction=ood_fraction, theta=theta, k=k)
    return Workload(name, dtype, dim, _store(cent, dtype), q, th, k, c_lab, q_lab, params)


# the stated sizes of the five configurations; ``scale`` arguments shrink them for parity tests
CONFIG_SIZES = {
    1: dict(n_centroids=1024, n_queries=4096, dim=384, n_clusters=64, sigma=0.05, dtype="f32",
            theta=(0.85, 0.85), k=1),
    2: dict(n_centroids=65536, n_queries=65536, dim=768, n_clusters=4096, sigma=0.08, dtype="bf16",
            zipf_s=1.1, theta=(0.80, 0.92), k=1),
    3: dict(n_centroids=32768, n_queries=0, dim=768, n_clusters=2048, sigma=0.06, dtype="f32", k=1),
    4: dict(n_centroids=1048576, n_queries=8192, dim=1024, n_clusters=65536, sigma=0.07, dtype="bf16",
            zipf_s=1.0, ood_fraction=0.20, theta=(0.78, 0.93), k=4),
}
MERGE_THRESHOLD_CONFIG3 = 0.90


def config(number: int, *, seed: int = 0, mode: str = "T", threads: int = 1, **override) -> Workload:
    """Configuration 1-4 at its stated sizes; keyword overrides give the scaled-down twins."""
    kw = dict(CONFIG_SIZES[number])
    kw.update(override)
    return clustered_lookup_workload(f"config{number}", seed=seed, mode=mode, threads=threads, **kw)


# ----------------------------------------------------------------------------
# configuration 5: a drifting, skewed query stream
# ----------------------------------------------------------------------------
@dataclasses.dataclass
class StreamSpec:
    capacity: int = 262144
    dim: int = 768
    n_queries: int = 10_000_000
    batch: int = 256
    n_clusters: int = 16384
    zipf_s: float = 1.2
    reshuffle_every: int = 1_000_000
    theta: float = 0.86
    mode: str = "P"
    sigma: float = 0.30            # used by modes T and L only
    dtype: str = "bf16"
    seed: int = 0

    @property
    def n_batches(self) -> int:
        return (self.n_queries + self.batch - 1) // self.batch


class QueryStream:
    """Micro-batches of configuration 5.  Batch t is a pure function of (spec, t)."""

    def __init__(self, spec: StreamSpec, threads: int = 1):
        self.spec = spec
        self.means = unit_gaussian_rows(spec.n_clusters, spec.dim, spec.seed, _TAG_MEANS, threads)
        self.spread = spread_for_mode(spec.mode, spec.sigma, spec.n_clusters, spec.dim, spec.seed)
        self._pop_epoch = -1
        self._cdf = None

    def _popularity(self, epoch: int) -> np.ndarray:
        if epoch != self._pop_epoch:
            p = zipf_probs(self.spec.n_clusters, self.spec.zipf_s, self.spec.seed, _TAG_POP, epoch)
            self._cdf = np.cumsum(p)
            self._cdf[-1] = 1.0
            self._pop_epoch = epoch
        return self._cdf

    def batch(self, t: int) -> Tuple[np.ndarray, np.ndarray]:
        """Returns (queries [b, D] in the stream's dtype convention, labels int32 [b])."""
        sp = self.spec
        lo = t * sp.batch
        b = min(sp.batch, sp.n_queries - lo)
        if b <= 0:
            raise IndexError("batch index past the end of the stream")
        cdf = self._popularity(lo // sp.reshuffle_every)
        r = _rng(sp.seed, _TAG_STREAM, t)
        lab = np.searchsorted(cdf, r.random(b), side="right").astype(np.int32)
        np.minimum(lab, sp.n_clusters - 1, out=lab)
        g = r.standard_normal((b, sp.dim), dtype=np.float32)
        g *= (self.spread[lab] * np.float32(1.0 / np.sqrt(sp.dim)))[:, None]
        g += self.means[lab]
        q = _normalise_rows(g)
        return _store(q, sp.dtype), lab

    def batches(self, start: int = 0, stop: Optional[int] = None) -> Iterator[Tuple[int, np.ndarray, np.ndarray]]:
        stop = self.spec.n_batches if stop is None else min(stop, self.spec.n_batches)
        for t in range(start, stop):
            q, lab = self.batch(t)
            yield t, q, lab

    def block(self, start: int, stop: int, threads: int = 1) -> np.ndarray:
        """Batches [start, stop) stacked into one [rows, D] array (rows of full batches except the last)."""
        stop = min(stop, self.spec.n_batches)
        sp = self.spec
        rows = min(sp.n_queries, stop * sp.batch) - start * sp.batch
        out = np.empty((rows, sp.dim), dtype=np.uint16 if sp.dtype == "bf16" else np.float32)
        # popularity tables are cached per epoch, so generate epoch by epoch, batches in parallel
        t = start
        while t < stop:
            epoch = (t * sp.batch) // sp.reshuffle_every
            first_of_next = -(-((epoch + 1) * sp.reshuffle_every) // sp.batch)   # ceil division
            epoch_end = min(stop, first_of_next)
            self._popularity(epoch)

            def job(tt):
                q, _ = self.batch(tt)
                o = (tt - start) * sp.batch
                out[o:o + q.shape[0]] = q

            _parallel(job, [(tt,) for tt in range(t, epoch_end)], threads)
            t = epoch_end
        return out
