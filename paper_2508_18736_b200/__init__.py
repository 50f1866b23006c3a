"""B200 (sm_100a) kernels for the hot path of a centroid-based semantic cache: exact batched
cosine lookup with top-k and a per-query hit threshold, running-mean hit updates,
MergeCentroids / FilteringCentroids and spare-space insertion, behind the C ABI of
``include/siso.h``.  This package is the thin Python binding: it marshals torch tensors to
pointers and calls ``libsiso.so``; every step runs in the library's own CUDA kernels."""
from .binding import (ACCESS_INF, EVICT_DECAY, MERGE_SIZES_ONLY, MERGE_WEIGHTED_MEAN, OPT_LOOKUP_PATH,
                      OPT_MERGE_MAX_CANDIDATES, OPT_MERGE_PATH, OPT_STREAM_FUSED, OPT_TENSOR_CTA_PAIR, OPT_SWEEP_FINALIZE,
                      OPT_STREAM_LIST, OPT_MERGE_SWEEP_PARTS, OPT_CHECKED, PATH_AUTO, PATH_SIMT,
                      PATH_STREAM, PATH_TENSOR, SisoCache, SisoError, combine_keys, load_library, lookup_small_noalloc, md1_wait,
                      choose_theta, correct_theta, tier_exit_sim, tier_finish, tier_select, route, select_evict)
from .tiered import TieredCache
from .sharded import ShardedCache, exchange, gather_keys, local_range, owner_of, run, run_lockstep, shard_rows

__all__ = ["SisoCache", "ShardedCache", "TieredCache", "tier_exit_sim", "tier_select", "tier_finish", "route", "select_evict", "combine_keys", "gather_keys", "exchange", "run", "run_lockstep", "shard_rows", "owner_of", "local_range", "SisoError", "load_library", "lookup_small_noalloc", "md1_wait", "choose_theta", "correct_theta", "ACCESS_INF", "EVICT_DECAY", "MERGE_SIZES_ONLY",
           "MERGE_WEIGHTED_MEAN", "OPT_LOOKUP_PATH", "OPT_MERGE_MAX_CANDIDATES", "OPT_MERGE_PATH", "OPT_STREAM_FUSED",
           "OPT_TENSOR_CTA_PAIR", "OPT_SWEEP_FINALIZE", "OPT_STREAM_LIST", "OPT_MERGE_SWEEP_PARTS", "OPT_CHECKED", "PATH_AUTO", "PATH_SIMT", "PATH_STREAM", "PATH_TENSOR"]
