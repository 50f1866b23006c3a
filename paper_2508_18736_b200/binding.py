"""ctypes binding of libsiso.so.  Argument marshalling only; names follow include/siso.h."""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libsiso.so")

ACCESS_INF = 0xFFFFFFFF
MERGE_SIZES_ONLY, MERGE_WEIGHTED_MEAN = 0, 1
EVICT_DECAY = 1
OPT_LOOKUP_PATH, OPT_MERGE_MAX_CANDIDATES, OPT_TENSOR_CTA_PAIR, OPT_STREAM_FUSED, OPT_MERGE_PATH = 1, 2, 3, 4, 5
OPT_SWEEP_FINALIZE, OPT_STREAM_LIST, OPT_MERGE_SWEEP_PARTS, OPT_CHECKED = 6, 7, 8, 9
PATH_AUTO, PATH_SIMT, PATH_TENSOR, PATH_STREAM = 0, 1, 2, 3
_STATUS_NAMES = {0: "SISO_OK", 1: "SISO_ERR_INVALID_ARG", 2: "SISO_ERR_UNSUPPORTED", 3: "SISO_ERR_OOM",
                 4: "SISO_ERR_CAPACITY", 5: "SISO_ERR_OVERFLOW", 6: "SISO_ERR_TIMEOUT", 7: "SISO_ERR_CUDA"}

EXPORTS = ["siso_cache_create", "siso_cache_destroy", "siso_set_option", "siso_insert", "siso_lookup",
           "siso_lookup_host", "siso_update", "siso_merge", "siso_evict", "siso_make_room", "siso_insert_misses",
           "siso_stream_step", "siso_export", "siso_import", "siso_get_stats", "siso_sync_status",
           "siso_launch_count", "siso_status_string", "siso_last_cuda_error", "siso_lookup_small_noalloc", "siso_cluster", "siso_cache_copy", "siso_update_centroids", "siso_lookup_keys", "siso_combine_keys", "siso_t2h", "siso_md1_wait",
           "siso_choose_theta", "siso_correct_theta", "siso_tier_exit_sim", "siso_tier_select", "siso_tier_finish",
           "siso_route", "siso_evict_keys", "siso_select_evict", "siso_evict_slots", "siso_selftest_wait_timeout",
           "siso_measure_fp32_fma", "siso_pair_sweep_block", "siso_merge_resolve", "siso_merge_pack",
           "siso_merge_apply_shard", "siso_tier_build", "siso_tier_work_bytes", "siso_tier_lookup", "siso_free_slots",
           "siso_shard_plan", "siso_route_planned", "siso_select_evict_planned", "siso_norm_deviation"]


class SisoError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        name = _STATUS_NAMES.get(status, str(status))
        super().__init__(f"{where}: {name}" + (f" ({detail})" if detail else ""))


_ALLOC_FN = ctypes.CFUNCTYPE(ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p, ctypes.c_void_p)
_FREE_FN = ctypes.CFUNCTYPE(None, ctypes.c_void_p, ctypes.c_void_p)


class _Allocator(ctypes.Structure):
    _fields_ = [("alloc", _ALLOC_FN), ("free", _FREE_FN), ("ctx", ctypes.c_void_p)]


class _Config(ctypes.Structure):
    _fields_ = [("capacity", ctypes.c_int64), ("dim", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("device", ctypes.c_int32), ("reserved", ctypes.c_int32), ("decay", ctypes.c_double),
                ("allocator", _Allocator)]


_lib = None


def load_library(path: Optional[str] = None) -> ctypes.CDLL:
    """Load libsiso.so.  There is no fallback: a missing library is an error."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or _LIB_PATH
    if not os.path.exists(p):
        raise ImportError(f"{p} not found: build it with `python -m paper_2508_18736_b200.build` "
                          "(nvcc, sm_100a); this package has no CPU or PyTorch fallback")
    L = ctypes.CDLL(p)
    vp, i64, i32, u32, f32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_uint32, ctypes.c_float
    L.siso_cache_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(_Config)]
    L.siso_cache_destroy.argtypes = [vp]
    L.siso_set_option.argtypes = [vp, i32, i64]
    L.siso_insert.argtypes = [vp, vp, vp, i64, vp, vp]
    L.siso_lookup.argtypes = [vp, vp, i64, vp, f32, i32, vp, vp, vp, vp]
    L.siso_lookup_host.argtypes = [vp, vp, i64, vp, f32, i32, vp, vp, vp, vp]
    L.siso_update.argtypes = [vp, vp, i64, vp, i32, vp, vp]
    L.siso_merge.argtypes = [vp, vp, vp, i64, f32, u32, vp, ctypes.POINTER(i64), vp]
    L.siso_evict.argtypes = [vp, i64, u32, vp, vp]
    L.siso_make_room.argtypes = [vp, vp, i64, u32, vp, vp]
    L.siso_insert_misses.argtypes = [vp, vp, i64, vp, vp, vp]
    L.siso_stream_step.argtypes = [vp, vp, i64, vp, f32, vp, vp, vp, vp, vp, vp]
    L.siso_lookup_small_noalloc.argtypes = [vp, vp, i64, i32, i32, vp, i64, vp, f32, i32, vp, vp, vp, vp]
    L.siso_t2h.argtypes = [vp, vp, i64, vp, i32, vp, vp]
    L.siso_lookup_keys.argtypes = [vp, vp, i64, i32, i64, vp, vp]
    L.siso_combine_keys.argtypes = [vp, i64, i32, i32, vp, f32, vp, vp, vp, vp]
    L.siso_cache_copy.argtypes = [vp, vp, vp]
    L.siso_update_centroids.argtypes = [vp, vp, i64, i64, vp]
    L.siso_cluster.argtypes = [vp, vp, i64, f32, vp, vp, vp, vp, ctypes.POINTER(i64), vp]
    L.siso_route.argtypes = [vp, i64, vp, i64, i64, i64, i64, i64, vp, vp, vp, vp]
    L.siso_evict_keys.argtypes = [vp, i64, i64, vp, vp]
    L.siso_select_evict.argtypes = [vp, i32, i64, i64, vp, vp]
    L.siso_evict_slots.argtypes = [vp, vp, i64, i64, u32, vp]
    L.siso_free_slots.argtypes = [vp, vp, vp]
    L.siso_norm_deviation.argtypes = [vp, ctypes.POINTER(ctypes.c_double), vp]
    L.siso_shard_plan.argtypes = [vp, i64, vp, i32, i32, vp, vp]
    L.siso_route_planned.argtypes = [vp, i64, vp, i64, i64, i64, vp, vp, vp, vp, vp]
    L.siso_select_evict_planned.argtypes = [vp, i32, i64, vp, vp, vp]
    L.siso_tier_exit_sim.argtypes = [ctypes.c_double] * 2
    L.siso_tier_exit_sim.restype = ctypes.c_double
    L.siso_tier_select.argtypes = [vp, i64, f32, vp, i64, vp, vp, vp, vp]
    L.siso_tier_finish.argtypes = [vp, i64, f32, vp, vp, i64, vp, vp, vp, f32, vp, vp, vp, vp]
    L.siso_md1_wait.argtypes = [ctypes.c_double] * 3
    L.siso_md1_wait.restype = ctypes.c_double
    L.siso_choose_theta.argtypes = [vp, vp, i32, ctypes.c_double, ctypes.c_double, ctypes.c_double,
                                    ctypes.POINTER(ctypes.c_double)]
    L.siso_correct_theta.argtypes = [vp, i32, i32, ctypes.c_double, ctypes.c_double]
    L.siso_export.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp]
    L.siso_import.argtypes = [vp, vp, vp, vp, vp, vp, ctypes.c_uint64, vp]
    L.siso_get_stats.argtypes = [vp, ctypes.POINTER(i64), vp]
    L.siso_sync_status.argtypes = [vp, vp]
    L.siso_selftest_wait_timeout.argtypes = [vp, u32, vp, vp]
    L.siso_measure_fp32_fma.argtypes = [vp, ctypes.POINTER(ctypes.c_double), vp]
    L.siso_pair_sweep_block.argtypes = [vp, i64, vp, vp, i64, i64, f32, vp, i64, vp, vp]
    L.siso_merge_resolve.argtypes = [vp, vp, i64, vp, i64, vp, vp, vp]
    L.siso_merge_pack.argtypes = [vp, vp, i64, i64, vp, vp, vp, vp, vp]
    L.siso_merge_apply_shard.argtypes = [vp, vp, i64, vp, vp, vp, i64, u32, vp]
    L.siso_tier_build.argtypes = [vp, i64, ctypes.c_double, vp, vp, vp, vp, ctypes.POINTER(i64), vp]
    L.siso_tier_work_bytes.argtypes = [i64, i32, i32]
    L.siso_tier_work_bytes.restype = i64
    L.siso_tier_lookup.argtypes = [vp, vp, vp, vp, vp, i64, f32, vp, f32, vp, vp, vp, vp, ctypes.POINTER(i64), vp]
    L.siso_launch_count.argtypes = [vp]
    L.siso_launch_count.restype = i64
    L.siso_status_string.argtypes = [i32]
    L.siso_status_string.restype = ctypes.c_char_p
    L.siso_last_cuda_error.argtypes = []
    L.siso_last_cuda_error.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name not in ("siso_launch_count", "siso_status_string", "siso_last_cuda_error", "siso_md1_wait", "siso_tier_exit_sim",
                        "siso_tier_work_bytes"):
            getattr(L, name).restype = i32
    if path is None:
        _lib = L
    return L


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream: Optional[torch.cuda.Stream]):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


class SisoCache:
    """Handle of one device-resident cache.  Methods mirror the C entry points one to one."""

    def __init__(self, capacity: int, dim: int, dtype: str = "bf16", device: int = 0, decay: float = 1.1,
                 use_torch_allocator: bool = True):
        if dtype not in ("f32", "bf16"):
            raise ValueError("dtype must be 'f32' or 'bf16'")
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required: this library has no CPU path")
        self._lib = load_library()
        self.capacity, self.dim, self.dtype, self.device = int(capacity), int(dim), dtype, int(device)
        self.torch_dtype = torch.float32 if dtype == "f32" else torch.bfloat16
        self._dev = torch.device("cuda", self.device)
        self._blocks = {}
        cfg = _Config()
        cfg.capacity, cfg.dim, cfg.dtype, cfg.device, cfg.decay = capacity, dim, 0 if dtype == "f32" else 1, device, decay
        if use_torch_allocator:
            # the cache's own state and scratch live in torch's caching allocator
            def _alloc(nbytes, stream, ctx):
                # the block is taken from the pool of the stream the library will first use it on (torch keeps one pool
                # per stream and orders a block's reuse only against that stream); the library waits for the device before
                # it hands a block back, so the release below needs no stream
                try:
                    with torch.cuda.device(self._dev):
                        if stream:
                            with torch.cuda.stream(torch.cuda.ExternalStream(int(stream), device=self._dev)):
                                t = torch.empty(int(nbytes), dtype=torch.uint8, device=self._dev)
                        else:
                            t = torch.empty(int(nbytes), dtype=torch.uint8, device=self._dev)
                except Exception:       # out of memory -> NULL -> SISO_ERR_OOM
                    return None
                self._blocks[t.data_ptr()] = t
                return t.data_ptr()

            def _free(ptr, ctx):
                self._blocks.pop(ptr, None)

            self._alloc_cb, self._free_cb = _ALLOC_FN(_alloc), _FREE_FN(_free)
            cfg.allocator = _Allocator(self._alloc_cb, self._free_cb, None)
        h = ctypes.c_void_p()
        st = self._lib.siso_cache_create(ctypes.byref(h), ctypes.byref(cfg))
        self._h = h if st == 0 else None
        self._check(st, "siso_cache_create")

    # ------------------------------------------------------------------ helpers
    def _check(self, st: int, where: str) -> None:
        if st != 0:
            raise SisoError(st, where, self._lib.siso_last_cuda_error().decode() if st == 7 else "")

    def _vec(self, t: torch.Tensor, name: str) -> torch.Tensor:
        if t.dtype != self.torch_dtype or t.device != self._dev or t.dim() != 2 or t.shape[1] != self.dim:
            raise ValueError(f"{name} must be a [{'n'}, {self.dim}] {self.torch_dtype} tensor on {self._dev}")
        return t.contiguous()

    def _new(self, shape, dtype) -> torch.Tensor:
        return torch.empty(shape, dtype=dtype, device=self._dev)

    def close(self) -> None:
        if getattr(self, "_h", None) is not None:
            self._lib.siso_cache_destroy(self._h)
            self._h = None
            self._blocks.clear()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ------------------------------------------------------------------ entry points
    def set_option(self, key: int, value: int) -> None:
        self._check(self._lib.siso_set_option(self._h, key, value), "siso_set_option")

    def set_lookup_path(self, path: int) -> None:
        self.set_option(OPT_LOOKUP_PATH, path)

    def insert(self, vecs: torch.Tensor, sizes: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        vecs = self._vec(vecs, "vecs")
        n = vecs.shape[0]
        if sizes is not None:
            sizes = sizes.to(device=self._dev, dtype=torch.float64).contiguous()
            assert sizes.numel() == n
        slots = self._new((n,), torch.int32)
        self._check(self._lib.siso_insert(self._h, _ptr(vecs), _ptr(sizes), n, _ptr(slots), _stream(stream)), "siso_insert")
        return slots

    def lookup(self, queries: torch.Tensor, theta, k: int = 1, stream=None, out=None
               ) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
        """theta: float (same threshold for all) or fp32 tensor [n].  Returns idx[n,k], sim[n,k], hit[n]."""
        q = self._vec(queries, "queries")
        n = q.shape[0]
        th_t, th_s = (theta.to(device=self._dev, dtype=torch.float32).contiguous(), 0.0) \
            if isinstance(theta, torch.Tensor) else (None, float(theta))
        if th_t is not None:
            assert th_t.numel() == n
        idx, sim, hit = out if out is not None else (self._new((n, k), torch.int32), self._new((n, k), torch.float32),
                                                      self._new((n,), torch.uint8))
        self._check(self._lib.siso_lookup(self._h, _ptr(q), n, _ptr(th_t), th_s, k, _ptr(idx), _ptr(sim), _ptr(hit),
                                          _stream(stream)), "siso_lookup")
        return idx, sim, hit

    def lookup_host(self, h_queries: torch.Tensor, h_theta: Optional[torch.Tensor], theta_scalar: float, k: int,
                    h_idx: torch.Tensor, h_sim: torch.Tensor, h_hit: torch.Tensor, stream=None) -> None:
        """All tensors live in (pinned) host memory; results are valid after the stream is synchronised."""
        n = h_queries.shape[0]
        self._check(self._lib.siso_lookup_host(self._h, _ptr(h_queries), n, _ptr(h_theta), float(theta_scalar), k,
                                               _ptr(h_idx), _ptr(h_sim), _ptr(h_hit), _stream(stream)), "siso_lookup_host")

    def update(self, queries: torch.Tensor, idx: torch.Tensor, hit: torch.Tensor, stream=None) -> None:
        q = self._vec(queries, "queries")
        n = q.shape[0]
        assert idx.dtype == torch.int32 and hit.dtype == torch.uint8 and idx.is_contiguous() and hit.is_contiguous()
        stride = 1 if idx.dim() == 1 else idx.shape[1]
        self._check(self._lib.siso_update(self._h, _ptr(q), n, _ptr(idx), stride, _ptr(hit), _stream(stream)), "siso_update")

    def merge(self, theta_c: float, flags: int = MERGE_WEIGHTED_MEAN, want_count: bool = True, stream=None,
              repo: Optional[torch.Tensor] = None, repo_sizes: Optional[torch.Tensor] = None
              ) -> Tuple[torch.Tensor, Optional[int]]:
        """MergeCentroids: the cache with itself, or (repo given) the cache as C_cur with the rows of `repo` as
        C_repo.  Returns (merge_map [capacity], number merged or None)."""
        mm = self._new((self.capacity,), torch.int32)
        n = ctypes.c_int64(0)
        n_repo = 0
        if repo is not None:
            repo = self._vec(repo, "repo")
            n_repo = repo.shape[0]
            if repo_sizes is not None:
                repo_sizes = repo_sizes.to(device=self._dev, dtype=torch.float64).contiguous()
        st = self._lib.siso_merge(self._h, _ptr(repo), _ptr(repo_sizes), n_repo, float(theta_c), flags, _ptr(mm),
                                  ctypes.byref(n) if want_count else None, _stream(stream))
        self._check(st, "siso_merge")
        return mm, (int(n.value) if want_count else None)

    def evict(self, n_evict: int, flags: int = 0, stream=None) -> torch.Tensor:
        victims = self._new((max(int(n_evict), 0),), torch.int32)
        self._check(self._lib.siso_evict(self._h, int(n_evict), flags, _ptr(victims), _stream(stream)), "siso_evict")
        return victims

    def make_room(self, hit: torch.Tensor, flags: int = 0, stream=None) -> torch.Tensor:
        n = hit.numel()
        victims = self._new((n,), torch.int32)
        self._check(self._lib.siso_make_room(self._h, _ptr(hit), n, flags, _ptr(victims), _stream(stream)), "siso_make_room")
        return victims

    def insert_misses(self, queries: torch.Tensor, hit: torch.Tensor, stream=None) -> torch.Tensor:
        q = self._vec(queries, "queries")
        n = q.shape[0]
        slots = self._new((n,), torch.int32)
        self._check(self._lib.siso_insert_misses(self._h, _ptr(q), n, _ptr(hit), _ptr(slots), _stream(stream)),
                    "siso_insert_misses")
        return slots

    def stream_step(self, queries: torch.Tensor, theta, stream=None, out=None):
        """lookup(k=1) -> update -> make_room -> insert_misses.  Returns idx, sim, hit, victims, slots."""
        q = self._vec(queries, "queries")
        n = q.shape[0]
        th_t, th_s = (theta.to(device=self._dev, dtype=torch.float32).contiguous(), 0.0) \
            if isinstance(theta, torch.Tensor) else (None, float(theta))
        if out is None:
            out = (self._new((n, 1), torch.int32), self._new((n, 1), torch.float32), self._new((n,), torch.uint8),
                   self._new((n,), torch.int32), self._new((n,), torch.int32))
        idx, sim, hit, victims, slots = out
        self._check(self._lib.siso_stream_step(self._h, _ptr(q), n, _ptr(th_t), th_s, _ptr(idx), _ptr(sim), _ptr(hit),
                                               _ptr(victims), _ptr(slots), _stream(stream)), "siso_stream_step")
        return out

    def lookup_keys(self, queries: torch.Tensor, k: int = 1, slot_offset: int = 0, stream=None) -> torch.Tensor:
        """This shard's top-k as packed keys [n, k] (int64 tensor holding the 64-bit patterns); see siso_lookup_keys."""
        q = self._vec(queries, "queries")
        keys = self._new((q.shape[0], k), torch.int64)
        self._check(self._lib.siso_lookup_keys(self._h, _ptr(q), q.shape[0], k, int(slot_offset), _ptr(keys), _stream(stream)),
                    "siso_lookup_keys")
        return keys

    def evict_keys(self, n: int, slot_offset: int = 0, stream=None) -> torch.Tensor:
        """This shard's n lowest entries in eviction order as keys [n, 3] (int64 tensor of the 64-bit words); see siso_evict_keys."""
        keys = self._new((max(int(n), 0), 3), torch.int64)
        self._check(self._lib.siso_evict_keys(self._h, int(n), int(slot_offset), _ptr(keys), _stream(stream)), "siso_evict_keys")
        return keys

    def evict_slots(self, victims: torch.Tensor, slot_offset: int = 0, flags: int = 0, stream=None) -> None:
        """Drops the global victims that this shard holds (see siso_evict_slots)."""
        v = victims.to(device=self._dev, dtype=torch.int64).contiguous()
        self._check(self._lib.siso_evict_slots(self._h, _ptr(v), v.numel(), int(slot_offset), flags, _stream(stream)),
                    "siso_evict_slots")

    def norm_deviation(self, stream=None) -> float:
        """Largest | |v| - 1 | over the live entries' lookup vectors (see siso_norm_deviation)."""
        out = ctypes.c_double(0.0)
        self._check(self._lib.siso_norm_deviation(self._h, ctypes.byref(out), _stream(stream)), "siso_norm_deviation")
        return float(out.value)

    def free_slots(self, stream=None) -> torch.Tensor:
        """[1] int64 on the device: capacity - occupancy, without a host read (see siso_free_slots)."""
        out = self._new((1,), torch.int64)
        self._check(self._lib.siso_free_slots(self._h, _ptr(out), _stream(stream)), "siso_free_slots")
        return out

    def copy_from(self, src: "SisoCache", stream=None) -> None:
        """C_new <- C_cur (first line of MergeCentroids, Algorithm 1): every slot of `src` into the same slot here."""
        self._check(self._lib.siso_cache_copy(self._h, src._h, _stream(stream)), "siso_cache_copy")

    def update_centroids(self, c_new: "SisoCache", first_slot: int, n_slots: int, stream=None) -> None:
        """UpdateCentroids of Algorithm 1, one group of destination slots (see include/siso.h)."""
        self._check(self._lib.siso_update_centroids(self._h, c_new._h, int(first_slot), int(n_slots), _stream(stream)),
                    "siso_update_centroids")

    def cluster(self, vecs: torch.Tensor, theta_c: float, want_centroids: bool = True, stream=None):
        """Community detection at theta_c over the rows of `vecs` (the cache's contents are not touched).
        Returns (label [n] int32, centres [k] int32 in founding order, sizes [k] float64, centroids [k, dim] or None)."""
        v = self._vec(vecs, "vecs")
        n = v.shape[0]
        label, centres = self._new((n,), torch.int32), self._new((n,), torch.int32)
        sizes = self._new((n,), torch.float64)
        cent = self._new((n, self.dim), self.torch_dtype) if want_centroids else None
        k = ctypes.c_int64(0)
        self._check(self._lib.siso_cluster(self._h, _ptr(v), n, float(theta_c), _ptr(label), _ptr(centres), _ptr(sizes),
                                           _ptr(cent), ctypes.byref(k), _stream(stream)), "siso_cluster")
        k = int(k.value)
        return label, centres[:k], sizes[:k], (cent[:k] if want_centroids else None)

    def t2h(self, queries: torch.Tensor, thetas: torch.Tensor, stream=None) -> torch.Tensor:
        """Threshold-to-hit-ratio counts: int64 [len(thetas)] = sampled queries whose best similarity > theta."""
        q = self._vec(queries, "queries")
        th = thetas.to(device=self._dev, dtype=torch.float32).contiguous()
        hits = self._new((th.numel(),), torch.int64)
        self._check(self._lib.siso_t2h(self._h, _ptr(q), q.shape[0], _ptr(th), th.numel(), _ptr(hits), _stream(stream)),
                    "siso_t2h")
        return hits

    def export(self, stream=None) -> dict:
        out = dict(vecs=self._new((self.capacity, self.dim), self.torch_dtype),
                   master=self._new((self.capacity, self.dim), torch.float32),
                   size=self._new((self.capacity,), torch.float64),
                   access=self._new((self.capacity,), torch.int32),        # bit pattern of the uint32 counters
                   last=self._new((self.capacity,), torch.int64),
                   valid=self._new((self.capacity,), torch.uint8))
        self._check(self._lib.siso_export(self._h, _ptr(out["vecs"]), _ptr(out["master"]), _ptr(out["size"]),
                                          _ptr(out["access"]), _ptr(out["last"]), _ptr(out["valid"]), _stream(stream)),
                    "siso_export")
        return out

    def import_(self, master: torch.Tensor, size: torch.Tensor, access: torch.Tensor, last: torch.Tensor,
                valid: torch.Tensor, clock: int, stream=None) -> None:
        args = [master.to(self._dev, torch.float32).contiguous(), size.to(self._dev, torch.float64).contiguous(),
                access.to(self._dev).contiguous(), last.to(self._dev).contiguous(),
                valid.to(self._dev, torch.uint8).contiguous()]
        assert args[0].shape == (self.capacity, self.dim) and args[2].element_size() == 4 and args[3].element_size() == 8
        self._check(self._lib.siso_import(self._h, *[_ptr(a) for a in args], int(clock), _stream(stream)), "siso_import")
        torch.cuda.current_stream().synchronize() if stream is None else stream.synchronize()

    def stats(self, stream=None) -> dict:
        buf = (ctypes.c_int64 * 8)()
        self._check(self._lib.siso_get_stats(self._h, buf, _stream(stream)), "siso_get_stats")
        names = ["occupancy", "lookups", "hits", "inserts", "evictions", "merges", "clock", "rescans"]
        return {n: int(buf[i]) for i, n in enumerate(names)}

    # ---- MergeCentroids over a cache partitioned across GPUs (see siso_pair_sweep_block ... in siso.h) ----
    def pair_sweep_block(self, own_offset: int, theta_c: float, cand: torch.Tensor, n_cand: torch.Tensor,
                         peer_master: Optional[torch.Tensor] = None, peer_valid: Optional[torch.Tensor] = None,
                         peer_offset: int = 0, stream=None) -> None:
        """Appends the pairs of this block with itself (no peer) or with a peer block to cand [max, 3] int32 at n_cand."""
        assert cand.dtype == torch.int32 and cand.dim() == 2 and cand.shape[1] == 3 and cand.is_contiguous()
        assert n_cand.dtype == torch.int64 and n_cand.numel() == 1
        n_peer = 0
        if peer_master is not None:
            peer_master = peer_master.to(self._dev, torch.float32).contiguous()
            peer_valid = peer_valid.to(self._dev, torch.uint8).contiguous()
            n_peer = peer_master.shape[0]
            assert peer_master.shape[1] == self.dim and peer_valid.numel() == n_peer
        self._check(self._lib.siso_pair_sweep_block(self._h, int(own_offset), _ptr(peer_master) if n_peer else None,
                                                    _ptr(peer_valid) if n_peer else None, n_peer, int(peer_offset), float(theta_c),
                                                    _ptr(cand), cand.shape[0], _ptr(n_cand), _stream(stream)), "siso_pair_sweep_block")

    def merge_resolve(self, cand: torch.Tensor, valid: torch.Tensor, stream=None):
        """Candidates of all shards [n, 3] int32 + live flags of all global slots -> (merge_map int32 [n_total], n_merged int64 [1])."""
        cand = cand.to(self._dev, torch.int32).contiguous()
        valid = valid.to(self._dev, torch.uint8).contiguous()
        mm = self._new((valid.numel(),), torch.int32)
        n = self._new((1,), torch.int64)
        self._check(self._lib.siso_merge_resolve(self._h, _ptr(cand) if cand.shape[0] else None, cand.shape[0], _ptr(valid),
                                                 valid.numel(), _ptr(mm), _ptr(n), _stream(stream)), "siso_merge_resolve")
        return mm, n

    def merge_pack(self, merge_map: torch.Tensor, own_offset: int, capacity: int, with_rows: bool, stream=None):
        """This shard's merged rows: (meta int32 [capacity, 2], sizes f64 [capacity], rows f32 [capacity, dim] or None, n int64 [1])."""
        cap = max(1, int(capacity))
        meta, sizes = self._new((cap, 2), torch.int32), self._new((cap,), torch.float64)
        rows = self._new((cap, self.dim), torch.float32) if with_rows else None
        n = self._new((1,), torch.int64)
        self._check(self._lib.siso_merge_pack(self._h, _ptr(merge_map), int(own_offset), cap, _ptr(meta), _ptr(sizes), _ptr(rows),
                                              _ptr(n), _stream(stream)), "siso_merge_pack")
        return meta, sizes, rows, n

    def merge_apply_shard(self, merge_map: torch.Tensor, own_offset: int, meta: torch.Tensor, sizes: torch.Tensor,
                          rows: Optional[torch.Tensor], flags: int, stream=None) -> None:
        meta, sizes = meta.contiguous(), sizes.contiguous()
        rows = None if rows is None else rows.contiguous()
        self._check(self._lib.siso_merge_apply_shard(self._h, _ptr(merge_map), int(own_offset), _ptr(meta), _ptr(sizes), _ptr(rows),
                                                     meta.shape[0], int(flags), _stream(stream)), "siso_merge_apply_shard")

    def selftest_wait_timeout(self, poll_limit: int = 4096, stream=None) -> torch.Tensor:
        """Lets one bounded device-side wait run out (see siso_selftest_wait_timeout); returns the device flag."""
        flag = torch.zeros(1, dtype=torch.int32, device=self._dev)
        self._check(self._lib.siso_selftest_wait_timeout(self._h, int(poll_limit), _ptr(flag), _stream(stream)),
                    "siso_selftest_wait_timeout")
        return flag

    def measure_fp32_fma(self, stream=None) -> float:
        """Measured FP32 FMA throughput of the CUDA cores in TFLOP/s."""
        v = ctypes.c_double(0.0)
        self._check(self._lib.siso_measure_fp32_fma(self._h, ctypes.byref(v), _stream(stream)), "siso_measure_fp32_fma")
        return float(v.value)

    def sync_status(self, stream=None) -> int:
        """Synchronise and return the device status word (0 = clear); it is cleared by the call."""
        return int(self._lib.siso_sync_status(self._h, _stream(stream)))

    def check_status(self, stream=None) -> None:
        st = self.sync_status(stream)
        if st != 0:
            raise SisoError(st, "device status")

    @property
    def launch_count(self) -> int:
        return int(self._lib.siso_launch_count(self._h))


def lookup_small_noalloc(centroids: torch.Tensor, queries: torch.Tensor, theta, k: int, idx: torch.Tensor,
                         sim: torch.Tensor, hit: torch.Tensor, valid: Optional[torch.Tensor] = None, stream=None) -> None:
    """Lookup of at most 8 queries that allocates no device memory: the caller owns every buffer, outputs
    included, and the library's scratch is a fixed array inside its image.  For callers that must not
    call the CUDA allocator (see include/siso.h).  Calls that can overlap on the GPU must be ordered by
    the caller.  Raises SisoError for sizes beyond the fixed limits."""
    L = load_library()
    dtype = {torch.float32: 0, torch.bfloat16: 1}[centroids.dtype]
    assert queries.dtype == centroids.dtype and centroids.is_contiguous() and queries.is_contiguous()
    th_t, th_s = (theta, 0.0) if isinstance(theta, torch.Tensor) else (None, float(theta))
    with torch.cuda.device(centroids.device):
        st = L.siso_lookup_small_noalloc(_ptr(centroids), _ptr(valid), centroids.shape[0], centroids.shape[1], dtype,
                                         _ptr(queries), queries.shape[0], _ptr(th_t), th_s, k, _ptr(idx), _ptr(sim),
                                         _ptr(hit), _stream(stream))
    if st != 0:
        raise SisoError(st, "siso_lookup_small_noalloc", L.siso_last_cuda_error().decode() if st == 7 else "")


def combine_keys(keys: torch.Tensor, theta, stream=None) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """keys [n, n_lists, k] (int64 tensor of packed keys on a GPU) -> (idx [n, k] int64 global slots, sim [n, k], hit [n])."""
    assert keys.dtype == torch.int64 and keys.dim() == 3 and keys.is_cuda
    keys = keys.contiguous()
    n, n_lists, k = keys.shape
    th_t, th_s = (theta.to(device=keys.device, dtype=torch.float32).contiguous(), 0.0) \
        if isinstance(theta, torch.Tensor) else (None, float(theta))
    idx = torch.empty((n, k), dtype=torch.int64, device=keys.device)
    sim = torch.empty((n, k), dtype=torch.float32, device=keys.device)
    hit = torch.empty((n,), dtype=torch.uint8, device=keys.device)
    with torch.cuda.device(keys.device):
        st = load_library().siso_combine_keys(_ptr(keys), n, n_lists, k, _ptr(th_t), th_s, _ptr(idx), _ptr(sim), _ptr(hit),
                                              _stream(stream))
    if st != 0:
        raise SisoError(st, "siso_combine_keys")
    return idx, sim, hit


def route(idx: torch.Tensor, hit: torch.Tensor, slot_lo: int, slot_hi: int, miss_skip: int = 0, miss_take: int = 0, stream=None,
          plan: Optional[torch.Tensor] = None):
    """Combined (idx [n] or [n, k] int64 global slots, hit [n]) -> (idx_local [n] int32, update_hit [n], insert_hit [n]) for
    the shard that owns [slot_lo, slot_hi) (see siso_route).  With `plan` (the device tensor shard_plan wrote) the two miss
    counts are read from it on the device (siso_route_planned)."""
    assert idx.dtype == torch.int64 and idx.is_cuda and hit.dtype == torch.uint8
    idx, hit = idx.contiguous(), hit.contiguous()
    n = hit.numel()
    stride = 1 if idx.dim() == 1 else idx.shape[1]
    idx_local = torch.empty((n,), dtype=torch.int32, device=idx.device)
    upd, ins = torch.empty_like(hit), torch.empty_like(hit)
    with torch.cuda.device(idx.device):
        if plan is None:
            st = load_library().siso_route(_ptr(idx), stride, _ptr(hit), n, int(slot_lo), int(slot_hi), int(miss_skip),
                                           int(miss_take), _ptr(idx_local), _ptr(upd), _ptr(ins), _stream(stream))
        else:
            assert plan.dtype == torch.int64 and plan.numel() == 4 and plan.device == idx.device
            st = load_library().siso_route_planned(_ptr(idx), stride, _ptr(hit), n, int(slot_lo), int(slot_hi), _ptr(plan),
                                                   _ptr(idx_local), _ptr(upd), _ptr(ins), _stream(stream))
    if st != 0:
        raise SisoError(st, "siso_route")
    return idx_local, upd, ins


def shard_plan(hit: torch.Tensor, free_all: torch.Tensor, rank: int, stream=None) -> torch.Tensor:
    """hit [n] of a combined lookup and free_all [world] int64 (every shard's free slots) -> plan [4] int64 on the device:
    misses, entries to evict over the whole cache, free slots before `rank`, free slots on `rank` (see siso_shard_plan)."""
    assert hit.dtype == torch.uint8 and hit.is_cuda and free_all.dtype == torch.int64 and free_all.device == hit.device
    hit, free_all = hit.contiguous(), free_all.reshape(-1).contiguous()
    plan = torch.empty((4,), dtype=torch.int64, device=hit.device)
    with torch.cuda.device(hit.device):
        st = load_library().siso_shard_plan(_ptr(hit), hit.numel(), _ptr(free_all), free_all.numel(), int(rank), _ptr(plan),
                                            _stream(stream))
    if st != 0:
        raise SisoError(st, "siso_shard_plan")
    return plan


def select_evict_planned(keys: torch.Tensor, plan: torch.Tensor, stream=None) -> torch.Tensor:
    """keys [n_lists, n, 3] -> victims [n] int64: the plan[1] lowest of all keys in eviction order, then -1."""
    assert keys.dtype == torch.int64 and keys.dim() == 3 and keys.shape[2] == 3 and keys.is_cuda
    assert plan.dtype == torch.int64 and plan.numel() == 4 and plan.device == keys.device
    keys = keys.contiguous()
    victims = torch.empty((keys.shape[1],), dtype=torch.int64, device=keys.device)
    with torch.cuda.device(keys.device):
        st = load_library().siso_select_evict_planned(_ptr(keys), keys.shape[0], keys.shape[1], _ptr(plan), _ptr(victims),
                                                      _stream(stream))
    if st != 0:
        raise SisoError(st, "siso_select_evict_planned")
    return victims


def select_evict(keys: torch.Tensor, n_take: int, stream=None) -> torch.Tensor:
    """keys [n_lists, n, 3] (the shards' siso_evict_keys lists) -> victims [n_take] int64 global slots in eviction order."""
    assert keys.dtype == torch.int64 and keys.dim() == 3 and keys.shape[2] == 3 and keys.is_cuda
    keys = keys.contiguous()
    victims = torch.empty((max(int(n_take), 0),), dtype=torch.int64, device=keys.device)
    with torch.cuda.device(keys.device):
        st = load_library().siso_select_evict(_ptr(keys), keys.shape[0], keys.shape[1], int(n_take), _ptr(victims), _stream(stream))
    if st != 0:
        raise SisoError(st, "siso_select_evict")
    return victims


def tier_exit_sim(sep_sim: float, norm_slack: float = 0.0) -> float:
    """Exit similarity of the locality-ordered search for a hot/cold separation bound (see siso_tier_exit_sim)."""
    return float(load_library().siso_tier_exit_sim(float(sep_sim), float(norm_slack)))


def tier_select(hot_keys: torch.Tensor, queries: torch.Tensor, exit_sim: float, stream=None):
    """hot_keys [n] or [n, 1] packed keys, queries [n, dim] -> (rows [n] int32, packed queries [n, dim], count [1] int64
    on the device): the queries that must also search the cold tier (see siso_tier_select)."""
    hk = hot_keys.reshape(-1).contiguous()
    q = queries.contiguous()
    n = q.shape[0]
    assert hk.dtype == torch.int64 and hk.numel() == n and q.is_cuda
    rows = torch.empty((n,), dtype=torch.int32, device=q.device)
    packed = torch.empty_like(q)
    count = torch.empty((1,), dtype=torch.int64, device=q.device)
    with torch.cuda.device(q.device):
        st = load_library().siso_tier_select(_ptr(hk), n, float(exit_sim), _ptr(q), q.shape[1] * q.element_size(), _ptr(packed),
                                             _ptr(rows), _ptr(count), _stream(stream))
    if st != 0:
        raise SisoError(st, "siso_tier_select")
    return rows, packed, count


def tier_finish(hot_keys: torch.Tensor, exit_sim: float, cold_keys: Optional[torch.Tensor], rows: torch.Tensor, n_cold: int,
                hot_slot: Optional[torch.Tensor], cold_slot: Optional[torch.Tensor], theta, stream=None):
    """-> (idx [n] int32, sim [n] fp32, hit [n] uint8): per query the better of its hot and cold keys (see siso_tier_finish)."""
    hk = hot_keys.reshape(-1).contiguous()
    n = hk.numel()
    ck = None if cold_keys is None else cold_keys.reshape(-1).contiguous()
    th_t, th_s = (theta.to(device=hk.device, dtype=torch.float32).contiguous(), 0.0) \
        if isinstance(theta, torch.Tensor) else (None, float(theta))
    idx = torch.empty((n,), dtype=torch.int32, device=hk.device)
    sim = torch.empty((n,), dtype=torch.float32, device=hk.device)
    hit = torch.empty((n,), dtype=torch.uint8, device=hk.device)
    with torch.cuda.device(hk.device):
        st = load_library().siso_tier_finish(_ptr(hk), n, float(exit_sim), _ptr(ck), _ptr(rows), int(n_cold), _ptr(hot_slot),
                                             _ptr(cold_slot), _ptr(th_t), th_s, _ptr(idx), _ptr(sim), _ptr(hit), _stream(stream))
    if st != 0:
        raise SisoError(st, "siso_tier_finish")
    return idx, sim, hit


def md1_wait(llm_latency: float, arrival_rate: float, hit_ratio: float) -> float:
    """Eq. 2 of the paper (M/D/1 mean waiting time with E = L(1 - h)); host arithmetic in the library."""
    return float(load_library().siso_md1_wait(float(llm_latency), float(arrival_rate), float(hit_ratio)))


def choose_theta(thetas, hit_ratio, llm_latency: float, arrival_rate: float, slo: float):
    """(index of the highest threshold whose estimated wait is below the SLO or -1, that wait)."""
    th = (ctypes.c_float * len(thetas))(*[float(x) for x in thetas])
    hr = (ctypes.c_double * len(hit_ratio))(*[float(x) for x in hit_ratio])
    w = ctypes.c_double(0.0)
    i = load_library().siso_choose_theta(th, hr, len(thetas), float(llm_latency), float(arrival_rate), float(slo),
                                         ctypes.byref(w))
    return int(i), float(w.value)


def correct_theta(thetas, chosen: int, wait_estimated: float, wait_measured: float) -> int:
    """One table entry down/up when estimate and measurement differ by more than 10 % (Sec. 4.3)."""
    th = (ctypes.c_float * len(thetas))(*[float(x) for x in thetas])
    return int(load_library().siso_correct_theta(th, len(thetas), int(chosen), float(wait_estimated), float(wait_measured)))
