"""CPU oracle (fp64) for the semantic-cache hot path: TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper around ``siso_oracle.c`` plus ``OracleCache``, a plain holder of
the cache state (fp64 master vectors, cluster_size, access_count, last_access,
valid mask, clock) whose methods call the C routines in the order a caller of the
GPU library would.  Nothing here is imported by, or imports, the CUDA package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "siso_oracle.c")
_LIBDIR = os.path.join(_HERE, "_build")
_LIB = os.path.join(_LIBDIR, "libsiso_oracle.so")

F32, BF16, F64 = 0, 1, 2
ACCESS_INF = 0xFFFFFFFF
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP across independent outer iterations only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        os.makedirs(_LIBDIR, exist_ok=True)
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fno-fast-math", "-ffp-contract=off", "-shared", "-fPIC",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        vp, i64, i32, f64 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_double
        L.siso_oracle_round_bf16.argtypes = [vp, vp, i64]
        L.siso_oracle_round_bf16.restype = None
        L.siso_oracle_lookup.argtypes = [vp, i32, vp, i64, i32, vp, i32, i64, vp, i32, vp, vp, vp]
        L.siso_oracle_lookup.restype = i32
        L.siso_oracle_update.argtypes = [vp, vp, vp, vp, vp, i64, i32, vp, i32, i64, vp, i64, vp, ctypes.c_uint64]
        L.siso_oracle_update.restype = i32
        L.siso_oracle_merge.argtypes = [vp, vp, vp, vp, i64, i32, vp, f64, i32, i32, vp]
        L.siso_oracle_merge.restype = i64
        L.siso_oracle_evict.argtypes = [vp, vp, vp, vp, i64, i64, i32, f64, vp]
        L.siso_oracle_evict.restype = i64
        L.siso_oracle_insert.argtypes = [vp, vp, vp, vp, vp, i64, i32, vp, i32, i64, vp, vp, ctypes.c_uint64, vp]
        L.siso_oracle_insert.restype = i64
        L.siso_oracle_t2h.argtypes = [vp, i64, vp, i32, vp, vp]
        L.siso_oracle_t2h.restype = None
        L.siso_oracle_md1_wait.argtypes = [f64, f64, f64]
        L.siso_oracle_md1_wait.restype = f64
        L.siso_oracle_choose_theta.argtypes = [vp, vp, i32, f64, f64, f64, ctypes.POINTER(f64)]
        L.siso_oracle_choose_theta.restype = i32
        L.siso_oracle_correct_theta.argtypes = [vp, i32, i32, f64, f64]
        L.siso_oracle_correct_theta.restype = i32
        L.siso_oracle_cluster.argtypes = [vp, i32, i64, i32, f64, vp, vp, vp, vp]
        L.siso_oracle_cluster.restype = i64
        _lib = L
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    if a.dtype == np.float64:
        return F64
    raise TypeError(f"vectors must be float32, float64 or uint16 (bfloat16 bits), got {a.dtype}")


def _c(a: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(a)


def round_bf16(x: np.ndarray) -> np.ndarray:
    """binary64 -> bfloat16 bit patterns, one rounding, ties to even."""
    x = _c(np.asarray(x, dtype=np.float64))
    out = np.empty(x.shape, dtype=np.uint16)
    lib().siso_oracle_round_bf16(_p(x), _p(out), x.size)
    return out


def widen(a: np.ndarray) -> np.ndarray:
    """fp32 / bfloat16 bits / fp64 -> fp64, exactly."""
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    return a.astype(np.float64)


def lookup(centroids: np.ndarray, queries: np.ndarray, theta, k: int = 1, valid: Optional[np.ndarray] = None
           ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Exact top-k by (similarity desc, slot asc) and the strict hit test.  Returns idx[B,k], sim[B,k] (fp64), hit[B]."""
    C, Q = _c(centroids), _c(queries)
    N, D = C.shape
    B = Q.shape[0]
    assert Q.shape[1] == D
    th = np.ascontiguousarray(np.broadcast_to(np.asarray(theta, dtype=np.float32), (B,)))
    v = None if valid is None else _c(valid.astype(np.uint8))
    idx = np.empty((B, k), dtype=np.int32)
    sim = np.empty((B, k), dtype=np.float64)
    hit = np.empty(B, dtype=np.uint8)
    rc = lib().siso_oracle_lookup(_p(C), _dtype_code(C), _p(v), N, D, _p(Q), _dtype_code(Q), B, _p(th), k,
                                  _p(idx), _p(sim), _p(hit))
    if rc:
        raise RuntimeError(f"oracle lookup failed ({rc})")
    return idx, sim, hit


def t2h_table(best_sims: np.ndarray, thetas: np.ndarray):
    """Threshold-to-hit-ratio table of Sec. 4.3: (hits int64 [T], ratio fp64 [T]) for a grid of thresholds."""
    b = _c(np.asarray(best_sims, dtype=np.float64))
    th = _c(np.asarray(thetas, dtype=np.float32))
    hits = np.empty(th.shape[0], dtype=np.int64)
    ratio = np.empty(th.shape[0], dtype=np.float64)
    lib().siso_oracle_t2h(_p(b), b.shape[0], _p(th), th.shape[0], _p(hits), _p(ratio))
    return hits, ratio


def md1_wait(L: float, lam: float, h: float) -> float:
    """Eq. 2: W = L(1-h) + lam L^2 (1-h)^2 / (2 (1 - lam L (1-h))); inf when lam L (1-h) >= 1."""
    return float(lib().siso_oracle_md1_wait(float(L), float(lam), float(h)))


def choose_theta(thetas: np.ndarray, ratio: np.ndarray, L: float, lam: float, slo: float):
    """Index of the highest threshold with W < slo (or -1), and that W."""
    th = _c(np.asarray(thetas, dtype=np.float32))
    r = _c(np.asarray(ratio, dtype=np.float64))
    w = ctypes.c_double(0.0)
    i = lib().siso_oracle_choose_theta(_p(th), _p(r), th.shape[0], float(L), float(lam), float(slo), ctypes.byref(w))
    return int(i), float(w.value)


def correct_theta(thetas: np.ndarray, chosen: int, w_est: float, w_meas: float) -> int:
    """Sec. 4.3 correction: one table entry down (measured wait longer) or up (shorter) if they differ by > 10 %."""
    th = _c(np.asarray(thetas, dtype=np.float32))
    return int(lib().siso_oracle_correct_theta(_p(th), th.shape[0], int(chosen), float(w_est), float(w_meas)))


def cluster(vecs: np.ndarray, theta_c: float, want_centroids: bool = True):
    """Community detection at theta_c (Sec. 4.1; the steps are stated at siso_oracle_cluster).
    Returns (label [n] int32, centres [k] int32 in founding order, sizes [k] float64, centroids [k, D] float64 or None)."""
    v = _c(vecs)
    n, D = v.shape
    label = np.empty(n, np.int32)
    centres = np.empty(n, np.int32)
    sizes = np.empty(n, np.float64)
    cent = np.empty((n, D), np.float64) if want_centroids else None
    k = lib().siso_oracle_cluster(_p(v), _dtype_code(v), n, D, float(theta_c), _p(label), _p(centres), _p(sizes), _p(cent))
    if k < 0:
        raise MemoryError("oracle clustering: allocation failed")
    return label, centres[:k].copy(), sizes[:k].copy(), (cent[:k].copy() if want_centroids else None)


class OracleCache:
    """Cache state in fp64 with the lookup copy derived by one rounding to the storage type."""

    def __init__(self, capacity: int, dim: int, dtype: str = "f32", decay: float = 1.1):
        assert dtype in ("f32", "bf16")
        self.capacity, self.dim, self.dtype, self.decay = int(capacity), int(dim), dtype, float(decay)
        self.master = np.zeros((capacity, dim), dtype=np.float64)
        self.size = np.zeros(capacity, dtype=np.float64)
        self.access = np.zeros(capacity, dtype=np.uint32)
        self.last = np.zeros(capacity, dtype=np.uint64)
        self.valid = np.zeros(capacity, dtype=np.uint8)
        self.clock = 0

    # -- state exchange ------------------------------------------------------
    def load_state(self, master, size, access, last, valid, clock: int) -> None:
        self.master[...] = widen(np.asarray(master))
        self.size[...] = size
        self.access[...] = access
        self.last[...] = last
        self.valid[...] = valid
        self.clock = int(clock)

    def copy_from(self, other: "OracleCache") -> None:
        """C_new <- C_cur, the first line of MergeCentroids (Algorithm 1): every slot of `other` into the same slot
        here (this cache may be larger; its remaining slots become empty)."""
        assert self.capacity >= other.capacity and self.dim == other.dim and self.dtype == other.dtype
        n = other.capacity
        self.valid[:] = 0
        self.master[:n], self.size[:n], self.access[:n] = other.master, other.size, other.access
        self.last[:n], self.valid[:n], self.clock = other.last, other.valid, other.clock

    def update_centroids(self, new: "OracleCache", first_slot: int, n_slots: int) -> None:
        """UpdateCentroids of Algorithm 1 (Sec. 4.2, update step), one group: the live entries of C_new, taken in
        ascending slot order, are numbered 0, 1, ...; slot d of this cache (first_slot <= d < first_slot + n_slots)
        receives entry number d, or becomes empty if C_new has no such entry.  Calling it for consecutive groups
        until the capacity is covered replaces C_cur by C_new."""
        assert self.dim == new.dim and self.dtype == new.dtype
        live = np.flatnonzero(new.valid)
        if len(live) > self.capacity:
            raise ValueError("C_new holds more entries than C_cur has slots")
        for d in range(first_slot, min(first_slot + n_slots, self.capacity)):
            if d < len(live):
                src = live[d]
                self.master[d], self.size[d], self.access[d] = new.master[src], new.size[src], new.access[src]
                self.last[d], self.valid[d] = new.last[src], 1
            else:
                self.valid[d] = 0

    def lookup_copy(self) -> np.ndarray:
        """What a lookup reads: the master rounded once to the storage type."""
        if self.dtype == "bf16":
            return round_bf16(self.master)
        return self.master.astype(np.float32)

    @property
    def occupancy(self) -> int:
        return int(self.valid.sum())

    # -- the steps -------------------------------------------------------------
    def lookup(self, queries, theta, k: int = 1):
        return lookup(self.lookup_copy(), queries, theta, k, self.valid)

    def update(self, queries, idx, hit) -> None:
        Q = _c(queries)
        idx = _c(np.asarray(idx, dtype=np.int32))
        stride = 1 if idx.ndim == 1 else idx.shape[1]
        hit = _c(np.asarray(hit, dtype=np.uint8))
        self.clock += 1
        rc = lib().siso_oracle_update(_p(self.master), _p(self.size), _p(self.access), _p(self.last), _p(self.valid),
                                      self.capacity, self.dim, _p(Q), _dtype_code(Q), Q.shape[0], _p(idx), stride,
                                      _p(hit), self.clock)
        if rc:
            raise RuntimeError(f"oracle update failed ({rc})")

    def merge(self, theta_c: float, weighted_mean: bool, n_seed: int = 0, new_access_inf: bool = False,
              seed_mask=None):
        """MergeCentroids over the slot array.  Seeds (C_cur) are the slots below n_seed, or those set in
        seed_mask; none = self-merge.  Returns (merge_map, n_merged)."""
        mm = np.empty(self.capacity, dtype=np.int32)
        if seed_mask is None and n_seed > 0:
            seed_mask = (np.arange(self.capacity) < n_seed)
        sm = None if seed_mask is None else _c(np.asarray(seed_mask).astype(np.uint8))
        n = lib().siso_oracle_merge(_p(self.master), _p(self.size), _p(self.access), _p(self.valid), self.capacity,
                                    self.dim, _p(sm), float(theta_c), int(weighted_mean), int(new_access_inf),
                                    _p(mm))
        if n < 0:
            raise MemoryError
        return mm, int(n)

    def evict(self, n_evict: int, decay: bool = False) -> np.ndarray:
        victims = np.empty(max(int(n_evict), 0), dtype=np.int32)
        lib().siso_oracle_evict(_p(self.size), _p(self.access), _p(self.last), _p(self.valid), self.capacity,
                                int(n_evict), int(decay), self.decay, _p(victims))
        return victims

    def insert(self, vectors, hit=None, sizes=None) -> np.ndarray:
        """Rows with hit == 0 (all rows if hit is None) take the free slots in ascending order."""
        Q = _c(vectors)
        h = None if hit is None else _c(np.asarray(hit, dtype=np.uint8))
        s = None if sizes is None else _c(np.asarray(sizes, dtype=np.float64))
        slots = np.empty(Q.shape[0], dtype=np.int32)
        n = lib().siso_oracle_insert(_p(self.master), _p(self.size), _p(self.access), _p(self.last), _p(self.valid),
                                     self.capacity, self.dim, _p(Q), _dtype_code(Q), Q.shape[0], _p(h), _p(s),
                                     self.clock, _p(slots))
        if n < 0:
            raise OverflowError("not enough free slots")
        return slots

    def stream_step(self, queries, theta, forced=None):
        """One micro-batch: lookup(k=1) -> update -> evict what is needed -> insert the misses.

        ``forced`` = (idx, hit) replaces this batch's own decisions (lock-step comparison with
        another implementation); the oracle's own (idx, sim, hit) are returned either way."""
        idx, sim, hit = self.lookup(queries, theta, 1)
        use_idx, use_hit = (idx, hit) if forced is None else forced
        use_idx = np.asarray(use_idx).reshape(len(hit), -1)[:, :1]
        self.update(queries, use_idx, use_hit)
        n_miss = int((np.asarray(use_hit) == 0).sum())
        free = self.capacity - self.occupancy
        victims = self.evict(n_miss - free) if n_miss > free else np.empty(0, dtype=np.int32)
        slots = self.insert(queries, use_hit)
        return idx, sim, hit, victims, slots
