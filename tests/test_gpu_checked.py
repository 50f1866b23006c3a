"""Checked mode (SISO_OPT_CHECKED): the library verifies on the device what it otherwise takes on trust - unit-norm
rows, numeric thresholds, 0/1 hit flags, slots of hits inside the cache - and reports a violation as
SISO_ERR_INVALID_ARG in the status word, never by a trap.  Tiny shapes that are no multiples of any tile size run
through every entry point under it with a clean status and the oracle's results."""
import numpy as np
import pytest
import torch

import oracle
from gen import workloads as W
from util import TOL, check_lookup, to_dev

pytestmark = pytest.mark.gpu

siso = pytest.importorskip("paper_2508_18736_b200")
INVALID = 1


@pytest.mark.parametrize("dtype,n,B,dim,k", [("bf16", 37, 5, 72, 3), ("f32", 3, 1, 8, 4), ("bf16", 301, 130, 264, 1), ("f32", 130, 33, 136, 8)])
def test_tiny_shapes_run_clean_under_checked_mode(dtype, n, B, dim, k):
    w = W.config(2 if dtype == "bf16" else 1, seed=5, mode="P", n_centroids=n, n_queries=B, dim=dim, n_clusters=max(2, n // 6),
                 dtype=dtype, theta=(0.80, 0.92), k=k)
    cap = n + B + 3
    cache = siso.SisoCache(cap, dim, dtype)
    cache.set_option(siso.OPT_CHECKED, 1)
    ora = oracle.OracleCache(cap, dim, dtype)
    cache.insert(to_dev(w.centroids, dtype))
    ora.insert(w.centroids)
    q, theta = to_dev(w.queries, dtype), torch.from_numpy(w.theta).cuda()
    for path in (siso.PATH_SIMT, siso.PATH_STREAM, siso.PATH_TENSOR, siso.PATH_AUTO):
        if path == siso.PATH_TENSOR and dtype == "f32" and k > 4:
            continue
        cache.set_lookup_path(path)
        got = [x.cpu().numpy() for x in cache.lookup(q, theta, k)]
        check_lookup(got, ora.lookup(w.queries, w.theta, k), ora.lookup_copy(), w.queries, w.theta, TOL[dtype], valid=ora.valid)
    idx, sim, hit = cache.lookup(q, theta, 1)
    cache.update(q, idx, hit)
    ora.update(w.queries, idx.cpu().numpy(), hit.cpu().numpy())
    out = [x.cpu().numpy() for x in cache.stream_step(q, theta)]
    ora.stream_step(w.queries, w.theta, forced=(out[0], out[2]))
    cache.merge(0.9, siso.MERGE_WEIGHTED_MEAN)
    ora.merge(0.9, True)
    free = cap - cache.stats()["occupancy"]
    if free >= 2:
        cache.merge(0.9, siso.MERGE_SIZES_ONLY, repo=q[:2].contiguous())
    assert (cache.evict(2).cpu().numpy() >= -1).all()
    cache.insert_misses(q, torch.ones(B, dtype=torch.uint8, device="cuda"))
    assert cache.sync_status() == 0, "a valid call tripped a check"
    cache.close()


def test_checked_mode_reports_what_the_unchecked_library_takes_on_trust():
    w = W.config(2, seed=6, mode="P", n_centroids=200, n_queries=64, dim=136, n_clusters=20)
    q = to_dev(w.queries, "bf16")
    bad_q = q.clone()
    bad_q[17] = bad_q[17] * 1.05                        # norm 1.05: outside the 1e-2 band
    nan_theta = torch.full((64,), 0.86, device="cuda")
    nan_theta[3] = float("nan")
    for checked in (0, 1):
        cache = siso.SisoCache(300, 136, "bf16")
        cache.set_option(siso.OPT_CHECKED, checked)
        want = INVALID if checked else 0
        cache.insert(to_dev(w.centroids, "bf16"))
        assert cache.sync_status() == 0
        cache.lookup(bad_q, 0.86, 2)
        assert cache.sync_status() == want and cache.sync_status() == 0         # reported once, then clear
        cache.lookup(q, nan_theta, 1)
        assert cache.sync_status() == want
        cache.insert((q[:4] * 0.5).contiguous())                                # half-length vectors
        assert cache.sync_status() == want
        idx, sim, hit = cache.lookup(q, 0.86, 1)
        assert cache.sync_status() == 0
        twos = torch.full_like(hit, 2)
        cache.insert_misses(q, twos)                                            # a hit flag that is neither 0 nor 1
        assert cache.sync_status() == want
        cache.stream_step(bad_q, 0.86)
        assert cache.sync_status() == want
        # an out-of-range slot of a hit is reported in either mode (the update looks the slot up), and skipped
        far = torch.full_like(idx, 10 ** 6)
        cache.update(q, far, torch.ones_like(hit))
        assert cache.sync_status() == INVALID
        # the handle is as usable as before
        got = [x.cpu().numpy() for x in cache.lookup(q, 0.86, 1)]
        assert cache.sync_status() == 0 and (got[0] >= 0).all()
        cache.close()
