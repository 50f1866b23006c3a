"""Locality-ordered exact search (hot tier first, exact early exit, cold tier for the rest) against the oracle's plain
top-1 over the whole cache, and the hot tier's membership against the oracle's eviction order."""
import numpy as np
import pytest
import torch

import oracle
from gen import workloads as W
from util import TOL, check_lookup, to_dev, widen64

pytestmark = pytest.mark.gpu

siso = pytest.importorskip("paper_2508_18736_b200")


def merged_cache(dtype, n, n_clusters, dim, theta_c, seed):
    """A cache after the usual life cycle: centroids inserted, one batch of hits folded in (so cluster_size and access
    counts differ), then MergeCentroids at theta_c: every pair of survivors is at most theta_c similar."""
    w = W.config(4 if dtype == "bf16" else 1, seed=seed, mode="T", n_centroids=n, n_queries=2000, dim=dim, n_clusters=n_clusters,
                 sigma=0.07, dtype=dtype, zipf_s=1.0, ood_fraction=0.2, theta=(0.78, 0.93), k=1)
    cache = siso.SisoCache(n, dim, dtype)
    cache.insert(to_dev(w.centroids, dtype))
    q = to_dev(w.queries, dtype)
    idx, sim, hit = cache.lookup(q, torch.from_numpy(w.theta).cuda(), 1)
    cache.update(q, idx, hit)
    cache.merge(theta_c, siso.MERGE_WEIGHTED_MEAN)
    cache.check_status()
    return cache, w


def oracle_of(cache, dtype):
    st = cache.export()
    torch.cuda.synchronize()
    ora = oracle.OracleCache(cache.capacity, cache.dim, dtype)
    ora.load_state(st["master"].cpu().numpy(), st["size"].cpu().numpy(), st["access"].cpu().numpy().view(np.uint32),
                   st["last"].cpu().numpy().view(np.uint64), st["valid"].cpu().numpy(), cache.stats()["clock"])
    return ora


@pytest.mark.parametrize("dtype,n,n_clusters,dim,hot", [
    ("bf16", 4000, 1000, 136, 120),
    ("f32", 2500, 600, 72, 64),
    ("bf16", 1500, 300, 264, 1),          # a hot tier of one entry
])
def test_tiered_lookup_equals_whole_cache(dtype, n, n_clusters, dim, hot):
    theta_c = 0.86
    cache, w = merged_cache(dtype, n, n_clusters, dim, theta_c, seed=51)
    ora = oracle_of(cache, dtype)
    stored, live = ora.lookup_copy(), ora.valid == 1
    occ = int(live.sum())
    assert 0.5 * n_clusters < occ < 1.2 * n_clusters
    # the precondition of the exit, checked on the stored vectors themselves: separation and norms
    S = widen64(stored[live]) @ widen64(stored[live]).T
    np.fill_diagonal(S, -1)
    w2 = W.config(4 if dtype == "bf16" else 1, seed=51, query_seed=52, mode="T", n_centroids=n, n_queries=700, dim=dim,
                  n_clusters=n_clusters, sigma=0.07, dtype=dtype, zipf_s=1.0, ood_fraction=0.2, theta=(0.78, 0.93), k=1)
    norms = np.concatenate([np.linalg.norm(widen64(stored[live]), axis=1), np.linalg.norm(widen64(w2.queries), axis=1)])
    slack = float(np.abs(norms - 1).max()) * 1.01 + 1e-7
    sep = float(S.max()) + 1e-9
    assert sep <= theta_c + (4e-3 if dtype == "bf16" else 1e-6) and slack < (4e-3 if dtype == "bf16" else 1e-5)

    # the library measures the entries' side of that bound itself, and refuses a slack the entries do not meet
    ent = float(np.abs(np.linalg.norm(widen64(stored[live]), axis=1) - 1).max())
    dev = cache.norm_deviation()
    assert ent <= dev <= ent * (1 + 1e-6) + 1e-12
    with pytest.raises(ValueError):
        siso.TieredCache(cache, hot, sep, 0.5 * dev)
    tiers = siso.TieredCache(cache, hot, sep, slack)
    # hot tier = what FilteringCentroids keeps when told to leave `hot` entries
    cold = np.sort(ora.evict(occ - hot))
    ora = oracle_of(cache, dtype)                                         # evict changed the oracle copy: take it again
    assert (tiers.cold_slot.cpu().numpy() == cold).all()
    assert (tiers.hot_slot.cpu().numpy() == np.setdiff1d(np.flatnonzero(live), cold)).all()
    assert tiers.n_hot == hot and tiers.n_cold == occ - hot

    q, theta = to_dev(w2.queries, dtype), torch.from_numpy(w2.theta).cuda()
    idx, sim, hit = [x.cpu().numpy() for x in tiers.lookup(q, theta)]
    o = ora.lookup(w2.queries, w2.theta, 1)
    check_lookup((idx[:, None], sim[:, None], hit), o, stored, w2.queries, w2.theta, TOL[dtype], valid=ora.valid)
    f_idx, f_sim, f_hit = [x.cpu().numpy() for x in cache.lookup(q, theta, 1)]
    assert (f_idx[:, 0] == idx).all() and (f_hit == hit).all() and np.abs(f_sim[:, 0] - sim).max() <= 2e-6
    # some queries ended in the hot tier, some went on; every one that ended there really has its best match there
    assert (0 < tiers.settled < 700) or hot == 1
    exit_sim = tiers.exit_sim
    assert abs(exit_sim - siso.tier_exit_sim(sep, slack)) == 0 and exit_sim > np.sqrt((1 + sep) / 2)
    hot_set = set(tiers.hot_slot.cpu().numpy().tolist())
    ended = np.array([i in hot_set for i in idx]) & (sim > exit_sim)
    assert ended.sum() == tiers.settled
    # the degenerate splits and an exit that never fires give the same answers
    for hot_rows, s in ((0, sep), (occ + 5, sep), (hot, 1.0)):
        t2 = siso.TieredCache(cache, hot_rows, s, slack)
        i2, s2, h2 = [x.cpu().numpy() for x in t2.lookup(q, theta)]
        assert (i2 == idx).all() and (h2 == hit).all() and np.abs(s2 - sim).max() <= 2e-6
        assert t2.settled == 0 or hot_rows > occ
        t2.close()
    tiers.close()
    cache.close()


def test_tier_kernels_on_hand_made_keys():
    """select / finish on keys written by hand: ordering of the packed rows, empty tiers, ties to the lower slot."""
    def key(sim, slot):
        u = int(np.float32(sim).view(np.uint32))
        u = (~u & 0xFFFFFFFF) if u & 0x80000000 else (u | 0x80000000)
        return np.uint64((u << 32) | (0xFFFFFFFF - slot))
    hot = np.array([key(0.99, 2), 0, key(0.5, 0), key(0.97, 1), key(0.9, 1)], dtype=np.uint64)
    hk = torch.from_numpy(hot.view(np.int64)).cuda()
    q = torch.arange(5 * 8, dtype=torch.float32, device="cuda").reshape(5, 8)
    rows, packed, count = siso.tier_select(hk, q, 0.95)
    assert int(count.item()) == 3 and rows[:3].cpu().tolist() == [1, 2, 4]
    assert (packed[:3] == q[[1, 2, 4]]).all().item()
    hot_slot = torch.tensor([10, 20, 30], dtype=torch.int32, device="cuda")
    cold_slot = torch.tensor([5, 25], dtype=torch.int32, device="cuda")
    cold = np.array([key(0.3, 1), key(0.5, 0), 0], dtype=np.uint64)       # for rows 1, 2, 4
    ck = torch.from_numpy(cold.view(np.int64)).cuda()
    idx, sim, hit = siso.tier_finish(hk, 0.95, ck, rows, 3, hot_slot, cold_slot, 0.4)
    assert idx.cpu().tolist() == [30, 25, 5, 20, 20]        # row 2: equal similarity 0.5, slot 5 (cold) < slot 10 (hot)
    assert np.allclose(sim.cpu().numpy(), [0.99, 0.3, 0.5, 0.97, 0.9]) and hit.cpu().tolist() == [1, 0, 1, 1, 1]
    # nothing anywhere: -1, -inf, miss
    z = torch.zeros(4, dtype=torch.int64, device="cuda")
    rows, packed, count = siso.tier_select(z, q[:4], 0.95)
    assert int(count.item()) == 4
    idx, sim, hit = siso.tier_finish(z, 0.95, z, rows, 4, None, None, -1.0)
    assert (idx == -1).all().item() and torch.isneginf(sim).all().item() and (hit == 0).all().item()
    with pytest.raises(siso.SisoError):
        siso.tier_select(z, torch.zeros(4, 3, dtype=torch.float32, device="cuda"), 0.5)     # rows of 12 bytes
