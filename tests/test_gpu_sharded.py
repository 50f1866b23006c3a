"""Centroid-sharded lookup on one GPU: the shards are separate caches on the same device, their key lists are stacked
as an all-gather would deliver them, and the combined result must equal the oracle's lookup over the whole cache
(and the unsharded cache's), whatever the number of shards."""
import numpy as np
import pytest
import torch

import oracle
from gen import workloads as W
from util import TOL, check_lookup, to_dev

pytestmark = pytest.mark.gpu

siso = pytest.importorskip("paper_2508_18736_b200")


@pytest.mark.parametrize("dtype,n,dim,B,k,shards", [
    ("bf16", 3000, 136, 300, 4, 3),       # ragged last shard
    ("bf16", 2048, 64, 40, 1, 8),
    ("f32", 700, 72, 130, 8, 2),
])
def test_sharded_lookup_equals_whole_cache(dtype, n, dim, B, k, shards):
    w = W.config(4 if dtype == "bf16" else 1, seed=41, mode="P", n_centroids=n, n_queries=B, dim=dim, n_clusters=max(2, n // 16),
                 dtype=dtype, theta=(0.78, 0.93), k=k)
    q, theta = to_dev(w.queries, dtype), torch.from_numpy(w.theta).cuda()
    parts = [siso.ShardedCache(n, dim, dtype, rank=r, world=shards) for r in range(shards)]
    all_rows = to_dev(w.centroids, dtype)
    for p in parts:
        p.fill(all_rows)
    assert [p.lo for p in parts] == [min(n, r * siso.shard_rows(n, shards)) for r in range(shards)]
    keys = torch.stack([p.local.lookup_keys(q, k, slot_offset=p.lo) for p in parts], dim=1)        # [B, shards, k]
    idx, sim, hit = siso.combine_keys(keys, theta)
    o = oracle.lookup(w.centroids, w.queries, w.theta, k)
    got = (idx.cpu().numpy().astype(np.int32), sim.cpu().numpy(), hit.cpu().numpy())
    check_lookup(got, o, w.centroids, w.queries, w.theta, TOL[dtype])
    # the same bits as one cache holding everything: the kernels accumulate alike and the keys order alike
    whole = siso.SisoCache(n, dim, dtype)
    whole.insert(all_rows)
    w_idx, w_sim, w_hit = whole.lookup(q, theta, k)
    assert (w_idx.cpu().numpy() == got[0]).all() and (w_hit.cpu().numpy() == got[2]).all()
    assert np.abs(w_sim.cpu().numpy() - got[1]).max() <= 2e-6
    # a single process without a process group is a world of one
    one = siso.ShardedCache(n, dim, dtype)
    one.fill(all_rows)
    i1, s1, h1 = one.lookup(q, theta, k)
    assert (i1.cpu().numpy() == got[0]).all() and (h1.cpu().numpy() == got[2]).all()
    for c in parts + [one]:
        c.close()
    whole.close()


def test_keys_of_an_empty_or_small_shard_and_bad_arguments():
    w = W.config(4, seed=42, mode="P", n_centroids=3, n_queries=5, dim=64, n_clusters=2)
    c = siso.SisoCache(8, 64, "bf16")
    keys = c.lookup_keys(to_dev(w.queries, "bf16"), 4, slot_offset=100)
    assert (keys.cpu().numpy() == 0).all()                                     # empty shard: no entries
    c.insert(to_dev(w.centroids, "bf16"))
    keys = c.lookup_keys(to_dev(w.queries, "bf16"), 4, slot_offset=100)
    idx, sim, hit = siso.combine_keys(keys.unsqueeze(1), -1.0)
    idx = idx.cpu().numpy()
    assert ((idx[:, :3] >= 100) & (idx[:, :3] < 103)).all() and (idx[:, 3] == -1).all() and hit.cpu().numpy().all()
    assert np.isneginf(sim.cpu().numpy()[:, 3]).all()
    with pytest.raises(siso.SisoError):
        c.lookup_keys(to_dev(w.queries, "bf16"), 4, slot_offset=(1 << 32))      # global slots are 32-bit
    c.close()
