"""Centroid-sharded lookup on one GPU: the shards are separate caches on the same device, their key lists are stacked
as an all-gather would deliver them, and the combined result must equal the oracle's lookup over the whole cache
(and the unsharded cache's), whatever the number of shards."""
import numpy as np
import pytest
import torch

import oracle
from gen import workloads as W
from util import TOL, check_lookup, to_dev, verify_merge_map

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


@pytest.mark.parametrize("dtype,total,dim,shards,batch,n_batches", [
    ("bf16", 301, 72, 3, 96, 14),         # ragged last shard (101 + 101 + 99); the cache fills up and evicts
    ("f32", 200, 64, 4, 130, 8),
    ("bf16", 5, 64, 8, 3, 6),             # more ranks than rows: ranks 5-7 hold nothing; one row per rank
])
def test_sharded_stream_equals_one_cache(dtype, total, dim, shards, batch, n_batches):
    """The owner-routed streaming step over several shards (driven in lockstep on one GPU, exchanges = stacks) against the
    oracle's step over ONE cache of the same global slots: lookup, victims, slots of the stored misses, and the whole state."""
    sp = W.StreamSpec(capacity=total, dim=dim, n_queries=batch * n_batches, batch=batch, n_clusters=max(8, 2 * total), zipf_s=1.1,
                      reshuffle_every=batch * 5, theta=0.80, mode="P", dtype=dtype, seed=61)
    stream = W.QueryStream(sp)
    parts = [siso.ShardedCache(total, dim, dtype, rank=r, world=shards) for r in range(shards)]
    ora = oracle.OracleCache(total, dim, dtype)
    evicted = 0
    for t in range(n_batches):
        qn, _ = stream.batch(t)
        theta = np.full(len(qn), sp.theta, np.float32)
        q = to_dev(qn, dtype)
        pre_copy, pre_valid = ora.lookup_copy(), ora.valid.copy()
        res = siso.run_lockstep([p.stream_steps(q, float(sp.theta)) for p in parts])
        for r in res[1:]:                                               # every rank holds the same answer
            assert all((a == b).all().item() for a, b in zip(res[0], r))
        idx, sim, hit, victims, slots = [x.cpu().numpy() for x in res[0]]
        o_idx, o_sim, o_hit, o_victims, o_slots = ora.stream_step(qn, theta, forced=(idx[:, None].astype(np.int32), hit))
        check_lookup((idx[:, None].astype(np.int32), sim[:, None], hit), (o_idx, o_sim, o_hit), pre_copy, qn, theta, TOL[dtype],
                     valid=pre_valid)
        nv = int((victims >= 0).sum())                                   # [batch]: eviction order, then -1
        assert len(victims) == len(qn) and (victims[nv:] == -1).all()
        assert (victims[:nv] == o_victims[:nv]).all() and nv == (o_victims >= 0).sum()
        assert (slots == o_slots).all()
        evicted += nv
        # the shards' states, laid side by side, are the one cache's state
        for p in parts:
            if p.hi == p.lo:
                assert p.local.stats()["occupancy"] == 0
                continue
            st = p.local.export()
            sl = slice(p.lo, p.hi)
            live = ora.valid[sl] == 1
            assert (st["valid"].cpu().numpy() == ora.valid[sl]).all()
            assert (st["size"].cpu().numpy()[live] == ora.size[sl][live]).all()
            assert (st["access"].cpu().numpy().view(np.uint32)[live] == ora.access[sl][live]).all()
            assert (st["last"].cpu().numpy().view(np.uint64)[live] == ora.last[sl][live]).all()
            assert np.abs(st["master"].cpu().numpy()[live] - ora.master[sl][live]).max(initial=0) <= 1e-6
    assert evicted > 0
    for p in parts:
        p.close()


def test_sharded_eviction_is_the_global_selection():
    """FilteringCentroids over shards: the victims are those of one cache, in the same order, with ties in cluster_size and
    access count that only last_access and the global slot break; also asking for more than a shard (or the cache) holds."""
    rng = np.random.default_rng(7)
    total, dim, shards = 900, 64, 4
    rows = rng.standard_normal((total, dim)).astype(np.float32)
    rows /= np.linalg.norm(rows, axis=1, keepdims=True)
    sizes = rng.integers(1, 4, total).astype(np.float64)              # many equal cluster sizes
    parts = [siso.ShardedCache(total, dim, "f32", rank=r, world=shards) for r in range(shards)]
    ora = oracle.OracleCache(total, dim, "f32")
    ora.insert(rows, sizes=sizes)
    for p in parts:
        p.local.insert(torch.from_numpy(rows[p.lo:p.hi]).cuda(), torch.from_numpy(sizes[p.lo:p.hi]).cuda())
    for m, decay in ((37, False), (300, True), (0, True), (700, False)):   # 300 > a shard's 225 rows; the last empties the cache
        res = siso.run_lockstep([p.evict_steps(m, siso.EVICT_DECAY if decay else 0) for p in parts])
        want = ora.evict(m, decay)
        got = res[0].cpu().numpy()
        assert all((r == res[0]).all().item() for r in res)
        live_before = len(want[want >= 0])
        assert (got[:live_before] == want[:live_before]).all() and (got[live_before:] == -1).all()
        for p in parts:
            st = p.local.export()
            sl = slice(p.lo, p.hi)
            live = ora.valid[sl] == 1
            assert (st["valid"].cpu().numpy() == ora.valid[sl]).all()
            assert (st["size"].cpu().numpy()[live] == ora.size[sl][live]).all()            # the decay reached every shard
            assert (st["access"].cpu().numpy().view(np.uint32)[live] == ora.access[sl][live]).all()
    assert sum(p.local.stats()["occupancy"] for p in parts) == 0 and sum(p.local.stats()["evictions"] for p in parts) == total
    for p in parts:
        p.close()


def test_world_of_one_through_the_distributed_driver():
    """Without a process group the torch.distributed driver (run) sees a world of one rank: the sharded step and the
    sharded eviction must then equal the plain cache's, bit for bit."""
    sp = W.StreamSpec(capacity=400, dim=64, n_queries=100 * 13, batch=100, n_clusters=900, zipf_s=1.1, reshuffle_every=500,
                      theta=0.80, mode="P", dtype="bf16", seed=62)
    stream = W.QueryStream(sp)
    one = siso.ShardedCache(400, 64, "bf16")
    plain = siso.SisoCache(400, 64, "bf16")
    for t in range(12):
        qn, _ = stream.batch(t)
        q = to_dev(qn, "bf16")
        idx, sim, hit, victims, slots = one.stream_step(q, float(sp.theta))
        p_idx, p_sim, p_hit, p_victims, p_slots = plain.stream_step(q, float(sp.theta))
        assert (idx.to(torch.int32) == p_idx[:, 0]).all().item() and (hit == p_hit).all().item()
        assert (sim == p_sim[:, 0]).all().item()
        assert victims.numel() == p_victims.numel() and (victims.to(torch.int32) == p_victims).all().item()
        assert (slots.to(torch.int32) == p_slots).all().item()
    a, b = one.local.export(), plain.export()
    assert all((a[k] == b[k]).all().item() for k in ("valid", "size", "access", "last", "master", "vecs"))
    assert one.local.stats()["evictions"] == plain.stats()["evictions"] > 0
    # the binding layer of a sharded step reads nothing back: misses, free slots and the eviction count stay on the device
    q = to_dev(stream.batch(12)[0], "bf16")
    torch.cuda.set_sync_debug_mode("error")
    try:
        res = one.stream_step(q, float(sp.theta))
    finally:
        torch.cuda.set_sync_debug_mode("default")
    p_res = plain.stream_step(q, float(sp.theta))
    assert (res[0].to(torch.int32) == p_res[0][:, 0]).all().item() and (res[3].to(torch.int32) == p_res[3]).all().item()
    v1 = one.evict(37, siso.EVICT_DECAY)
    v2 = plain.evict(37, siso.EVICT_DECAY)
    assert (v1.to(torch.int32) == v2).all().item()
    a, b = one.local.export(), plain.export()
    assert all((a[k] == b[k]).all().item() for k in ("valid", "size", "access"))
    one.close()
    plain.close()


@pytest.mark.parametrize("dtype,n,dim,shards,weighted,theta_c", [
    ("f32", 1500, 136, 3, True, 0.90),        # ragged last shard; an odd number of blocks
    ("f32", 1400, 72, 4, False, 0.86),        # an even number: the opposite blocks are swept by the lower rank only
    ("bf16", 2100, 264, 2, True, 0.90),
    ("f32", 900, 64, 8, True, 0.90),          # shards smaller than a tile of the sweep
    ("f32", 40, 64, 6, True, 0.90),           # more ranks than rows can fill: empty shards at the end
])
def test_sharded_merge_equals_one_cache(dtype, n, dim, shards, weighted, theta_c):
    """MergeCentroids over a partitioned cache, the blocks travelling round a ring: merge map, cluster sizes, live flags
    and vectors of every shard against the oracle's pass over the whole cache, pass after pass until nothing merges."""
    w = W.config(3, seed=17, mode="P", n_centroids=n, dim=dim, n_clusters=max(2, n // 18), sigma=0.06, dtype=dtype)
    sizes = np.random.default_rng(3).integers(1, 9, n).astype(np.float64)
    parts = [siso.ShardedCache(n, dim, dtype, rank=r, world=shards) for r in range(shards)]
    all_rows = to_dev(w.centroids, dtype)
    for p in parts:
        if p.hi > p.lo:
            p.local.insert(all_rows[p.lo:p.hi], torch.from_numpy(sizes[p.lo:p.hi]))
    ora = oracle.OracleCache(n, dim, dtype)
    ora.insert(w.centroids, sizes=sizes)
    flags = siso.MERGE_WEIGHTED_MEAN if weighted else siso.MERGE_SIZES_ONLY
    total_merged = 0
    for rounds in range(40):
        entry, valid0, sizes0 = ora.master.copy(), ora.valid.copy(), ora.size.copy()
        results = siso.run_lockstep([p.merge_steps(theta_c, flags) for p in parts])
        mm, n_merged = results[0][0].cpu().numpy(), results[0][1]
        for other, cnt in results[1:]:
            assert (other.cpu().numpy() == mm).all() and cnt == n_merged           # every rank holds the same map
        o_mm, o_n = ora.merge(theta_c, weighted)
        same = (mm == o_mm).all()
        if not same:       # only a decision within 1e-5 of the threshold or of the runner-up may differ
            verify_merge_map(entry, valid0, np.zeros(n, np.uint8), sizes0, mm, theta_c, tol=1e-5)
        else:
            assert n_merged == o_n
        total_merged += n_merged
        for p in parts:
            if p.hi == p.lo:
                continue
            st = p.local.export()
            torch.cuda.synchronize()
            lo, hi = p.lo, p.hi
            surv = mm[lo:hi] == np.arange(lo, hi)
            assert (st["valid"].cpu().numpy() == surv).all()
            if same:
                live = ora.valid[lo:hi] == 1
                assert (st["size"].cpu().numpy()[live] == ora.size[lo:hi][live]).all()
                assert np.abs(st["master"].cpu().numpy()[live] - ora.master[lo:hi][live]).max(initial=0) <= 1e-6
            assert p.local.stats()["occupancy"] == int(surv.sum())
            p.local.check_status()
        if not same or n_merged == 0:
            break
    assert total_merged > (n // 3 if n > 100 else 0)
    if same:
        assert n_merged == 0, "no fixed point within 40 passes"
    # the candidate buffer of a shard that is too small is reported, not overrun
    if n >= 900:
        fresh = [siso.ShardedCache(n, dim, dtype, rank=r, world=shards) for r in range(shards)]
        for p in fresh:
            if p.hi > p.lo:
                p.local.insert(all_rows[p.lo:p.hi])
        with pytest.raises(siso.SisoError) as e:
            siso.run_lockstep([p.merge_steps(theta_c, flags, cand_capacity=8) for p in fresh])
        assert e.value.status == 5
        for p in fresh:
            p.close()
    for p in parts:
        p.close()


def test_one_rank_nccl_group_runs_the_real_collectives():
    """A process group of ONE rank over NCCL on this GPU: the exchanges of the sharded operations then go through
    all_gather_into_tensor / all_reduce of the real backend (a ring step with one rank is a copy), and the results must
    equal the plain cache's bit for bit: lookup, streaming steps, a MergeCentroids pass."""
    import socket
    import torch.distributed as dist
    if dist.is_initialized():
        pytest.skip("a process group is already initialised in this process")
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    try:
        dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                                device_id=torch.device("cuda", torch.cuda.current_device()))
    except Exception as e:      # the environment, not the library under test: no NCCL group can be made on this machine
        pytest.skip(f"NCCL process group could not be created here: {e}")
    try:
        sp = W.StreamSpec(capacity=300, dim=128, n_queries=128 * 10, batch=128, n_clusters=1200, zipf_s=1.1, reshuffle_every=640,
                          theta=0.80, mode="P", dtype="bf16", seed=63)
        stream = W.QueryStream(sp)
        one = siso.ShardedCache(300, 128, "bf16")
        assert one.world == 1 and one.rank == 0
        plain = siso.SisoCache(300, 128, "bf16")
        for t in range(10):
            q = to_dev(stream.batch(t)[0], "bf16")
            a = one.stream_step(q, float(sp.theta))
            b = plain.stream_step(q, float(sp.theta))
            assert (a[0].to(torch.int32) == b[0][:, 0]).all().item() and (a[2] == b[2]).all().item()
            assert (a[3].to(torch.int32) == b[3]).all().item() and (a[4].to(torch.int32) == b[4]).all().item()
        q = to_dev(stream.batch(3)[0], "bf16")
        i1, s1, h1 = one.lookup(q, 0.8, 4)
        i2, s2, h2 = plain.lookup(q, 0.8, 4)
        assert (i1.to(torch.int32) == i2).all().item() and (s1 == s2).all().item() and (h1 == h2).all().item()
        mm1, n1 = one.merge(0.75, siso.MERGE_WEIGHTED_MEAN)
        mm2, n2 = plain.merge(0.75, siso.MERGE_WEIGHTED_MEAN)
        assert n1 == n2 and (mm1 == mm2[:300]).all().item()
        x, y = one.local.export(), plain.export()
        assert all((x[k] == y[k]).all().item() for k in ("valid", "size", "master", "vecs"))
        assert plain.stats()["evictions"] > 0
        one.close()
        plain.close()
    finally:
        dist.destroy_process_group()
