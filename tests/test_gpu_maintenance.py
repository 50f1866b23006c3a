"""GPU parity of update, merge, evict, insert and the streaming step against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from gen import workloads as W
from util import TOL, check_lookup, to_dev, verify_merge_map, widen64

pytestmark = pytest.mark.gpu

siso = pytest.importorskip("paper_2508_18736_b200")
VEC_TOL = {"f32": 1e-6, "bf16": 2.5e-4}       # max-abs on vector elements (1 ulp of bf16 at 1/sqrt(D) magnitudes)



# the pairwise sweep of a merge: CUDA cores, or tensor cores as a filter (one bf16 product, or three bf16 parts) + exact check
SWEEPS = [pytest.param((siso.PATH_SIMT, 1), id="cuda-cores"), pytest.param((siso.PATH_TENSOR, 1), id="tensor-one-part"),
          pytest.param((siso.PATH_TENSOR, 3), id="tensor-three-parts")]


def set_sweep(cache, sweep):
    cache.set_option(siso.OPT_MERGE_PATH, sweep[0])
    cache.set_option(siso.OPT_MERGE_SWEEP_PARTS, sweep[1])


def state_np(cache):
    st = cache.export()
    torch.cuda.synchronize()
    return dict(vecs=(st["vecs"].view(torch.int16).cpu().numpy().view(np.uint16) if cache.dtype == "bf16"
                      else st["vecs"].cpu().numpy()),
                master=st["master"].cpu().numpy(), size=st["size"].cpu().numpy(),
                access=st["access"].cpu().numpy().view(np.uint32), last=st["last"].cpu().numpy().view(np.uint64),
                valid=st["valid"].cpu().numpy())


def assert_state_equal(cache, ora, dtype, what=""):
    g = state_np(cache)
    assert (g["valid"] == ora.valid).all(), what
    live = ora.valid == 1
    np.testing.assert_array_equal(g["size"][live], ora.size[live], err_msg=what)      # fp64 on both sides: exact
    np.testing.assert_array_equal(g["access"][live], ora.access[live], err_msg=what)
    np.testing.assert_array_equal(g["last"][live], ora.last[live], err_msg=what)
    assert np.abs(g["master"][live].astype(np.float64) - ora.master[live]).max(initial=0) <= 1e-6, what
    gm = g["master"][live].astype(np.float64)
    cosine = np.einsum("ij,ij->i", gm, ora.master[live]) / (np.linalg.norm(gm, axis=1) * np.linalg.norm(ora.master[live], axis=1))
    assert (cosine >= 1 - 1e-6).all(), what
    a, b = widen64(g["vecs"][live]), widen64(ora.lookup_copy()[live])
    if dtype == "bf16":
        # the GPU rounds its fp32 master, the oracle its fp64 master: where the master lies within 1e-6 of a rounding
        # boundary the two copies are neighbours, so the bound is one bf16 ulp of the value (2.5e-4 is that ulp below
        # 0.125) and such elements are few
        ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(b), 1e-30))) - 7)
        assert (np.abs(a - b) <= np.maximum(ulp, VEC_TOL[dtype])).all() and (a != b).sum() <= 0.01 * a.size, what
    else:
        assert np.abs(a - b).max(initial=0) <= VEC_TOL[dtype], what
    if dtype == "bf16":   # the lookup copy is the master rounded once
        m = torch.from_numpy(g["master"]).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        assert (m[live] == g["vecs"][live]).all(), what
    assert cache.stats()["occupancy"] == int(live.sum()) and cache.stats()["clock"] == ora.clock, what


def adopt_gpu_merge(cache, ora, mm, entry, valid0, seed, sizes0, theta_c, weighted, what):
    """The GPU's merge map differs from the oracle's.  That is accepted only if the map is a valid outcome of
    Algorithm 1 with every comparison within 1e-5 of the oracle's (a decision at the threshold or between two
    equally close survivors, and what follows from it); the applied state is then checked against that map's own
    closed form, and the oracle carries on from the GPU's state."""
    size = verify_merge_map(entry, valid0, seed, sizes0, mm, theta_c, tol=1e-5)
    g = state_np(cache)
    surv = (mm == np.arange(len(mm)))
    assert (g["valid"] == surv).all(), what
    np.testing.assert_array_equal(g["size"][surv], size[surv], err_msg=what)
    for s in np.flatnonzero(surv):
        members = np.flatnonzero(mm == s)
        if weighted and len(members) > 1:
            v = (sizes0[members, None] * entry[members]).sum(0)
            assert np.abs(g["master"][s] - v / np.linalg.norm(v)).max() <= 1e-6, what
        else:
            assert np.abs(g["master"][s] - entry[s]).max() <= 1e-6, what
    ora.load_state(g["master"], g["size"], g["access"], g["last"], g["valid"], ora.clock)


def dataclass_slice(w, lo, hi):
    """The workload with only rows lo..hi of its centroids."""
    import dataclasses
    return dataclasses.replace(w, centroids=w.centroids[lo:hi], centroid_labels=w.centroid_labels[lo:hi])


def make_pair(w, capacity=None, sizes=None):
    cap = capacity or w.centroids.shape[0]
    cache = siso.SisoCache(cap, w.dim, w.dtype)
    slots = cache.insert(to_dev(w.centroids, w.dtype), None if sizes is None else torch.from_numpy(sizes))
    ora = oracle.OracleCache(cap, w.dim, w.dtype)
    o_slots = ora.insert(w.centroids, sizes=sizes)
    assert (slots.cpu().numpy() == o_slots).all()
    return cache, ora


@pytest.mark.parametrize("cfg,over,mode", [
    (2, dict(n_centroids=2048, n_queries=4096, dim=768, n_clusters=64), "T"),        # radix-sort grouping, hot rows
    (2, dict(n_centroids=500, n_queries=300, dim=136, n_clusters=40), "P"),          # single-CTA grouping
    (1, dict(n_centroids=700, n_queries=2500, dim=384, n_clusters=32), "T"),         # fp32 cache
    (4, dict(n_centroids=900, n_queries=3000, dim=1024, n_clusters=24), "T"),        # widest row of the warp-per-position kernel
    (2, dict(n_centroids=600, n_queries=1500, dim=264, n_clusters=20), "T"),         # dim not a multiple of 128: CTA-per-position kernel
    (1, dict(n_centroids=800, n_queries=2000, dim=1024, n_clusters=20), "T"),        # fp32 rows of 4 KiB in the warp kernel
    (2, dict(n_centroids=40, n_queries=6000, dim=128, n_clusters=4), "T"),           # a few centroids take over a thousand hits each: runs of chunks
])
def test_update_matches_oracle(cfg, over, mode):
    w = W.config(cfg, mode=mode, **over)
    sizes = (np.random.default_rng(5).integers(1, 50, w.centroids.shape[0]) / 1.1).astype(np.float64)
    cache, ora = make_pair(w, sizes=sizes)
    assert_state_equal(cache, ora, w.dtype, "after insert")
    q = to_dev(w.queries, w.dtype)
    for rep in range(2):
        idx, sim, hit = cache.lookup(q, torch.from_numpy(w.theta).cuda(), 1)
        o = ora.lookup(w.queries, w.theta, 1)
        check_lookup((idx.cpu().numpy(), sim.cpu().numpy(), hit.cpu().numpy()), o, ora.lookup_copy(), w.queries,
                     w.theta, TOL[w.dtype])
        assert hit.sum().item() > 0.3 * len(w.theta) or mode != "T"
        cache.update(q, idx, hit)
        ora.update(w.queries, idx.cpu().numpy(), hit.cpu().numpy())       # the oracle takes the GPU's decisions
        assert_state_equal(cache, ora, w.dtype, f"after update {rep}")
    cache.check_status()
    # determinism: the same update on a fresh cache gives the same bits
    a = state_np(cache)["master"]
    cache2, _ = make_pair(w, sizes=sizes)
    for rep in range(2):
        idx, sim, hit = cache2.lookup(q, torch.from_numpy(w.theta).cuda(), 1)
        cache2.update(q, idx, hit)
    assert (state_np(cache2)["master"] == a).all()
    # access_count saturates at infinity: entries inserted with infinity stay there
    assert (state_np(cache)["access"][ora.valid == 1] == siso.ACCESS_INF).all()


def test_update_counts_accesses_after_decay_reset():
    w = W.config(2, n_centroids=256, n_queries=512, dim=64, n_clusters=16)
    cache, ora = make_pair(w)
    cache.evict(0, siso.EVICT_DECAY)
    ora.evict(0, decay=True)
    q = to_dev(w.queries, w.dtype)
    idx, sim, hit = cache.lookup(q, 0.5, 1)
    cache.update(q, idx, hit)
    ora.update(w.queries, idx.cpu().numpy(), hit.cpu().numpy())
    assert_state_equal(cache, ora, w.dtype)
    assert state_np(cache)["access"].max() > 1


@pytest.mark.parametrize("dtype,mode,theta_c,weighted", [
    ("f32", "T", 0.90, True), ("f32", "P", 0.90, True), ("f32", "P", 0.86, False), ("bf16", "P", 0.90, True),
])
@pytest.mark.parametrize("sweep", SWEEPS)
def test_self_merge_matches_oracle(dtype, mode, theta_c, weighted, sweep):
    w = W.config(3, n_centroids=1500, dim=136, n_clusters=90, mode=mode, sigma=0.06, dtype=dtype)
    sizes = np.random.default_rng(9).integers(1, 9, 1500).astype(np.float64)
    cache, ora = make_pair(w, capacity=1536, sizes=sizes)
    set_sweep(cache, sweep)
    entry = ora.master.copy()
    flags = siso.MERGE_WEIGHTED_MEAN if weighted else siso.MERGE_SIZES_ONLY
    for rounds in range(40):
        before = state_np(cache)
        mm, n = cache.merge(theta_c, flags)
        o_mm, o_n = ora.merge(theta_c, weighted)
        mm = mm.cpu().numpy()
        if not (mm == o_mm).all():
            adopt_gpu_merge(cache, ora, mm, before["master"].astype(np.float64), before["valid"],
                            np.zeros(len(mm), np.uint8), before["size"], theta_c, weighted, f"merge pass {rounds}")
            o_n = int((mm[mm >= 0] != np.flatnonzero(mm >= 0)).sum())
        assert n == o_n
        assert_state_equal(cache, ora, dtype, f"merge pass {rounds}")
        if rounds == 0:
            assert n > 100
            if not weighted:
                live = ora.valid == 1
                assert (state_np(cache)["master"][live].astype(np.float64) == entry[live]).all()
        if n == 0:
            break
    assert n == 0, "no fixed point within 40 passes"
    g = state_np(cache)
    live = np.flatnonzero(g["valid"])
    if weighted:
        S = g["master"][live].astype(np.float64) @ g["master"][live].astype(np.float64).T
        np.fill_diagonal(S, -1)
        assert S.max() <= theta_c + 1e-6           # at the fixed point no two survivors exceed the threshold
    assert abs(g["size"][live].sum() - sizes.sum()) < 1e-9
    cache.check_status()


@pytest.mark.parametrize("sweep", SWEEPS)
def test_merge_keeps_pairs_whose_bf16_products_fall_below_the_threshold(sweep):
    """Rows of +-1/sqrt(232): that magnitude loses 0.34 % when rounded to bf16 (nearly the worst case, 2^-8), so the
    product of the ROUNDED rows of a planted pair lies 6e-3 below the exact similarity.  theta_C sits 1e-4 under the
    exact similarity, so the pair merges (the oracle says so); a tensor-core filter must keep it for the exact check."""
    N, D, flips = 4096, 232, 11
    rng = np.random.default_rng(77)
    m = np.float32(1.0 / np.sqrt(D))
    rows = np.where(rng.random((N, D)) < 0.5, -m, m).astype(np.float32)
    planted = 48
    for p in range(planted):
        a, b = 40 * p + 3, 40 * p + 29
        rows[b] = rows[a]
        rows[b, rng.choice(D, flips, replace=False)] *= -1
    exact = float(rows[3].astype(np.float64) @ rows[29].astype(np.float64))
    rounded = torch.from_numpy(rows[[3, 29]]).to(torch.bfloat16).to(torch.float64)
    assert exact - float(rounded[0] @ rounded[1]) > 5e-3            # far outside a margin meant for fp32 rounding
    theta_c = float(np.float32(exact - 1e-4))
    cache = siso.SisoCache(N, D, "f32")
    set_sweep(cache, sweep)
    cache.insert(torch.from_numpy(rows).cuda())
    ora = oracle.OracleCache(N, D, "f32")
    ora.insert(rows)
    mm, n = cache.merge(theta_c, siso.MERGE_WEIGHTED_MEAN)
    o_mm, o_n = ora.merge(theta_c, True)
    assert o_n == planted and n == o_n
    assert (mm.cpu().numpy() == o_mm).all()
    assert_state_equal(cache, ora, "f32", "planted pairs")
    cache.check_status()


@pytest.mark.parametrize("sweep", SWEEPS)
def test_merge_extremes_holes_and_overflow(sweep):
    w = W.config(3, n_centroids=700, dim=64, n_clusters=30, mode="P")
    cache, ora = make_pair(w, capacity=1000)
    set_sweep(cache, sweep)
    victims = cache.evict(50).cpu().numpy()
    assert (victims == ora.evict(50)).all()
    mm, n = cache.merge(1.0, siso.MERGE_WEIGHTED_MEAN)
    assert n == 0 and (mm.cpu().numpy() == ora.merge(1.0, True)[0]).all()
    cache.set_option(2, 1000)                       # a candidate buffer that cannot hold the pairs
    before = state_np(cache)
    with pytest.raises(siso.SisoError) as e:
        cache.merge(-1.0, siso.MERGE_SIZES_ONLY)
    assert e.value.status == 5
    after = state_np(cache)
    assert all((before[k] == after[k]).all() for k in before)
    cache.set_option(2, 400000)
    mm, n = cache.merge(-1.0, siso.MERGE_SIZES_ONLY)
    o_mm, o_n = ora.merge(-1.0, False)
    assert n == o_n == 649 and (mm.cpu().numpy() == o_mm).all()
    assert_state_equal(cache, ora, "f32")
    cache.close()


@pytest.mark.parametrize("dtype,weighted", [("f32", True), ("bf16", False)])
@pytest.mark.parametrize("sweep", SWEEPS)
def test_two_set_merge_matches_oracle(dtype, weighted, sweep):
    """Algorithm 1 as printed: C_cur = the cache, C_repo = new rows; holes in the cache interleave the two."""
    w = W.config(3, n_centroids=1400, dim=136, n_clusters=80, mode="P", sigma=0.06, dtype=dtype)
    cur, repo = w.centroids[:800], w.centroids[800:]
    rng = np.random.default_rng(4)
    cur_sizes = rng.integers(1, 9, 800).astype(np.float64)
    repo_sizes = rng.integers(1, 5, 600).astype(np.float64)
    cap = 1500
    cache = siso.SisoCache(cap, w.dim, dtype)
    set_sweep(cache, sweep)
    ora = oracle.OracleCache(cap, w.dim, dtype)
    cache.insert(to_dev(cur, dtype), torch.from_numpy(cur_sizes))
    ora.insert(cur, sizes=cur_sizes)
    assert (cache.evict(90).cpu().numpy() == ora.evict(90)).all()           # punch holes below the live entries
    cache.evict(0, siso.EVICT_DECAY)
    ora.evict(0, decay=True)                                                  # access_count of C_cur becomes finite
    seed = ora.valid.copy()
    flags = siso.MERGE_WEIGHTED_MEAN if weighted else siso.MERGE_SIZES_ONLY
    before = state_np(cache)
    # not enough room: nothing changes
    with pytest.raises(siso.SisoError) as e:
        cache.merge(0.9, flags, repo=to_dev(w.centroids[:cap], dtype)[: cap - 700])
    assert e.value.status == 4
    after = state_np(cache)
    assert all((before[k] == after[k]).all() for k in before) and cache.stats()["occupancy"] == 710
    # candidate buffer too small: the inserted rows are taken out again
    cache.set_option(2, 50)
    with pytest.raises(siso.SisoError) as e:
        cache.merge(0.9, flags, repo=to_dev(repo, dtype), repo_sizes=torch.from_numpy(repo_sizes))
    assert e.value.status == 5
    after = state_np(cache)
    assert (before["valid"] == after["valid"]).all() and cache.stats()["occupancy"] == 710
    cache.set_option(2, 200000)
    mm, n = cache.merge(0.9, flags, repo=to_dev(repo, dtype), repo_sizes=torch.from_numpy(repo_sizes))
    ora.insert(repo, sizes=repo_sizes)
    entry, valid0, sizes0 = ora.master.copy(), ora.valid.copy(), ora.size.copy()
    o_mm, o_n = ora.merge(0.9, weighted, seed_mask=seed, new_access_inf=True)
    mm = mm.cpu().numpy()
    if not (mm == o_mm).all():
        adopt_gpu_merge(cache, ora, mm, entry, valid0, seed, sizes0, 0.9, weighted, "two-set merge")
        o_n = int((mm[mm >= 0] != np.flatnonzero(mm >= 0)).sum())
    assert n == o_n and n > 100
    assert_state_equal(cache, ora, dtype, "two-set merge")
    live = ora.valid == 1
    assert (mm[seed == 1] == np.flatnonzero(seed == 1)).all()                 # C_cur is never merged away
    new_surv = live & (seed == 0)
    assert (state_np(cache)["access"][new_surv] == siso.ACCESS_INF).all()
    # FilteringCentroids back to the capacity M of Algorithm 1, then the decay
    m = int(live.sum()) - 900
    assert m > 0 and (cache.evict(m, siso.EVICT_DECAY).cpu().numpy() == ora.evict(m, decay=True)).all()
    assert_state_equal(cache, ora, dtype, "after filtering")
    cache.check_status()
    cache.close()


@pytest.mark.parametrize("capacity,n,m", [(700, 650, 37), (5000, 5000, 300), (70000, 66000, 1), (70000, 66000, 4000),
                                          (3000, 40, 40)])
def test_evict_order_matches_oracle(capacity, n, m):
    rng = np.random.default_rng(capacity + m)
    dim = 8
    vec = np.zeros((n, dim), dtype=np.float32)
    vec[:, 0] = 1
    sizes = rng.choice([1.0, 1.0, 1.0, 2.0, 3.0, 1 / 1.1, 2 / 1.1, 5.0], n)
    cache = siso.SisoCache(capacity, dim, "f32")
    cache.insert(torch.from_numpy(vec).cuda(), torch.from_numpy(sizes))
    ora = oracle.OracleCache(capacity, dim, "f32")
    ora.insert(vec, sizes=sizes)
    # vary access_count and last_access through the public path: a few update rounds on random subsets
    for r in range(3):
        rows = rng.choice(n, n // 3, replace=False).astype(np.int32)
        if r == 0:
            cache.evict(0, siso.EVICT_DECAY)
            ora.evict(0, decay=True)
        q = torch.from_numpy(vec[: len(rows)]).cuda()
        idx = torch.from_numpy(rows).cuda()
        hit = torch.ones(len(rows), dtype=torch.uint8, device="cuda")
        cache.update(q, idx, hit)
        ora.update(vec[: len(rows)], rows, np.ones(len(rows), dtype=np.uint8))
    got = cache.evict(m, siso.EVICT_DECAY).cpu().numpy()
    want = ora.evict(m, decay=True)
    assert (got == want).all()
    assert_state_equal(cache, ora, "f32")
    # evicting more than there is pads with -1 and empties the cache
    left = int(ora.valid.sum())
    got = cache.evict(left + 5).cpu().numpy()
    want = ora.evict(left + 5)
    assert (got == want).all() and cache.stats()["occupancy"] == 0
    cache.check_status()


def test_insert_misses_and_capacity_error():
    w = W.config(2, n_centroids=100, n_queries=64, dim=64, n_clusters=10)
    cache, ora = make_pair(w, capacity=140)
    cache.evict(7)
    ora.evict(7)
    q = to_dev(w.queries, w.dtype)
    hit = (np.random.default_rng(0).random(64) < 0.5).astype(np.uint8)
    hit[:20] = 0
    slots = cache.insert_misses(q, torch.from_numpy(hit).cuda()).cpu().numpy()
    assert (slots == ora.insert(w.queries, hit)).all()
    assert_state_equal(cache, ora, w.dtype)
    n_free = 140 - int(ora.valid.sum())
    before = state_np(cache)
    slots = cache.insert_misses(q, torch.zeros(64, dtype=torch.uint8, device="cuda")).cpu().numpy()
    assert n_free < 64 and (slots == -1).all() and cache.sync_status() == 4
    after = state_np(cache)
    assert all((before[k] == after[k]).all() for k in before)


@pytest.mark.parametrize("theta_mode,dtype,batch,capacity,dim,n_batches,n_clusters", [
    ("fixed", "bf16", 256, 1024, 128, 60, 400), ("per_query", "bf16", 256, 1024, 128, 60, 400),
    ("fixed", "f32", 256, 1024, 128, 60, 400),
    ("fixed", "bf16", 100, 1024, 128, 60, 400),           # 100: a batch that is padded to a query tile
    ("fixed", "bf16", 256, 4096, 768, 782, 1024),         # the scaled twin of the streaming configuration: 200,000 queries
])
def test_streaming_step_lockstep_on_a_scaled_twin(theta_mode, dtype, batch, capacity, dim, n_batches, n_clusters):
    n_queries = 200_000 if n_batches == 782 else batch * n_batches
    sp = W.StreamSpec(capacity=capacity, dim=dim, n_queries=n_queries, batch=batch, n_clusters=n_clusters, zipf_s=1.2,
                      reshuffle_every=n_queries // 2, theta=0.86, mode="P", dtype=dtype)
    st = W.QueryStream(sp)
    cache = siso.SisoCache(sp.capacity, sp.dim, dtype)
    ora = oracle.OracleCache(sp.capacity, sp.dim, dtype)
    rng = np.random.default_rng(2)
    evictions = 0
    for t, q, _ in st.batches():
        theta = np.full(len(q), sp.theta, np.float32) if theta_mode == "fixed" else rng.uniform(0.80, 0.92, len(q)).astype(np.float32)
        th = float(sp.theta) if theta_mode == "fixed" else torch.from_numpy(theta).cuda()
        idx, sim, hit, victims, slots = [x.cpu().numpy() for x in cache.stream_step(to_dev(q, dtype), th)]
        pre_copy, pre_valid = ora.lookup_copy(), ora.valid.copy()
        o_idx, o_sim, o_hit, o_victims, o_slots = ora.stream_step(q, theta, forced=(idx, hit))
        check_lookup((idx, sim, hit), (o_idx, o_sim, o_hit), pre_copy, q, theta, TOL[dtype], valid=pre_valid)
        nv = len(o_victims)
        assert (victims[:nv] == o_victims).all() and (victims[nv:] == -1).all(), f"batch {t}"
        assert (slots == o_slots).all(), f"batch {t}"
        evictions += nv
        if t % 10 == 9 or t < 3:
            assert_state_equal(cache, ora, dtype, f"batch {t}")
            # resynchronise the oracle's fp64 master with the GPU's fp32 master so rounding does not accumulate
            g = state_np(cache)
            ora.load_state(g["master"], g["size"], g["access"], g["last"], g["valid"], ora.clock)
    assert evictions > 0
    s = cache.stats()
    assert s["inserts"] - s["evictions"] == s["occupancy"] and s["lookups"] == sp.n_queries
    cache.check_status()


@pytest.mark.parametrize("fused", [1, 0])
def test_streaming_step_reproduces_the_hand_computed_example(golden_dir, fused):
    """The two pencil-computed batches of tests/golden/streaming_two_batches.json (capacity 4; one hit and two misses
    each; one free slot, then none) through siso_stream_step itself, not through the oracle: outputs and the whole
    state after each batch.  The vectors are padded with zeros from dim 4 to dim 8 (rows must be multiples of 8)."""
    import json, os
    ex = json.load(open(os.path.join(golden_dir, "streaming_two_batches.json")))
    inf = lambda a: np.array([siso.ACCESS_INF if x == "inf" else x for x in a], dtype=np.uint32)
    pad = lambda v: np.pad(np.array(v, dtype=np.float32), ((0, 0), (0, 4)))
    cache = siso.SisoCache(ex["capacity"], 8, "f32")
    cache.set_option(siso.OPT_STREAM_FUSED, fused)
    init = ex["initial"]
    cache.import_(torch.from_numpy(pad(init["vectors"])), torch.tensor(init["size"], dtype=torch.float64),
                  torch.from_numpy(inf(init["access"]).view(np.int32)), torch.tensor(init["last"], dtype=torch.int64),
                  torch.tensor(init["valid"], dtype=torch.uint8), ex["clock_before"])
    for b in ex["batches"]:
        out = [x.cpu().numpy() for x in cache.stream_step(torch.from_numpy(pad(b["queries"])).cuda(), float(ex["theta"]))]
        idx, sim, hit, victims, slots = out
        assert idx[:, 0].tolist() == b["idx"] and hit.tolist() == b["hit"]
        assert np.abs(sim[:, 0] - np.array(b["sim"])).max() <= 1e-6
        nv = len(b["victims"])
        assert victims[:nv].tolist() == b["victims"] and (victims[nv:] == -1).all()
        assert slots.tolist() == b["slots"]
        g, a = state_np(cache), b["after"]
        assert g["valid"].tolist() == a["valid"] and cache.stats()["clock"] == a["clock"]
        assert np.abs(g["master"][:, :4] - np.array(a["vectors"])).max() <= 1e-6 and (g["master"][:, 4:] == 0).all()
        assert g["size"].tolist() == a["size"] and g["access"].tolist() == inf(a["access"]).tolist()
        assert g["last"].tolist() == a["last"]
    cache.check_status()
    cache.close()


def test_fused_streaming_maintenance_equals_separate_kernels_bit_for_bit():
    sp = W.StreamSpec(capacity=1000, dim=72, n_queries=256 * 40, batch=256, n_clusters=700, zipf_s=1.2,
                      reshuffle_every=256 * 20, theta=0.86, mode="P", dtype="bf16")
    st = W.QueryStream(sp)
    caches = []
    for fused in (1, 0):
        c = siso.SisoCache(sp.capacity, sp.dim, "bf16")
        c.set_option(4, fused)
        caches.append(c)
    for t, q, _ in st.batches():
        outs = [[x.cpu().numpy() for x in c.stream_step(to_dev(q, "bf16"), float(sp.theta))] for c in caches]
        for x, y in zip(*outs):
            assert (x == y).all(), f"batch {t}"
    a, b = state_np(caches[0]), state_np(caches[1])
    live = a["valid"] == 1
    assert (a["valid"] == b["valid"]).all() and caches[0].stats() == caches[1].stats()
    for k in ("master", "vecs", "size", "access", "last"):
        assert (a[k][live] == b[k][live]).all(), k
    assert caches[0].stats()["evictions"] > 0
    assert caches[0].launch_count < caches[1].launch_count
    for c in caches:
        c.check_status()
        c.close()


@pytest.mark.parametrize("seed", [11, 12, 13, 14, 15, 16])
def test_three_forms_of_the_streaming_step_agree_on_random_shapes(seed):
    """The fused step with the eviction-order list kept across batches (default), the fused step without it and the
    separate kernels, on a random capacity / dim / batch size / threshold, with evictions (with and without decay),
    merges and plain lookups + updates thrown in between the batches: every output of every batch and the whole state
    must agree bit for bit (each form is also compared with the oracle elsewhere; this guards their equivalence where
    the oracle is too slow to follow)."""
    rng = np.random.default_rng(seed)
    dtype = "bf16" if rng.random() < 0.7 else "f32"
    cap = int(rng.choice([300, 1000, 4096, 9000]))
    dim = int(rng.choice([64, 128, 264, 768]))
    batch = int(rng.choice([1, 7, 64, 200, 256]))
    nb = int(rng.integers(80, 160))
    theta = float(rng.choice([0.7, 0.8, 0.86, 0.9]))
    ncl = max(8, int(cap * rng.choice([0.5, 1.5, 4.0])))
    sp = W.StreamSpec(capacity=cap, dim=dim, n_queries=batch * nb, batch=batch, n_clusters=ncl, zipf_s=1.2,
                      reshuffle_every=max(batch, batch * nb // 3), theta=theta, mode="P", dtype=dtype, seed=seed)
    q_all = to_dev(W.QueryStream(sp).block(0, nb), dtype)
    caches = []
    for fused, list_off in ((1, 0), (1, 1), (0, 0)):
        c = siso.SisoCache(cap, dim, dtype)
        c.set_option(siso.OPT_STREAM_FUSED, fused)
        c.set_option(siso.OPT_STREAM_LIST, list_off)
        caches.append(c)
    pre = int(cap * rng.choice([0.0, 0.6, 0.98]))
    if pre:
        fill_sp = W.StreamSpec(capacity=cap, dim=dim, n_queries=pre, batch=pre, n_clusters=ncl, theta=theta, mode="P", dtype=dtype,
                               seed=seed + 100)
        filler = to_dev(W.QueryStream(fill_sp).block(0, 1), dtype)[:pre]
        for c in caches:
            c.insert(filler)
    other = rng.random(nb)
    for t in range(nb):
        q = q_all[t * batch:(t + 1) * batch]
        outs = [[x.clone() for x in c.stream_step(q, theta)] for c in caches]
        for o in outs[1:]:
            assert all(torch.equal(x, y) for x, y in zip(outs[0], o)), f"batch {t}"
        if other[t] < 0.04:
            m, flags = int(rng.integers(1, 40)), (siso.EVICT_DECAY if rng.random() < 0.5 else 0)
            vs = [c.evict(m, flags) for c in caches]
            assert all(torch.equal(vs[0], v) for v in vs[1:]), f"evict after batch {t}"
        elif other[t] < 0.06:
            ms = []
            for c in caches:
                try:
                    ms.append(c.merge(0.95, siso.MERGE_WEIGHTED_MEAN))
                except siso.SisoError as e:          # more pairs than the candidate buffer holds: nothing is modified
                    assert e.status == 5
                    ms.append(None)
            if any(m is None for m in ms):
                assert all(m is None for m in ms), f"merge after batch {t}: overflow in some forms only"
            else:
                assert all(torch.equal(ms[0][0], m[0]) and ms[0][1] == m[1] for m in ms[1:]), f"merge after batch {t}"
        elif other[t] < 0.10:
            for c in caches:
                i, _, h = c.lookup(q, theta, 1)
                c.update(q, i, h)
        if t % 40 == 39 or t == nb - 1:
            sts = [state_np(c) for c in caches]
            for s2 in sts[1:]:
                for k in ("valid", "size", "access", "last", "master", "vecs"):
                    assert (sts[0][k] == s2[k]).all(), f"{k} after batch {t}"
    assert caches[0].stats() == caches[1].stats()
    for c in caches:
        c.check_status()
        c.close()


def test_streaming_eviction_is_exact_when_the_sample_misleads():
    """The fused step chooses its victims with the help of a strided sample of 256 entries.  Here exactly the
    sampled entries hold the smallest keys, so the sample says that hardly any entry is small; the selection
    must notice (fewer candidates than victims) and still return the m smallest keys in key order."""
    cap, D, B = 4096, 64, 256
    cent = W.f32_to_bf16_bits(W.unit_gaussian_rows(cap, D, 5, 901))
    cache = siso.SisoCache(cap, D, "bf16")
    cache.insert(to_dev(cent, "bf16"))
    g = state_np(cache)
    clock = cache.stats()["clock"]
    # for this many victims the step's sampler sorts one entry per 16-slot window w: the first live one of the window's
    # first quarter, slot 16 w + ((clock + 1) * 2654435761 mod 4)
    off = ((clock + 1) * 2654435761) % (cap // 256 // 4)
    size = np.ones(cap)
    size[np.arange(256) * (cap // 256) + off] = 0.5
    cache.import_(torch.from_numpy(g["master"]), torch.from_numpy(size), torch.from_numpy(g["access"].view(np.int32)),
                  torch.from_numpy(g["last"].view(np.int64)), torch.from_numpy(g["valid"]), clock)
    ora = oracle.OracleCache(cap, D, "bf16")
    ora.load_state(g["master"], size, g["access"], g["last"], g["valid"], clock)
    q = W.f32_to_bf16_bits(W.unit_gaussian_rows(B, D, 6, 902))          # unrelated directions: every row misses
    idx, sim, hit, victims, slots = [x.cpu().numpy() for x in cache.stream_step(to_dev(q, "bf16"), 0.86)]
    assert hit.sum() == 0
    o_idx, o_sim, o_hit, o_victims, o_slots = ora.stream_step(q, np.full(B, 0.86, np.float32), forced=(idx, hit))
    assert len(o_victims) == B and (np.sort(o_victims) == np.arange(256) * (cap // 256) + off).all()
    assert (victims == o_victims).all() and (slots == o_slots).all()
    assert_state_equal(cache, ora, "bf16")
    cache.check_status()
    cache.close()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_algorithm1_with_progressive_update_matches_oracle(dtype):
    """Algorithm 1 end to end on a second handle as C_new (copy, MergeCentroids with a repository, FilteringCentroids with
    the decay), then UpdateCentroids a group of slots at a time with lookups in between (Sec. 4.2, update step)."""
    w = W.config(3, seed=31, mode="P", n_centroids=1600, n_queries=300, dim=72, n_clusters=90, sigma=0.06, dtype=dtype)
    M, n_repo, group = 1000, 700, 256
    cur, o_cur = make_pair(dataclass_slice(w, 0, 900), capacity=M,
                           sizes=np.random.default_rng(3).integers(1, 9, 900).astype(np.float64))
    assert (cur.evict(60).cpu().numpy() == o_cur.evict(60)).all()                      # holes in C_cur
    new = siso.SisoCache(M + n_repo, w.dim, dtype)
    o_new = oracle.OracleCache(M + n_repo, w.dim, dtype)
    new.copy_from(cur)
    o_new.copy_from(o_cur)
    assert_state_equal(new, o_new, dtype, "C_new <- C_cur")
    repo, repo_sizes = w.centroids[900:], np.random.default_rng(4).integers(1, 5, n_repo).astype(np.float64)
    seed = o_new.valid.copy()
    mm, n_merged = new.merge(0.9, siso.MERGE_SIZES_ONLY, repo=to_dev(repo, dtype), repo_sizes=torch.from_numpy(repo_sizes))
    o_new.insert(repo, sizes=repo_sizes)
    entry, valid0, sizes0 = o_new.master.copy(), o_new.valid.copy(), o_new.size.copy()
    o_mm, o_n = o_new.merge(0.9, False, seed_mask=seed, new_access_inf=True)
    if not (mm.cpu().numpy() == o_mm).all():
        adopt_gpu_merge(new, o_new, mm.cpu().numpy(), entry, valid0, seed, sizes0, 0.9, False, "C_new after the merge")
    over = o_new.occupancy - M
    assert over > 0 and (new.evict(over, siso.EVICT_DECAY).cpu().numpy() == o_new.evict(over, decay=True)).all()
    assert_state_equal(new, o_new, dtype, "C_new after filtering")
    # the live cache keeps serving while it is replaced group by group
    q, theta = w.queries, np.full(300, 0.86, np.float32)
    for g in range(0, M, group):
        cur.update_centroids(new, g, group)
        o_cur.update_centroids(o_new, g, group)
        got = [x.cpu().numpy() for x in cur.lookup(to_dev(q, dtype), 0.86, 2)]
        want = o_cur.lookup(q, theta, 2)
        check_lookup(got, want, o_cur.lookup_copy(), q, theta, TOL[dtype], valid=o_cur.valid)
        g_state = state_np(cur)
        assert (g_state["valid"] == o_cur.valid).all(), f"group at {g}"
    assert cur.stats()["occupancy"] == M == o_cur.occupancy
    live = np.flatnonzero(o_new.valid)
    g_state = state_np(cur)
    assert (g_state["size"] == o_new.size[live]).all() and (g_state["access"] == 0).all()
    assert np.abs(g_state["master"].astype(np.float64) - o_new.master[live]).max() <= 1e-6
    # a C_new with more entries than C_cur has slots is refused and nothing changes
    before = state_np(cur)
    big = siso.SisoCache(M + n_repo, w.dim, dtype)
    big.insert(to_dev(w.centroids[:1200], dtype))
    cur.update_centroids(big, 0, group)
    assert cur.sync_status() == 4
    after = state_np(cur)
    assert all((before[k] == after[k]).all() for k in before)
    for c in (cur, new, big):
        c.close()
