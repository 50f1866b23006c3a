"""Pins for the oracle's update, merge, evict, insert and streaming step: closed forms, the
hand-computed example, independent transcriptions of Algorithm 1 in pure Python, invariants."""
import json
import os

import numpy as np
import pytest

import oracle
from gen import workloads as W
from util import verify_merge_map

INF = oracle.ACCESS_INF


def make_cache(vectors, sizes=None, dtype="f32", capacity=None):
    vectors = np.asarray(vectors)
    n, d = vectors.shape
    c = oracle.OracleCache(capacity or n, d, dtype)
    c.insert(vectors, sizes=sizes)
    return c


@pytest.fixture(scope="module")
def example(golden_dir):
    return json.load(open(os.path.join(golden_dir, "four_centroid_example.json")))


# ---------------------------------------------------------------------------- update
def test_update_worked_example(example):
    c = make_cache(np.array(example["centroids"], dtype=np.float64), sizes=example["sizes"])
    q = np.array([example["lookup"]["query"]], dtype=np.float64)
    idx, _, hit = c.lookup(q, 0.90)
    c.update(q, idx, hit)
    u = example["update"]
    np.testing.assert_allclose(c.master[u["slot"]], u["new_vector"], atol=1e-6)
    assert c.size[u["slot"]] == u["new_size"]
    others = [i for i in range(4) if i != u["slot"]]
    np.testing.assert_array_equal(c.master[others], np.array(example["centroids"], dtype=np.float64)[others])
    assert c.clock == 1 and c.last[u["slot"]] == 1 and (c.last[others] == 0).all()


def test_update_closed_form_unit_norm_and_counters():
    rng = np.random.default_rng(1)
    w = W.config(1, n_centroids=40, n_queries=64, dim=24, n_clusters=5, mode="T", sigma=0.2)
    sizes = rng.integers(1, 9, 40).astype(np.float64) / 1.1          # fractional, as after a decay
    c = make_cache(w.centroids, sizes=sizes)
    c.access[:] = rng.integers(0, 5, 40)
    c.access[7] = INF - 1
    before, acc0 = c.master.copy(), c.access.copy()
    idx = rng.integers(0, 40, 64).astype(np.int32)
    idx[:3] = 7
    hit = (rng.random(64) < 0.6).astype(np.uint8)
    hit[:3] = 1
    c.update(w.queries, idx, hit)
    Q = w.queries.astype(np.float64)
    for j in range(40):
        H = [b for b in range(64) if hit[b] and idx[b] == j]
        if not H:
            np.testing.assert_array_equal(c.master[j], before[j])
            assert c.size[j] == sizes[j] and c.access[j] == acc0[j] and c.last[j] == 0
            continue
        v = sizes[j] * before[j] + Q[H].sum(0)
        np.testing.assert_allclose(c.master[j], v / np.linalg.norm(v), rtol=0, atol=1e-14)
        assert abs(np.linalg.norm(c.master[j]) - 1.0) < 1e-12
        assert c.size[j] == sizes[j] + len(H)
        assert c.access[j] == min(INF, int(acc0[j]) + len(H))
        assert c.last[j] == 1
    assert c.access[7] == INF                                        # saturates, never wraps


def test_update_special_cases():
    w = W.config(1, n_centroids=8, n_queries=16, dim=12, n_clusters=8, mode="T", sigma=0.3)
    # q == c: the vector does not move, the count grows
    c = make_cache(w.centroids, sizes=[3.0] * 8)
    c.update(w.centroids[[5]], np.array([5]), np.array([1]))
    np.testing.assert_allclose(c.master[5], w.centroids[5].astype(np.float64) /
                               np.linalg.norm(w.centroids[5].astype(np.float64)), atol=1e-15)
    assert c.size[5] == 4.0
    # order inside the batch does not matter (up to fp64 rounding of the sum)
    idx = np.array([2] * 16, dtype=np.int32)
    hit = np.ones(16, dtype=np.uint8)
    a, b = make_cache(w.centroids), make_cache(w.centroids)
    p = np.random.default_rng(0).permutation(16)
    a.update(w.queries, idx, hit)
    b.update(w.queries[p], idx, hit)
    np.testing.assert_allclose(a.master, b.master, atol=1e-15)
    # k identical hits equal one hit of weight k:  normalise(n c + k q)
    k = 5
    d = make_cache(w.centroids, sizes=[2.0] * 8)
    d.update(np.repeat(w.queries[[0]], k, 0), np.full(k, 1, dtype=np.int32), np.ones(k, dtype=np.uint8))
    v = 2.0 * w.centroids[1].astype(np.float64) + k * w.queries[0].astype(np.float64)
    np.testing.assert_allclose(d.master[1], v / np.linalg.norm(v), atol=1e-14)
    # misses change nothing but the clock
    e = make_cache(w.centroids)
    m0 = e.master.copy()
    e.update(w.queries, idx, np.zeros(16, dtype=np.uint8))
    np.testing.assert_array_equal(e.master, m0)
    assert e.clock == 1 and (e.last == 0).all()


def test_lookup_copy_is_one_rounding_of_the_master():
    w = W.config(2, n_centroids=32, n_queries=8, dim=64, n_clusters=4)
    c = make_cache(w.centroids, dtype="bf16")
    assert (c.lookup_copy() == w.centroids).all()                   # inserted bits survive untouched
    c.update(w.queries, np.zeros(8, dtype=np.int32), np.ones(8, dtype=np.uint8))
    assert (c.lookup_copy()[0] == oracle.round_bf16(c.master[0])).all()


# ---------------------------------------------------------------------------- merge
def alg1_merge_python(vec, size, n_seed, theta):
    """Independent transcription of MergeCentroids: C_new grows, closest = max cosine, strict '>'."""
    c_new = list(range(n_seed))
    size = list(size)
    mp = list(range(len(vec)))
    for i in range(n_seed, len(vec)):
        best, best_s = None, None
        for j in c_new:
            s = float(np.dot(vec[i], vec[j]))
            if best is None or s > best_s:
                best, best_s = j, s
        if best is not None and best_s > theta:
            size[best] += size[i]
            mp[i] = best
        else:
            c_new.append(i)
    return mp, size, c_new


def test_merge_worked_example(example):
    C = np.array(example["centroids"], dtype=np.float64)
    m = example["merge"]
    c = make_cache(C, sizes=example["sizes"])
    mm, n = c.merge(0.90, weighted_mean=True)
    assert mm.tolist() == m["theta_0.90"]["map"] and n == 0
    np.testing.assert_array_equal(c.master, C)
    for weighted in (False, True):
        c = make_cache(C, sizes=example["sizes"])
        mm, n = c.merge(0.75, weighted_mean=weighted)
        e = m["theta_0.75"]
        assert mm.tolist() == e["map"] and n == e["n_merged"]
        assert c.size[1] == e["size_of_1"] and c.valid.tolist() == [1, 1, 0, 1]
        want = e["weighted_mean_vector_1"] if weighted else e["sizes_only_vector_1"]
        np.testing.assert_allclose(c.master[1], want, atol=1e-6)
        assert float(c.master[0] @ c.master[1]) < 0.75
        np.testing.assert_array_equal(c.master[[0, 3]], C[[0, 3]])


@pytest.mark.parametrize("n_seed", [0, 30])
def test_merge_equals_python_transcription(n_seed):
    w = W.config(3, n_centroids=160, dim=20, n_clusters=12, mode="P")
    sizes = np.random.default_rng(2).integers(1, 6, 160).astype(np.float64)
    c = make_cache(w.centroids, sizes=sizes)
    entry = c.master.copy()
    c.access[:] = 3
    mm, n = c.merge(0.9, weighted_mean=False, n_seed=n_seed, new_access_inf=True)
    mp, size, c_new = alg1_merge_python(entry, sizes, n_seed, 0.9)
    assert mm.tolist() == mp and n == sum(1 for i, t in enumerate(mp) if t != i) and n > 5
    np.testing.assert_array_equal(c.size[c_new], np.array(size)[c_new])
    np.testing.assert_array_equal(c.master, entry)                  # sizes only: no vector moves, bit for bit
    assert c.size[c.valid == 1].sum() == sizes.sum()                # cluster_size is conserved
    assert set(np.flatnonzero(c.valid)) == set(c_new)
    new = [i for i in c_new if i >= n_seed]
    assert (c.access[new] == INF).all() and (c.access[:n_seed] == 3).all()


def test_merge_invariants_and_extremes():
    w = W.config(3, n_centroids=200, dim=24, n_clusters=10, mode="P")
    c = make_cache(w.centroids)
    entry = c.master.copy()
    theta = 0.88
    mm, n = c.merge(theta, weighted_mean=True)
    surv = np.flatnonzero(c.valid)
    S = entry[surv] @ entry[surv].T
    np.fill_diagonal(S, -1)
    assert S.max() <= theta                                          # survivors' entry vectors are separated
    for i in range(200):
        t = mm[i]
        assert t <= i and mm[t] == t
        if t != i:
            assert entry[i] @ entry[t] > theta
            earlier = [s for s in surv if s < i]                     # closest among the survivors before i
            assert t == earlier[int(np.argmax(entry[i] @ entry[earlier].T))]
    np.testing.assert_allclose(np.linalg.norm(c.master[surv], axis=1), 1.0, atol=1e-12)
    for s in surv:                                                   # count-weighted mean of the members
        members = np.flatnonzero(mm == s)
        v = entry[members].sum(0)
        if len(members) > 1:
            np.testing.assert_allclose(c.master[s], v / np.linalg.norm(v), atol=1e-13)
        else:
            np.testing.assert_array_equal(c.master[s], entry[s])
    # fixed point: repeat until a pass merges nothing, then the FINAL vectors are separated too
    for _ in range(50):
        if c.merge(theta, weighted_mean=True)[1] == 0:
            break
    surv = np.flatnonzero(c.valid)
    S = c.master[surv] @ c.master[surv].T
    np.fill_diagonal(S, -1)
    assert S.max() <= theta
    # theta = 1 merges nothing; theta = -1 sends everything to slot 0
    c = make_cache(w.centroids)
    assert c.merge(1.0, weighted_mean=True)[1] == 0 and c.valid.all()
    mm, n = c.merge(-1.0, weighted_mean=False)
    assert n == 199 and (mm == 0).all() and c.size[0] == 200 and c.valid.sum() == 1


def test_merge_skips_invalid_slots_and_tie_goes_to_earliest():
    C = np.eye(4, dtype=np.float64)[[0, 1, 0, 0]]                    # slots 0, 2, 3 identical
    c = make_cache(C)
    c.valid[0] = 0
    mm, n = c.merge(0.5, weighted_mean=False)
    assert mm.tolist() == [-1, 1, 2, 2] and n == 1
    c = make_cache(np.array([[1.0, 0], [1.0, 0], [1.0, 0]]))
    # seeds 0 and 1 are never compared with each other; slot 2 ties and joins the earliest
    mm, n = c.merge(0.5, weighted_mean=False, n_seed=2)
    assert mm.tolist() == [0, 1, 0] and n == 1 and c.size.tolist()[:2] == [2.0, 1.0]


# ---------------------------------------------------------------------------- evict
def test_evict_worked_example(example):
    e = example["evict"]
    for m, want in ((2, e["evict_2"]), (4, e["full_order"])):
        c = make_cache(np.eye(4), sizes=e["sizes"])
        c.access[:] = [INF if a == "inf" else a for a in e["access"]]
        assert c.evict(m, decay=(m == 2)).tolist() == want
        if m == 2:
            assert c.valid.tolist() == [1, 0, 0, 1]
            assert c.size[0] == c.size[3] == 5 / 1.1 and abs(c.size[0] - e["decayed_size_of_survivors"]) < 1e-14
            assert (c.access[[0, 3]] == 0).all()


def test_evict_equals_full_sort_and_literal_resorting_loop():
    rng = np.random.default_rng(4)
    n = 300
    c = make_cache(np.eye(n)[:, :8] + 1.0, sizes=rng.integers(1, 4, n) / 1.1 ** rng.integers(0, 3, n))
    c.access[:] = rng.choice([0, 1, 2, INF], n)
    c.last[:] = rng.integers(0, 5, n)
    c.valid[rng.random(n) < 0.2] = 0
    keys = [(c.size[i], int(c.access[i]), int(c.last[i]), i) for i in range(n) if c.valid[i]]
    order = [k[3] for k in sorted(keys)]
    # the algorithm as printed: while over capacity { sort ascending; remove the first }
    live, literal = list(keys), []
    for _ in range(57):
        live.sort()
        literal.append(live.pop(0)[3])
    size0 = c.size.copy()
    got = c.evict(57, decay=True).tolist()
    assert got == order[:57] == literal
    rest = order[57:]
    assert sorted(np.flatnonzero(c.valid)) == sorted(rest)
    np.testing.assert_array_equal(c.size[rest], size0[rest] / 1.1)
    assert (c.access[rest] == 0).all()
    # asking for more than there is empties the cache and pads with -1
    got = c.evict(len(rest) + 3).tolist()
    assert got[:len(rest)] == [k[3] for k in sorted((c.size[i], 0, int(c.last[i]), i) for i in rest)]
    assert got[len(rest):] == [-1] * 3 and c.valid.sum() == 0


def test_decay_closed_form_and_new_entries_outlive_equal_size_old_ones():
    c = make_cache(np.eye(3), sizes=[7.0, 7.0, 7.0])
    for _ in range(6):
        c.evict(0, decay=True)
    np.testing.assert_allclose(c.size, 7.0 / 1.1 ** 6, rtol=1e-15)
    c = make_cache(np.eye(3), sizes=[2.0, 2.0, 2.0])
    c.access[:] = [INF, 40, INF]                                     # slots 0, 2 are new (infinity)
    c.last[:] = [3, 9, 1]
    assert c.evict(3).tolist() == [1, 2, 0]                          # finite first, then older last_access


# ---------------------------------------------------------------------------- insert + stream
def test_insert_takes_free_slots_in_order_and_checks_capacity():
    c = oracle.OracleCache(6, 4, "bf16")
    v = W.f32_to_bf16_bits(np.eye(4, dtype=np.float32))
    c.clock = 9
    assert c.insert(v[:3]).tolist() == [0, 1, 2]
    c.valid[1] = 0
    slots = c.insert(v, hit=np.array([0, 1, 0, 0]))
    assert slots.tolist() == [1, -1, 3, 4]
    assert (c.lookup_copy()[[1, 3, 4]] == v[[0, 2, 3]]).all()
    assert (c.size[[1, 3, 4]] == 1).all() and (c.access[[1, 3, 4]] == INF).all() and (c.last[[1, 3, 4]] == 9).all()
    before = (c.master.copy(), c.valid.copy())
    with pytest.raises(OverflowError):
        c.insert(v[:2])
    np.testing.assert_array_equal(c.master, before[0])
    np.testing.assert_array_equal(c.valid, before[1])


def test_stream_conservation_and_recovery_after_reshuffle():
    sp = W.StreamSpec(capacity=64, dim=32, n_queries=64 * 120, batch=64, n_clusters=96, zipf_s=1.2,
                      reshuffle_every=64 * 60, theta=0.86, mode="T", sigma=0.25, dtype="bf16")
    st = W.QueryStream(sp)
    c = oracle.OracleCache(sp.capacity, sp.dim, "bf16")
    inserted = evicted = 0
    hits = []
    for t, q, _ in st.batches():
        occ0 = c.occupancy
        idx, sim, hit, victims, slots = c.stream_step(q, np.float32(sp.theta))
        inserted += int((slots >= 0).sum())
        evicted += len(victims)
        assert c.occupancy - occ0 == int((slots >= 0).sum()) - len(victims)
        assert c.occupancy <= sp.capacity
        assert (hit == 0).sum() == (slots >= 0).sum()
        hits.append(hit.mean())
        live = c.valid == 1
        np.testing.assert_allclose(np.linalg.norm(c.master[live], axis=1), 1.0, atol=2e-2)
    assert inserted - evicted == c.occupancy and evicted > 0
    hits = np.array(hits)
    assert hits[50:60].mean() > hits[:5].mean()                     # the cache warms up
    assert hits[60:63].mean() < hits[50:60].mean()                  # popularity reshuffle hurts ...
    assert hits[110:].mean() > hits[60:63].mean()                   # ... and the cache recovers


def _run_streaming_example(ex, step):
    """Feeds the hand-computed two-batch example through `step(cache, queries, theta)` and compares every output and
    the whole state after each batch with the pencil values.  Returns normally or raises AssertionError."""
    inf = lambda a: np.array([INF if x == "inf" else x for x in a], dtype=np.uint32)
    init = ex["initial"]
    c = oracle.OracleCache(ex["capacity"], ex["dim"], "f32")
    c.load_state(np.array(init["vectors"], dtype=np.float64), np.array(init["size"], dtype=np.float64),
                 inf(init["access"]), np.array(init["last"], dtype=np.uint64), np.array(init["valid"], dtype=np.uint8),
                 ex["clock_before"])
    for b in ex["batches"]:
        q = np.array(b["queries"], dtype=np.float64)
        idx, sim, hit, victims, slots = step(c, q, np.float32(ex["theta"]))
        assert idx[:, 0].tolist() == b["idx"] and hit.tolist() == b["hit"]
        np.testing.assert_allclose(sim[:, 0], b["sim"], atol=1e-6)
        assert victims.tolist() == b["victims"], "victims"
        assert slots.tolist() == b["slots"], "slots"
        a = b["after"]
        assert c.clock == a["clock"] and c.valid.tolist() == a["valid"]
        np.testing.assert_allclose(c.master, np.array(a["vectors"], dtype=np.float64), atol=1e-6)
        assert c.size.tolist() == a["size"] and c.access.tolist() == inf(a["access"]).tolist()
        assert c.last.tolist() == a["last"]


@pytest.fixture(scope="module")
def streaming_example(golden_dir):
    return json.load(open(os.path.join(golden_dir, "streaming_two_batches.json")))


def test_stream_step_worked_example(streaming_example):
    """lookup -> update -> evict(#miss - free) -> insert on a capacity-4 cache, two batches, every number by hand:
    Algorithm 1 (MergeCentroids' else-branch, FilteringCentroids' order) and Sec. 5.2.5 (spare-space vectors under LRU)."""
    _run_streaming_example(streaming_example, lambda c, q, th: c.stream_step(q, th))


def _evicts_one_per_miss(c, q, th):
    idx, sim, hit = c.lookup(q, th, 1)
    c.update(q, idx, hit)
    victims = c.evict(int((hit == 0).sum()))                     # forgets the free slots
    return idx, sim, hit, victims, c.insert(q, hit)


def _evicts_before_updating(c, q, th):
    idx, sim, hit = c.lookup(q, th, 1)
    n_miss, free = int((hit == 0).sum()), c.capacity - c.occupancy
    victims = c.evict(n_miss - free) if n_miss > free else np.empty(0, np.int32)
    c.update(q, idx, hit)                                        # the hit no longer protects its entry
    return idx, sim, hit, victims, c.insert(q, hit)


def _inserts_in_victim_order(c, q, th):
    idx, sim, hit = c.lookup(q, th, 1)
    c.update(q, idx, hit)
    n_miss, free = int((hit == 0).sum()), c.capacity - c.occupancy
    free_slots = np.flatnonzero(c.valid == 0).tolist()
    victims = c.evict(n_miss - free) if n_miss > free else np.empty(0, np.int32)
    order = free_slots + victims.tolist()                        # free slots first, then victims as evicted
    slots = np.full(len(q), -1, np.int32)
    for b, s in zip(np.flatnonzero(hit == 0), order):
        c.master[s], c.size[s], c.access[s], c.last[s], c.valid[s] = q[b], 1.0, INF, c.clock, 1
        slots[b] = s
    return idx, sim, hit, victims, slots


def _sees_its_own_batch(c, q, th):
    outs = [c.stream_step(q[b:b + 1], th) for b in range(len(q))]       # one query at a time: not batch-synchronous
    c.clock -= len(q) - 1
    cat = lambda j: np.concatenate([o[j] for o in outs])
    return cat(0), cat(1), cat(2), cat(3), cat(4)


def _keeps_the_old_clock(c, q, th):
    out = c.stream_step(q, th)
    c.last[c.last == c.clock] = c.clock - 1
    return out


@pytest.mark.parametrize("mistake", [_evicts_one_per_miss, _evicts_before_updating, _inserts_in_victim_order,
                                     _sees_its_own_batch, _keeps_the_old_clock])
def test_stream_step_worked_example_catches_planted_mistakes(streaming_example, mistake):
    """The example is chosen so that each plausible mistake in the composition changes a number in it."""
    with pytest.raises((AssertionError, RuntimeError)):          # RuntimeError: the oracle refuses an update of an empty slot
        _run_streaming_example(streaming_example, mistake)


def test_two_set_merge_with_interleaved_slots_equals_transcription():
    """C_cur and the repository entries may sit in any slots: seeds are given by a mask."""
    w = W.config(3, n_centroids=180, dim=20, n_clusters=14, mode="P")
    rng = np.random.default_rng(8)
    sizes = rng.integers(1, 6, 180).astype(np.float64)
    seed = rng.random(180) < 0.4
    c = make_cache(w.centroids, sizes=sizes)
    c.valid[rng.random(180) < 0.1] = 0
    c.access[:] = 5
    entry, valid0 = c.master.copy(), c.valid.copy()
    mm, n = c.merge(0.9, weighted_mean=True, seed_mask=seed, new_access_inf=True)
    # Algorithm 1 by hand: C_new starts as C_cur (slot order); repository entries in slot order
    c_new = [i for i in range(180) if valid0[i] and seed[i]]
    size, mp = list(sizes), [i if valid0[i] else -1 for i in range(180)]
    for i in range(180):
        if not valid0[i] or seed[i]:
            continue
        sims = [float(entry[i] @ entry[j]) for j in c_new]
        b = int(np.argmax(sims)) if sims else -1          # argmax returns the first maximum: earliest in C_new
        if b >= 0 and sims[b] > 0.9:
            size[c_new[b]] += sizes[i]
            mp[i] = c_new[b]
        else:
            c_new.append(i)
    assert mm.tolist() == mp and n == sum(1 for i, t in enumerate(mp) if t >= 0 and t != i) and n > 5
    assert sorted(np.flatnonzero(c.valid)) == sorted(c_new)
    np.testing.assert_array_equal(c.size[c_new], np.array(size)[c_new])
    new = [i for i in c_new if not seed[i]]
    assert (c.access[new] == INF).all() and (c.access[[i for i in c_new if seed[i]]] == 5).all()
    for s in c_new:                                        # weighted mean: survivor first, then members by slot
        members = [m for m in range(180) if mp[m] == s and m != s]
        if members:
            v = sizes[s] * entry[s] + sum(sizes[m] * entry[m] for m in members)
            np.testing.assert_allclose(c.master[s], v / np.linalg.norm(v), atol=1e-13)
    # a tie between a seed in a high slot and an earlier repository survivor goes to the seed (earlier in C_new)
    c = make_cache(np.array([[1.0, 0], [0, 1.0], [1.0, 0], [1.0, 0]]))
    mm, n = c.merge(0.5, weighted_mean=False, seed_mask=np.array([0, 0, 0, 1]))
    assert mm.tolist() == [3, 1, 3, 3] and n == 2


def test_tolerant_merge_verifier_accepts_the_oracle_and_rejects_wrong_maps():
    """The GPU tests accept a merge map that differs from the oracle's only through `verify_merge_map`; here that
    verifier is held against the oracle itself (one-set and two-set) and against planted wrong maps."""
    w = W.config(3, n_centroids=160, dim=20, n_clusters=12, mode="P")
    rng = np.random.default_rng(3)
    sizes = rng.integers(1, 6, 160).astype(np.float64)
    for seeded in (False, True):
        seed = (rng.random(160) < 0.4).astype(np.uint8) if seeded else np.zeros(160, np.uint8)
        c = make_cache(w.centroids, sizes=sizes)
        c.valid[rng.random(160) < 0.1] = 0
        entry, valid0 = c.master.copy(), c.valid.copy()
        mm, n = c.merge(0.9, weighted_mean=False, seed_mask=seed if seeded else None, new_access_inf=seeded)
        assert n > 5
        size = verify_merge_map(entry, valid0, seed, sizes, mm, 0.9, tol=0.0)
        live = c.valid == 1
        np.testing.assert_array_equal(size[live], c.size[live])
        merged = [i for i in range(160) if mm[i] >= 0 and mm[i] != i]
        surv = [i for i in range(160) if mm[i] == i and not seed[i]]
        S = entry @ entry.T
        bad = mm.copy()
        bad[merged[0]] = merged[0]                             # a merged entry declared a survivor
        with pytest.raises(AssertionError):
            verify_merge_map(entry, valid0, seed, sizes, bad, 0.9)
        bad = mm.copy()
        i = merged[-1]
        other = [s for s in surv if s < i and s != mm[i] and S[i, s] < S[i, mm[i]] - 1e-3]
        bad[i] = other[0]                                      # merged into a survivor that is not the closest
        with pytest.raises(AssertionError):
            verify_merge_map(entry, valid0, seed, sizes, bad, 0.9)
        bad = mm.copy()
        lone = [s for s in surv if s > 0 and S[s, [t for t in surv if t < s] or [s]].max() < 0.8]
        if lone:
            bad[lone[-1]] = [t for t in surv if t < lone[-1]][0]    # a survivor merged below the threshold
            with pytest.raises(AssertionError):
                verify_merge_map(entry, valid0, seed, sizes, bad, 0.9)
        bad = mm.copy()
        later = [(i, s) for i in merged for s in surv if s > i]
        bad[later[0][0]] = later[0][1]                         # merged into a LATER survivor
        with pytest.raises(AssertionError):
            verify_merge_map(entry, valid0, seed, sizes, bad, 0.9)


# ---------------------------------------------------------------------------- Algorithm 1 as a whole
def test_algorithm1_pipeline_and_progressive_update():
    """MergeCentroids -> FilteringCentroids -> UpdateCentroids (Algorithm 1), the update taken a group of slots at a
    time (Sec. 4.2, update step): after the last group C_cur holds exactly the entries of C_new, in C_new's slot order;
    in between, every slot is wholly old or wholly new."""
    w = W.config(3, seed=21, mode="P", n_centroids=90, dim=16, n_clusters=12, sigma=0.06)
    M = 50
    cur = make_cache(w.centroids[:40].astype(np.float64), sizes=np.arange(1, 41, dtype=np.float64), capacity=M)
    cur.evict(5)                                    # holes in C_cur
    old = {k: getattr(cur, k).copy() for k in ("master", "size", "access", "last", "valid")}
    new = oracle.OracleCache(M + 50, 16, "f32")
    new.copy_from(cur)
    assert (new.valid[:M] == cur.valid).all() and (new.valid[M:] == 0).all() and (new.master[:M] == cur.master).all()
    seed = new.valid.copy()
    new.insert(w.centroids[40:].astype(np.float64), sizes=np.full(50, 2.0))
    new.merge(0.9, False, seed_mask=seed, new_access_inf=True)
    over = new.occupancy - M
    assert over > 0
    new.evict(over, decay=True)
    assert new.occupancy == M
    live = np.flatnonzero(new.valid)
    for g in range(0, M, 16):
        cur.update_centroids(new, g, 16)
        done = min(M, g + 16)
        assert (cur.valid[:done] == 1).all()
        assert (cur.master[:done] == new.master[live[:done]]).all() and (cur.size[:done] == new.size[live[:done]]).all()
        for k in old:                               # the slots not yet reached are untouched
            assert (getattr(cur, k)[done:] == old[k][done:]).all()
    assert (cur.access == 0).all()                  # FilteringCentroids reset them
    np.testing.assert_allclose(cur.size, new.size[live])
    # a C_new with fewer entries than slots empties the tail
    new.evict(10)
    cur.update_centroids(new, 0, M)
    assert cur.occupancy == M - 10 and (cur.valid[M - 10:] == 0).all()
    # more entries than slots is refused
    big = oracle.OracleCache(M + 50, 16, "f32")
    big.insert(w.centroids[:60].astype(np.float64))
    with pytest.raises(ValueError):
        cur.update_centroids(big, 0, 16)
