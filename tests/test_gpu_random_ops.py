"""Seeded random sequences of every cache operation, each step compared with the oracle (lookups by the comparison rules,
state after every change), the oracle resynchronised from the exported GPU state after each verified step so that
rounding of the fp32 master does not accumulate into a false alarm.  What single-operation tests cannot see shows here:
holes left by merges and evictions, derived copies that must be refreshed, counters and clocks across operations."""
import numpy as np
import pytest
import torch

import oracle
from gen import workloads as W
from test_gpu_maintenance import assert_state_equal, state_np
from util import TOL, check_lookup, to_dev

pytestmark = pytest.mark.gpu

siso = pytest.importorskip("paper_2508_18736_b200")


def resync(cache, dtype):
    st = cache.export()
    torch.cuda.synchronize()
    ora = oracle.OracleCache(cache.capacity, cache.dim, dtype)
    ora.load_state(st["master"].cpu().numpy(), st["size"].cpu().numpy(), st["access"].cpu().numpy().view(np.uint32),
                   st["last"].cpu().numpy().view(np.uint64), st["valid"].cpu().numpy(), cache.stats()["clock"])
    return ora


@pytest.mark.parametrize("dtype,dim,seed,cap", [
    ("bf16", 72, 0, 700), ("bf16", 128, 1, 700), ("f32", 72, 2, 700), ("f32", 136, 3, 700), ("bf16", 264, 4, 700),
    ("f32", 384, 5, 700), ("bf16", 1024, 6, 700), ("f32", 8, 7, 700),
    ("f32", 136, 8, 4500), ("bf16", 136, 9, 4500),          # large enough for the tensor-core merge sweep
])
def test_random_operation_sequences_match_the_oracle(dtype, dim, seed, cap):
    rng = np.random.default_rng(100 + seed)
    pool = W.config(2 if dtype == "bf16" else 1, seed=70 + seed, mode="P", n_centroids=3000, n_queries=3000, dim=dim, n_clusters=150,
                    dtype=dtype, theta=(0.78, 0.93))
    rows = np.concatenate([pool.centroids, pool.queries])              # 6000 vectors around 150 cluster means

    def draw(n):
        return rows[rng.integers(0, len(rows), n)]

    cache = siso.SisoCache(cap, dim, dtype)
    ora = oracle.OracleCache(cap, dim, dtype)
    done = {k: 0 for k in ("insert", "lookup+update", "stream", "merge", "evict", "room+insert")}
    for step in range(80):
        occ = int(ora.valid.sum())
        op = rng.choice(list(done), p=[0.15, 0.25, 0.25, 0.1, 0.1, 0.15])
        what = f"seed {seed} step {step} {op}"
        if op == "insert":
            n = int(rng.integers(0, min(cap - occ, max(200, cap // 3)) + 1))
            v = draw(n)
            sizes = rng.integers(1, 20, n).astype(np.float64) if rng.random() < 0.5 else None
            slots = cache.insert(to_dev(v, dtype), None if sizes is None else torch.from_numpy(sizes)) if n else None
            if n:
                assert (slots.cpu().numpy() == ora.insert(v, sizes=sizes)).all(), what
        elif op == "lookup+update":
            n, k = int(rng.integers(1, 1500)), int(rng.integers(1, 9))
            q = draw(n)
            theta = rng.uniform(0.75, 0.95, n).astype(np.float32)
            per_query = rng.random() < 0.5
            if not per_query:
                theta[:] = theta[0]
            got = cache.lookup(to_dev(q, dtype), torch.from_numpy(theta).cuda() if per_query else float(theta[0]), k)
            idx, sim, hit = [x.cpu().numpy() for x in got]
            check_lookup((idx, sim, hit), ora.lookup(q, theta, k), ora.lookup_copy(), q, theta, TOL[dtype], valid=ora.valid)
            cache.update(to_dev(q, dtype), got[0], got[2])
            ora.update(q, idx, hit)
        elif op == "stream":
            n = int(rng.integers(1, 300))
            q = draw(n)
            theta = np.full(n, rng.uniform(0.8, 0.92), np.float32)
            pre_copy, pre_valid = ora.lookup_copy(), ora.valid.copy()
            idx, sim, hit, victims, slots = [x.cpu().numpy() for x in cache.stream_step(to_dev(q, dtype), float(theta[0]))]
            o_idx, o_sim, o_hit, o_victims, o_slots = ora.stream_step(q, theta, forced=(idx, hit))
            check_lookup((idx, sim, hit), (o_idx, o_sim, o_hit), pre_copy, q, theta, TOL[dtype], valid=pre_valid)
            nv = len(o_victims)
            assert (victims[:nv] == o_victims).all() and (victims[nv:] == -1).all() and (slots == o_slots).all(), what
        elif op == "merge":
            theta_c, weighted = float(rng.uniform(0.85, 0.95)), bool(rng.random() < 0.6)
            before = state_np(cache)["master"].astype(np.float64)
            mm, n = cache.merge(theta_c, siso.MERGE_WEIGHTED_MEAN if weighted else siso.MERGE_SIZES_ONLY)
            o_mm, o_n = ora.merge(theta_c, weighted)
            mm = mm.cpu().numpy()
            if not (mm == o_mm).all():
                for i in np.flatnonzero(mm != o_mm):       # only a decision within 1e-5 of the threshold or of the runner-up may differ
                    sims = [float(before[i] @ before[t]) for t in (mm[i], o_mm[i]) if t != i]
                    assert min(abs(s - theta_c) for s in sims) < 1e-5 or (len(sims) == 2 and abs(sims[0] - sims[1]) < 1e-5), what
                ora = resync(cache, dtype)
            else:
                assert n == o_n, what
        elif op == "evict":
            m, decay = int(rng.integers(0, occ + 3)), bool(rng.random() < 0.5)
            got = cache.evict(m, siso.EVICT_DECAY if decay else 0).cpu().numpy()
            assert (got == ora.evict(m, decay)).all(), what
        else:
            n = int(rng.integers(1, 250))
            q = draw(n)
            hit = (rng.random(n) < 0.6).astype(np.uint8)
            n_miss = int((hit == 0).sum())
            if n_miss > cap:
                continue
            h = torch.from_numpy(hit).cuda()
            victims = cache.make_room(h).cpu().numpy()
            lack = max(0, n_miss - (cap - occ))
            want = ora.evict(lack)
            assert (victims[:lack] == want).all() and (victims[lack:] == -1).all(), what
            assert (cache.insert_misses(to_dev(q, dtype), h).cpu().numpy() == ora.insert(q, hit)).all(), what
        cache.check_status()
        assert_state_equal(cache, ora, dtype, what)
        ora = resync(cache, dtype)
        done[op] += 1
    assert all(v > 0 for v in done.values()), done
    s = cache.stats()
    assert s["inserts"] - s["evictions"] - s["merges"] == s["occupancy"]
    cache.close()
