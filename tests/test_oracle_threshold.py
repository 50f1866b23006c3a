"""Pins for the oracle's threshold control: Eq. 1 / Eq. 2 closed forms and the T2H table."""
import math

import numpy as np

import oracle
from gen import workloads as W


def test_md1_wait_closed_forms():
    # Eq. 2 by hand: L = 12, lambda = 0.1, h = 0.5  =>  E = 6, W = 6 + 0.1*36 / (2*(1 - 0.6)) = 10.5
    assert abs(oracle.md1_wait(12.0, 0.1, 0.5) - 10.5) < 1e-12
    # no arrivals: waiting time is the service time; all hits: nothing reaches the LLM
    assert oracle.md1_wait(12.0, 0.0, 0.25) == 9.0 and oracle.md1_wait(12.0, 0.3, 1.0) == 0.0
    # Eq. 1 in its textbook M/D/1 form W = E (2 - rho) / (2 (1 - rho)) with rho = lambda E
    for L, lam, h in ((3.0, 0.2, 0.1), (11.98, 0.05, 0.4), (1.0, 0.9, 0.0)):
        E = L * (1 - h)
        rho = lam * E
        assert abs(oracle.md1_wait(L, lam, h) - E * (2 - rho) / (2 * (1 - rho))) < 1e-12
    # unstable queue
    assert math.isinf(oracle.md1_wait(12.0, 0.1, 0.1)) and math.isinf(oracle.md1_wait(10.0, 0.1, 0.0))
    # more hits never wait longer
    ws = [oracle.md1_wait(12.0, 0.08, h) for h in np.linspace(0, 1, 21)]
    assert all(a >= b for a, b in zip(ws, ws[1:]))


def test_t2h_table_counts_and_is_monotone():
    w = W.config(1, n_centroids=256, n_queries=500, dim=32, n_clusters=24, mode="P")
    best = oracle.lookup(w.centroids, w.queries, 0.0, 1)[1][:, 0]
    thetas = np.round(np.arange(0.98, 0.59, -0.02), 2).astype(np.float32)      # 0.98 down to 0.60
    hits, ratio = oracle.t2h_table(best, thetas)
    assert len(thetas) == 20 and thetas[0] == np.float32(0.98) and thetas[-1] == np.float32(0.6)
    want = [(best > np.float64(t)).sum() for t in thetas]
    assert hits.tolist() == want and np.allclose(ratio, np.array(want) / 500.0)
    assert (np.diff(hits) >= 0).all() and 0 < hits[-1] and hits[0] < 500      # lower threshold, more hits
    # each entry equals the hit count of an actual lookup at that threshold
    for t in (0, 7, 19):
        assert hits[t] == oracle.lookup(w.centroids, w.queries, float(thetas[t]), 1)[2].sum()
    # strict comparison: a similarity equal to the threshold is a miss
    h, _ = oracle.t2h_table(np.array([0.5, 0.75, 0.75]), np.array([0.75, 0.5], dtype=np.float32))
    assert h.tolist() == [0, 2]


def test_choose_theta_takes_the_highest_threshold_that_meets_the_slo():
    thetas = np.array([0.98, 0.9, 0.8, 0.7, 0.6], dtype=np.float32)
    ratio = np.array([0.1, 0.3, 0.5, 0.7, 0.85])
    L, lam = 12.0, 0.1
    ws = [oracle.md1_wait(L, lam, h) for h in ratio]          # inf, 26.04, 10.5, 4.61, 1.98
    assert math.isinf(ws[0]) and abs(ws[2] - 10.5) < 1e-12
    i, w = oracle.choose_theta(thetas, ratio, L, lam, 11.0)
    assert i == 2 and abs(w - 10.5) < 1e-12
    assert oracle.choose_theta(thetas, ratio, L, lam, 10.5)[0] == 3          # S > W is strict
    assert oracle.choose_theta(thetas, ratio, L, lam, 100.0)[0] == 1         # the unstable entry never qualifies
    assert oracle.choose_theta(thetas, ratio, L, lam, 1.0) == (-1, math.inf)
    # order of the table does not matter
    p = np.array([3, 0, 4, 2, 1])
    i, _ = oracle.choose_theta(thetas[p], ratio[p], L, lam, 11.0)
    assert thetas[p][i] == np.float32(0.8)


def test_correction_step_moves_one_entry_when_estimate_is_off_by_more_than_ten_percent():
    thetas = np.array([0.9, 0.98, 0.8, 0.7], dtype=np.float32)          # unordered on purpose
    assert oracle.correct_theta(thetas, 0, 10.0, 10.9) == 0             # |10 - 10.9| / 10.9 = 8 %: keep
    assert oracle.correct_theta(thetas, 0, 10.0, 12.0) == 2             # measured longer: next lower threshold (0.8)
    assert oracle.correct_theta(thetas, 0, 10.0, 8.0) == 1              # measured shorter: next higher (0.98)
    assert oracle.correct_theta(thetas, 3, 10.0, 20.0) == 3             # already the lowest entry
    assert oracle.correct_theta(thetas, 1, 10.0, 5.0) == 1              # already the highest entry


def test_library_host_functions_equal_the_oracle():
    """The library's scalar threshold-control functions need no GPU: compare them with the oracle here."""
    import paper_2508_18736_b200 as siso
    from paper_2508_18736_b200 import build
    build.build()
    rng = np.random.default_rng(3)
    thetas = np.round(np.arange(0.98, 0.59, -0.02), 2).astype(np.float32)
    for _ in range(200):
        ratio = np.sort(rng.random(20))
        L, lam, slo = rng.uniform(0.5, 15), rng.uniform(0.0, 0.5), rng.uniform(0.5, 30)
        for h in ratio[::5]:
            a, b = siso.md1_wait(L, lam, h), oracle.md1_wait(L, lam, h)
            assert a == b or abs(a - b) <= 1e-12 * abs(b)
        gi, gw = siso.choose_theta(thetas, ratio, L, lam, slo)
        oi, ow = oracle.choose_theta(thetas, ratio, L, lam, slo)
        assert gi == oi and (gw == ow or abs(gw - ow) <= 1e-12 * abs(ow))
        c = int(rng.integers(0, 20))
        w_est, w_meas = rng.uniform(1, 20), rng.uniform(1, 20)
        assert siso.correct_theta(thetas, c, w_est, w_meas) == oracle.correct_theta(thetas, c, w_est, w_meas)
