"""GPU parity of the threshold-to-hit-ratio table (Sec. 4.3) against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from gen import workloads as W
from util import TOL, to_dev

pytestmark = pytest.mark.gpu

siso = pytest.importorskip("paper_2508_18736_b200")


@pytest.mark.parametrize("dtype,n_cent,n_q,dim", [("bf16", 5000, 3000, 768), ("f32", 1500, 700, 384), ("bf16", 900, 2, 64)])
def test_t2h_counts_match_oracle(dtype, n_cent, n_q, dim):
    w = W.config(2 if dtype == "bf16" else 1, n_centroids=n_cent, n_queries=n_q, dim=dim, n_clusters=max(8, n_cent // 20),
                 mode="P", dtype=dtype)
    cache = siso.SisoCache(n_cent, dim, dtype)
    cache.insert(to_dev(w.centroids, dtype))
    thetas = np.round(np.arange(0.98, 0.59, -0.02), 2).astype(np.float32)
    before = cache.stats()
    hits = cache.t2h(to_dev(w.queries, dtype), torch.from_numpy(thetas)).cpu().numpy()
    cache.check_status()
    best = oracle.lookup(w.centroids, w.queries, 0.0, 1)[1][:, 0]
    o_hits, o_ratio = oracle.t2h_table(best, thetas)
    tol = TOL[dtype]
    for t in range(len(thetas)):
        band = int((np.abs(best - np.float64(thetas[t])) < tol).sum())      # queries too close to the threshold to call
        assert abs(int(hits[t]) - int(o_hits[t])) <= band
    assert (np.diff(hits) >= 0).all()
    after = cache.stats()
    assert after["hits"] == before["hits"] and after["occupancy"] == before["occupancy"]
    # the table drives the controller: same choice as the oracle's table whenever the counts agree
    if (hits == o_hits).all():
        gi, _ = siso.choose_theta(thetas, hits / float(n_q), 12.0, 0.1, 9.0)
        oi, _ = oracle.choose_theta(thetas, o_ratio, 12.0, 0.1, 9.0)
        assert gi == oi
    # each entry equals a real lookup's hit count at that threshold (same kernels, same comparison)
    idx, sim, hit = cache.lookup(to_dev(w.queries, dtype), float(thetas[7]), 1)
    assert int(hit.sum().item()) == int(hits[7])
    cache.close()


def test_t2h_rejects_bad_arguments():
    cache = siso.SisoCache(64, 64, "bf16")
    q = torch.zeros(4, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(siso.SisoError):
        cache.t2h(q, torch.zeros(2000))              # more thresholds than the entry point accepts
    with pytest.raises(siso.SisoError):
        cache.t2h(q[:0], torch.zeros(3))
    cache.close()
