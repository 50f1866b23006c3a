"""GPU parity of siso_cluster (community detection at theta_C, Sec. 4.1) against the CPU oracle, the planted-cluster
property at a size the oracle does not reach, and the hand-over of the centroids to MergeCentroids as C_repo."""
import numpy as np
import pytest
import torch

import oracle
from gen import workloads as W
from util import to_dev, widen64

pytestmark = pytest.mark.gpu

siso = pytest.importorskip("paper_2508_18736_b200")


def near_threshold(vecs, theta, tol):
    S = widen64(vecs) @ widen64(vecs).T
    np.fill_diagonal(S, -2)
    return int((np.abs(S - theta) < tol).sum())


@pytest.mark.parametrize("dtype,mode,theta,n,dim", [
    ("f32", "P", 0.86, 1500, 136),      # spread clusters: neighbourhoods overlap, founders compete
    ("f32", "T", 0.90, 2300, 64),       # tight clusters
    ("bf16", "P", 0.80, 1300, 200),
    ("bf16", "T", 0.88, 2900, 768),     # bf16 rows go to the tensor cores as they are (one product per pair of elements)
    ("f32", "L", 0.30, 700, 24),        # loose: long chains of dependent decisions
    ("f32", "P", 0.86, 5, 8),           # smaller than one tile
])
def test_cluster_matches_oracle(dtype, mode, theta, n, dim):
    w = W.config(3, seed=11, mode=mode, n_centroids=n, dim=dim, n_clusters=max(2, n // 16), sigma=0.06, dtype=dtype)
    cache = siso.SisoCache(64, dim, dtype)           # supplies dim, dtype and scratch; its contents play no part
    label, centres, sizes, cent = cache.cluster(to_dev(w.centroids, dtype), theta)
    o_label, o_centres, o_sizes, o_cent = oracle.cluster(w.centroids, theta)
    # both sides decide every pair in fp64 from the same bits; only a pair within rounding of theta could differ
    assert near_threshold(w.centroids, theta, 1e-12) == 0
    assert (label.cpu().numpy() == o_label).all()
    assert (centres.cpu().numpy() == o_centres).all()
    assert (sizes.cpu().numpy() == o_sizes).all()
    if dtype == "f32":
        # the same fp64 sums in the same order, rounded once to fp32
        assert (cent.cpu().numpy() == o_cent.astype(np.float32)).all()
    else:
        # the oracle's fp64 centroid rounded once to bf16; the GPU rounds fp64 -> fp32 -> bf16, which differs from one
        # rounding only in rare double-rounding cases, and then by one unit in the last place
        got = cent.view(torch.int16).cpu().numpy().view(np.uint16)
        want = oracle.round_bf16(o_cent)
        diff = got != want
        assert diff.mean() < 1e-3
        assert (np.abs(got.astype(np.int32) - want.astype(np.int32))[diff] <= 1).all()
    assert cache.stats()["occupancy"] == 0
    cache.check_status()
    cache.close()


def test_planted_clusters_at_a_larger_size_and_overflow():
    # 20,000 vectors in 800 tight clusters: the communities must be the planted clusters, whatever the order
    w = W.config(3, seed=12, mode="T", n_centroids=20000, dim=128, n_clusters=800, sigma=0.06)
    cache = siso.SisoCache(64, 128, "f32")
    label, centres, sizes, _ = cache.cluster(to_dev(w.centroids, "f32"), 0.9, want_centroids=False)
    label, centres, sizes = label.cpu().numpy(), centres.cpu().numpy(), sizes.cpu().numpy()
    planted = w.centroid_labels
    assert len(centres) == len(np.unique(planted)) and sizes.sum() == 20000
    assert (planted[label] == planted).all()                                   # every vector sits with a centre of its own cluster
    assert (sizes == np.bincount(planted, minlength=800)[planted[centres]]).all()
    assert (np.diff(sizes) <= 0).all()          # disjoint, equal-sized neighbourhood sets: founding order = size order
    cache.check_status()
    # one community of everything needs 2e8 pairs: more than the candidate buffer holds
    with pytest.raises(siso.SisoError) as e:
        cache.cluster(to_dev(w.centroids, "f32"), -1.0, want_centroids=False)
    assert e.value.status == 5
    cache.close()


def test_clusters_feed_merge_as_repository():
    """Sec. 4: SISO-Cluster fills the centroid repository, MergeCentroids promotes it into the cache."""
    w = W.config(3, seed=13, mode="T", n_centroids=3000, dim=64, n_clusters=150, sigma=0.06)
    cache = siso.SisoCache(1024, 64, "f32")
    ora = oracle.OracleCache(1024, 64, "f32")
    label, centres, sizes, cent = cache.cluster(to_dev(w.centroids, "f32"), 0.9)
    o_label, o_centres, o_sizes, o_cent = oracle.cluster(w.centroids, 0.9)
    assert (centres.cpu().numpy() == o_centres).all() and (sizes.cpu().numpy() == o_sizes).all()
    k = len(o_centres)
    assert k == 150
    mm, n_merged = cache.merge(0.9, siso.MERGE_SIZES_ONLY, repo=cent, repo_sizes=sizes)
    seed = ora.valid.copy()
    ora.insert(cent.cpu().numpy(), sizes=o_sizes)
    o_mm, o_n = ora.merge(0.9, False, seed_mask=seed, new_access_inf=True)
    assert n_merged == o_n == 0 and (mm.cpu().numpy() == o_mm).all()           # distinct clusters: all are promoted
    st = cache.export()
    live = st["valid"].cpu().numpy() == 1
    assert live.sum() == k and (st["size"].cpu().numpy()[live] == o_sizes).all()
    cache.check_status()
    cache.close()
