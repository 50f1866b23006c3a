"""Pins for the oracle's clustering routine (Sec. 4.1, community detection at theta_C): two hand-computed examples,
an independent transcription in pure Python over a numpy similarity matrix, invariants, limiting thresholds, and the
recovery of planted clusters."""
import json
import os

import numpy as np
import pytest

import oracle
from gen import workloads as W


@pytest.fixture(scope="module")
def example(golden_dir):
    return json.load(open(os.path.join(golden_dir, "four_centroid_example.json")))


def reference_communities(V: np.ndarray, theta: float):
    """Independent statement: numpy similarity matrix, Python sets, an explicit visiting loop."""
    V = V.astype(np.float64)
    S = V @ V.T
    n = len(V)
    nbrs = [set(np.flatnonzero(S[v] > theta).tolist()) | {v} for v in range(n)]
    order = sorted(range(n), key=lambda v: (-len(nbrs[v]), v))
    owner = {}
    centres, sizes = [], []
    for v in order:
        if v in owner:
            continue
        members = sorted(u for u in nbrs[v] if u not in owner)
        for u in members:
            owner[u] = v
        centres.append(v)
        sizes.append(len(members))
    return np.array([owner[v] for v in range(n)], np.int32), np.array(centres, np.int32), np.array(sizes, np.float64), S


def test_hand_computed_four_centroids(example):
    ex = example["cluster"]["four_centroids_theta_0.75"]
    V = np.array(example["centroids"], dtype=np.float64)
    label, centres, sizes, cent = oracle.cluster(V, 0.75)
    assert label.tolist() == ex["label"] and centres.tolist() == ex["centres"] and sizes.tolist() == ex["sizes"]
    np.testing.assert_allclose(cent[0], ex["centroid_of_first"], atol=1e-6)
    np.testing.assert_allclose(cent[1], V[0], atol=1e-15)            # a community of one: its own vector


def test_hand_computed_circle(example):
    ex = example["cluster"]["five_on_a_circle"]
    a = np.deg2rad(np.array(ex["angles_deg"], dtype=np.float64))
    V = np.stack([np.cos(a), np.sin(a)], axis=1)
    label, centres, sizes, cent = oracle.cluster(V, ex["theta"])
    assert label.tolist() == ex["label"] and centres.tolist() == ex["centres"] and sizes.tolist() == ex["sizes"]
    np.testing.assert_allclose(cent[0], ex["centroid_of_first"], atol=1e-6)


@pytest.mark.parametrize("seed,mode,theta", [(0, "P", 0.86), (1, "P", 0.70), (2, "T", 0.90), (3, "L", 0.30)])
def test_equals_independent_transcription(seed, mode, theta):
    w = W.config(3, seed=seed, mode=mode, n_centroids=180, dim=24, n_clusters=12, sigma=0.06)
    V = w.centroids
    label, centres, sizes, cent = oracle.cluster(V, theta)
    r_label, r_centres, r_sizes, S = reference_communities(V, theta)
    # the two sum in different orders; a pair within rounding of theta would make the comparison meaningless
    off = S[~np.eye(len(V), dtype=bool)]
    assert np.abs(off - theta).min() > 1e-12
    assert (label == r_label).all() and (centres == r_centres).all() and (sizes == r_sizes).all()
    for c, v in enumerate(centres):
        m = V[label == v].astype(np.float64).sum(0)
        np.testing.assert_allclose(cent[c], m / np.linalg.norm(m), atol=1e-12)


def test_engineered_ties_go_to_the_lower_index():
    # two identical triples: both centres have three neighbours; the lower index is visited first
    e = np.eye(6)
    V = np.stack([e[0], e[0], e[0], e[1], e[1], e[1], e[2]])
    label, centres, sizes, _ = oracle.cluster(V, 0.5)
    assert label.tolist() == [0, 0, 0, 3, 3, 3, 6] and centres.tolist() == [0, 3, 6] and sizes.tolist() == [3, 3, 1]


def test_invariants_and_limits():
    w = W.config(3, seed=5, mode="P", n_centroids=400, dim=32, n_clusters=25, sigma=0.06)
    V = w.centroids.astype(np.float64)
    theta = 0.8
    label, centres, sizes, cent = oracle.cluster(w.centroids, theta)
    S = V @ V.T
    n = len(V)
    assert sizes.sum() == n and set(label.tolist()) == set(centres.tolist())           # a partition
    assert (label[centres] == centres).all()                                            # a centre is its own member
    assert (S[np.arange(n), label][label != np.arange(n)] > theta).all()                 # members are neighbours of the centre
    Sc = S[np.ix_(centres, centres)].copy()
    np.fill_diagonal(Sc, -2)
    assert Sc.max() <= theta                                                             # no two centres are neighbours
    deg = (S > theta).sum(1) + (np.diag(S) <= theta)                                     # self counted once
    assert sizes[0] == deg.max() and centres[0] == int(np.flatnonzero(deg == deg.max())[0])
    np.testing.assert_allclose(np.linalg.norm(cent, axis=1), 1.0, atol=1e-12)
    # nothing above the threshold: everyone alone, in index order; everything above: one community around index 0
    l1, c1, s1, _ = oracle.cluster(w.centroids, 1.01, want_centroids=False)
    assert (l1 == np.arange(n)).all() and (c1 == np.arange(n)).all() and (s1 == 1).all()
    l2, c2, s2, _ = oracle.cluster(w.centroids, -1.01, want_centroids=False)
    assert (l2 == 0).all() and c2.tolist() == [0] and s2.tolist() == [n]


def test_planted_clusters_are_recovered():
    # tight clusters far apart (spread 0.06 around random unit means, dim 64): members of a cluster have cosine about
    # 0.996 with one another and about 0 +- 0.13 with the rest, so at theta_C = 0.9 the communities are the planted clusters
    w = W.config(3, seed=7, mode="T", n_centroids=600, dim=64, n_clusters=40, sigma=0.06)
    label, centres, sizes, _ = oracle.cluster(w.centroids, 0.9)
    planted = w.centroid_labels
    assert len(centres) == len(np.unique(planted))
    for v, s in zip(centres, sizes):
        members = np.flatnonzero(label == v)
        assert len(set(planted[members].tolist())) == 1 and s == (planted == planted[v]).sum()


def test_bf16_inputs_are_widened_exactly():
    w = W.config(3, seed=8, mode="P", n_centroids=150, dim=16, n_clusters=10, sigma=0.06, dtype="bf16")
    a = oracle.cluster(w.centroids, 0.85)
    b = oracle.cluster(w.centroids_f32(), 0.85)
    assert all((x == y).all() for x, y in zip(a[:3], b[:3])) and np.abs(a[3] - b[3]).max() == 0.0
