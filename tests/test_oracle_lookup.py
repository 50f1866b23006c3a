"""Pins for the oracle's lookup: the hand-computed example, an independently written numpy
brute force (with engineered exact ties), self-queries, equivariances and the threshold rule."""
import json
import os

import numpy as np
import pytest
import torch

import oracle
from gen import workloads as W


def numpy_topk(C, Q, k, valid=None):
    """Second, independent statement: full fp64 similarity matrix, stable argsort of its negation."""
    S = Q.astype(np.float64) @ C.astype(np.float64).T
    if valid is not None:
        S = np.where(valid[None, :] != 0, S, -np.inf)
    order = np.argsort(-S, axis=1, kind="stable")[:, :k]
    return order, np.take_along_axis(S, order, 1)


def test_worked_example(golden_dir):
    g = json.load(open(os.path.join(golden_dir, "four_centroid_example.json")))
    C = np.array(g["centroids"], dtype=np.float64)
    q = np.array([g["lookup"]["query"]], dtype=np.float64)
    idx, sim, hit = oracle.lookup(C, q, 0.90, k=4)
    assert idx[0].tolist() == g["lookup"]["top4"]
    np.testing.assert_allclose(sim[0], np.array(g["lookup"]["sims"])[g["lookup"]["top4"]], atol=1e-12)
    assert hit[0] == g["lookup"]["hit_at_theta_0.90"]
    assert oracle.lookup(C, q, 0.97, k=1)[2][0] == g["lookup"]["hit_at_theta_0.97"]
    # bf16 storage of 0.6 / 0.8 (relative error up to 2^-9 per factor) moves the similarities by < 4e-3, order kept
    idx_b, sim_b, _ = oracle.lookup(W.f32_to_bf16_bits(C.astype(np.float32)),
                                    W.f32_to_bf16_bits(q.astype(np.float32)), 0.90, k=4)
    assert idx_b[0].tolist()[:3] == g["lookup"]["top4"][:3]
    assert np.abs(sim_b[0] - sim[0]).max() < 4e-3


@pytest.mark.parametrize("dtype", [np.float32, np.float64, "bf16"])
def test_matches_numpy_brute_force_with_ties(dtype):
    rng = np.random.default_rng(7)
    N, D, B, k = 61, 13, 37, 5
    # small integers: every dot product is exact in every format, ties are exact ties
    C = rng.integers(-2, 3, (N, D)).astype(np.float32)
    C[17] = C[3]
    C[40] = C[3]
    C[9] = C[55]
    Q = rng.integers(-2, 3, (B, D)).astype(np.float32)
    Q[0] = C[3]
    if dtype == "bf16":
        Cx, Qx = W.f32_to_bf16_bits(C), W.f32_to_bf16_bits(Q)
    else:
        Cx, Qx = C.astype(dtype), Q.astype(dtype)
    idx, sim, _ = oracle.lookup(Cx, Qx, 0.5, k=k)
    ref_idx, ref_sim = numpy_topk(C, Q, k)
    assert (idx == ref_idx).all()
    assert (sim == ref_sim).all()
    # the duplicate rows tie exactly and must come out in ascending slot order
    ties = [j for j in idx[0].tolist() if j in (3, 17, 40)]
    assert ties == sorted(ties) and len(ties) == 3


def test_matches_numpy_on_random_unit_vectors_and_mask():
    w = W.config(1, n_centroids=64, n_queries=50, dim=16, n_clusters=8, mode="P")
    valid = (np.random.default_rng(3).random(64) < 0.7).astype(np.uint8)
    idx, sim, hit = oracle.lookup(w.centroids, w.queries, w.theta, k=4, valid=valid)
    ref_idx, ref_sim = numpy_topk(w.centroids, w.queries, 4, valid)
    assert (idx == ref_idx).all()
    np.testing.assert_allclose(sim, ref_sim, rtol=0, atol=1e-14)
    assert (valid[idx] == 1).all()
    assert (hit == (ref_sim[:, 0] > w.theta.astype(np.float64))).all()


def test_self_query_returns_own_centroid_with_similarity_one():
    for dtype, tol in (("f32", 1e-5), ("bf16", 2e-3)):
        # dim 384: |bf16(c)|^2 deviates from 1 by about 2^-9 / sqrt(D) per unit of norm, well inside 2e-3
        w = W.config(1, n_centroids=200, n_queries=0, dim=384, n_clusters=200, mode="L", dtype=dtype)
        idx, sim, _ = oracle.lookup(w.centroids, w.centroids, 0.5, k=1)
        assert (idx[:, 0] == np.arange(200)).all()
        assert np.abs(sim[:, 0] - 1.0).max() < tol


def test_query_and_centroid_permutations():
    w = W.config(1, n_centroids=90, n_queries=40, dim=24, n_clusters=10, mode="P")
    idx, sim, hit = oracle.lookup(w.centroids, w.queries, w.theta, k=3)
    rng = np.random.default_rng(11)
    pq = rng.permutation(40)
    idx2, sim2, hit2 = oracle.lookup(w.centroids, w.queries[pq], w.theta[pq], k=3)
    assert (idx2 == idx[pq]).all() and (sim2 == sim[pq]).all() and (hit2 == hit[pq]).all()
    pc = rng.permutation(90)
    idx3, sim3, _ = oracle.lookup(w.centroids[pc], w.queries, w.theta, k=3)
    assert (pc[idx3] == idx).all()          # random unit vectors: no exact ties
    np.testing.assert_array_equal(sim3, sim)


def test_threshold_rule_is_strict_and_monotone():
    C = np.eye(6, dtype=np.float32)
    Q = np.eye(6, dtype=np.float32)[[2, 4]]
    _, sim, hit = oracle.lookup(C, Q, 1.0, k=1)
    assert (sim[:, 0] == 1.0).all() and (hit == 0).all()        # similarity exactly 1 is not > 1
    assert (oracle.lookup(C, Q, -1.0, k=1)[2] == 1).all()
    w = W.config(1, n_centroids=128, n_queries=256, dim=32, n_clusters=16, mode="P")
    prev = None
    for th in np.linspace(0.60, 0.98, 20):
        hit = oracle.lookup(w.centroids, w.queries, th, k=1)[2].astype(bool)
        if prev is not None:
            assert not (hit & ~prev).any()                      # raising theta never creates a hit
        prev = hit
    # the comparison happens against the fp32 threshold widened to fp64
    s = oracle.lookup(w.centroids, w.queries, 0.0, k=1)[1][:, 0]
    th32 = s.astype(np.float32)
    hit = oracle.lookup(w.centroids, w.queries, th32, k=1)[2]
    assert (hit == (s > th32.astype(np.float64))).all()


def test_fewer_valid_entries_than_k_and_empty_cache():
    C = np.eye(5, dtype=np.float32)
    valid = np.array([0, 1, 0, 1, 0], dtype=np.uint8)
    Q = np.array([[0.1, 0.2, 0.3, 0.9, 0.0]], dtype=np.float32)
    idx, sim, hit = oracle.lookup(C, Q, 0.5, k=4, valid=valid)
    assert idx[0].tolist() == [3, 1, -1, -1]
    assert np.isneginf(sim[0, 2:]).all() and hit[0] == 1
    idx, sim, hit = oracle.lookup(C, Q, -1.0, k=2, valid=np.zeros(5, dtype=np.uint8))
    assert idx[0].tolist() == [-1, -1] and hit[0] == 0


def test_bf16_rounding_matches_a_library_conversion_and_rounds_once():
    rng = np.random.default_rng(5)
    x32 = np.concatenate([rng.standard_normal(20000).astype(np.float32) * np.float32(0.05),
                          np.array([0.0, -0.0, 1.0, -1.0, 1e-40, -3e-39, 65504.0, 1 + 2 ** -8, 1 + 3 * 2 ** -8],
                                   dtype=np.float32)])
    ours = oracle.round_bf16(x32.astype(np.float64))
    lib = torch.from_numpy(x32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert (ours == lib).all()
    assert (ours == W.f32_to_bf16_bits(x32)).all()
    # 1 + 2^-8 + 2^-30 lies above the tie: one rounding gives 1 + 2^-7, rounding via fp32 first would give 1
    assert oracle.round_bf16(np.array([1 + 2.0 ** -8 + 2.0 ** -30]))[0] == 0x3F81
    assert oracle.round_bf16(np.array([1 + 2.0 ** -8]))[0] == 0x3F80
