"""Shared helpers of the GPU parity tests: tensor conversion and the comparison rules.

Rules (absolute tolerance tol = 1e-5 for fp32 inputs, 2e-3 for bf16 inputs):
  * similarities agree within tol;
  * indices, hit flags, merge targets and eviction order are bit-exact, except where the oracle's own
    numbers say the decision is closer than tol (top-2 gap, or |similarity - threshold|): there the GPU's
    choice must still be a valid one (its true similarity within tol of the oracle's).
"""
import numpy as np
import torch

TOL = {"f32": 1e-5, "bf16": 2e-3}


def to_dev(a: np.ndarray, dtype: str) -> torch.Tensor:
    """numpy fp32 array or uint16 bf16 bit patterns -> CUDA tensor of the cache dtype."""
    if dtype == "bf16":
        assert a.dtype == np.uint16
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    assert a.dtype == np.float32
    return torch.from_numpy(a).cuda()


def widen64(a: np.ndarray) -> np.ndarray:
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    return a.astype(np.float64)


def check_lookup(gpu, ora, centroids, queries, theta, tol, valid=None, strict_tol=None):
    """gpu / ora = (idx, sim, hit) as numpy.  Returns a dict of counts; asserts the rules."""
    gi, gs, gh = gpu
    oi, osim, oh = ora
    B, k = oi.shape
    assert gi.shape == oi.shape and gs.shape == osim.shape and gh.shape == oh.shape
    C64, Q64 = widen64(centroids), widen64(queries)
    theta = np.broadcast_to(np.asarray(theta, dtype=np.float32), (B,)).astype(np.float64)
    have = oi >= 0
    assert ((gi >= 0) == have).all(), "number of returned entries differs"
    assert np.isneginf(gs[~have]).all()
    # similarities
    err = np.abs(gs[have].astype(np.float64) - osim[have])
    assert err.max(initial=0.0) <= tol, f"similarity error {err.max()} > {tol}"
    # indices
    mism = have & (gi != oi)
    excused = 0
    for b, j in zip(*np.nonzero(mism)):
        g = int(gi[b, j])
        assert valid is None or valid[g], "GPU returned an empty slot"
        true_sim = float(Q64[b] @ C64[g])
        assert true_sim >= osim[b, j] - tol, f"row {b} rank {j}: slot {g} is not within {tol} of the best"
        excused += 1
    for b in np.unique(np.nonzero(mism)[0]):
        row = gi[b][gi[b] >= 0]
        assert len(set(row.tolist())) == len(row), "duplicate slot in a top-k row"
    # hit flags
    hm = gh != oh
    margin = np.abs(osim[:, 0] - theta)
    assert (margin[hm] < tol).all(), "hit flag differs outside the excused band"
    out = dict(idx_mismatch=int(mism.sum()), hit_mismatch=int(hm.sum()), max_sim_err=float(err.max(initial=0.0)))
    if strict_tol is not None:
        # diagnostic: how many rows would still differ under a much tighter band
        gap_ok = np.ones(B, dtype=bool)
        out["idx_mismatch_rows"] = int(mism.any(1).sum())
    return out
