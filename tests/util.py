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


STRICT = 1e-5        # what the kernels really achieve: bf16 products are exact and the sums are fp32 (error about 2e-6)


def check_lookup(gpu, ora, centroids, queries, theta, tol, valid=None, strict=STRICT):
    """gpu / ora = (idx, sim, hit) as numpy.  Asserts the rules above and returns the three numbers that say how
    hard they bit:
      outside_band    index or hit decisions that differ where the oracle's own margin is at least `tol` (must be 0);
      excused         decisions that differ inside the band (the GPU's choice is checked to be within tol of the best);
      strict_mismatch decisions that differ although the oracle's margin is at least `strict` = 1e-5, far below the
                      bf16 band (must be 0 as well: the stated band is much wider than the kernels' error, and a wrong
                      neighbour picked inside it would otherwise pass)."""
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
    # indices: a differing slot must be a live one whose true similarity is within the band of the oracle's
    mism = have & (gi != oi)
    outside = strict_bad = 0
    for b, j in zip(*np.nonzero(mism)):
        g = int(gi[b, j])
        assert valid is None or valid[g], "GPU returned an empty slot"
        short = float(osim[b, j]) - float(Q64[b] @ C64[g])        # how far the GPU's slot falls short of the rank's best
        outside += short > tol
        strict_bad += short > strict
    for b in np.unique(np.nonzero(mism)[0]):
        row = gi[b][gi[b] >= 0]
        assert len(set(row.tolist())) == len(row), "duplicate slot in a top-k row"
    # hit flags
    hm = gh != oh
    margin = np.abs(osim[:, 0] - theta)
    outside += int((margin[hm] >= tol).sum())
    strict_bad += int((margin[hm] >= strict).sum())
    out = dict(rows=int(B), outside_band=int(outside), excused=int(mism.sum() + hm.sum()),
               excused_rows_frac=float((mism.any(1) | hm).mean()) if B else 0.0, strict_mismatch=int(strict_bad),
               idx_mismatch=int(mism.sum()), hit_mismatch=int(hm.sum()), max_sim_err=float(err.max(initial=0.0)))
    assert outside == 0, f"decisions differ outside the band of {tol}: {out}"
    assert strict_bad == 0, f"decisions differ where the oracle's margin exceeds {strict}: {out}"
    return out


def verify_merge_map(entry, valid0, seed, sizes0, mm, theta_c, tol=1e-5):
    """Is `mm` a valid outcome of MergeCentroids (Algorithm 1) when every comparison may be off by `tol`?
    entry = the vectors as at the call (fp64), valid0 / seed = live entries and the members of C_cur (uint8),
    mm = merge map under test (slot -> surviving slot, own slot for survivors, -1 for empty slots).
    Follows the map's own survivor set, so a legitimately flipped decision and everything that follows from it
    are accepted, and nothing else is.  Returns the expected cluster_size of every slot."""
    n = len(mm)
    S = entry @ entry.T
    order = [i for i in range(n) if valid0[i] and seed[i]] + [i for i in range(n) if valid0[i] and not seed[i]]
    c_new, size, member = [], np.array(sizes0, dtype=np.float64).copy(), set()
    for i in order:
        if seed[i]:
            assert mm[i] == i, f"slot {i} of C_cur was merged away"
            c_new.append(i)
            member.add(i)
            continue
        best = S[i, c_new].max() if c_new else -np.inf
        if mm[i] == i:
            assert best <= theta_c + tol, f"slot {i} survives although a survivor is {best} similar"
            c_new.append(i)
            member.add(i)
        else:
            t = int(mm[i])
            assert t in member, f"slot {i} merged into {t}, which is not an earlier survivor"
            assert S[i, t] > theta_c - tol and S[i, t] >= best - tol, f"slot {i} -> {t}: {S[i, t]} against best {best}"
            size[t] += sizes0[i]
    assert all(mm[i] == -1 for i in range(n) if not valid0[i])
    return size
