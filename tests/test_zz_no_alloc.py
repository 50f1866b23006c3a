"""The allocation-free small-batch lookup against the ordinary lookup.

Some users of the library call it from places where the CUDA allocator is off limits (a serving loop
with all device memory handed out at start-up, a callback under an allocator lock).  For them the
library has one entry point whose scratch is a fixed array inside the library image.  This test calls
it through the C ABI twice in a row on different inputs - the shared scratch still holds the first
call's partial results when the second runs - and checks both results against siso_lookup and against
the CPU oracle, checks that the calls leave the amount of allocated device memory unchanged, then checks
that sizes beyond the fixed limits are refused.  It is collected last on purpose."""
import numpy as np
import pytest
import torch

from gen import workloads as W
import oracle
from util import TOL, check_lookup, to_dev

pytestmark = pytest.mark.gpu

siso = pytest.importorskip("paper_2508_18736_b200")


@pytest.mark.parametrize("dtype,dim,shift", [("bf16", 768, 0), ("f32", 384, 0), ("bf16", 768, 4)])
def test_no_alloc_lookup_matches_ordinary_lookup_twice_in_a_row(dtype, dim, shift):
    cfg = 2 if dtype == "bf16" else 1
    w = W.config(cfg, n_centroids=5003, n_queries=16, dim=dim, n_clusters=200, mode="P", dtype=dtype)
    cent, q_all = to_dev(w.centroids, dtype), to_dev(w.queries, dtype)
    valid = torch.ones(5003, dtype=torch.uint8, device="cuda")
    valid[::7] = 0
    cache = siso.SisoCache(5003, dim, dtype)
    cache.insert(cent)
    st = cache.export()
    cache.import_(st["master"], st["size"], st["access"], st["last"], valid, 0)
    cache.set_lookup_path(siso.PATH_STREAM)
    if shift:       # a matrix that does not start on a 16-byte boundary: the kernel's scalar loads instead of 128-bit ones
        buf = torch.empty(cent.numel() + shift, dtype=cent.dtype, device="cuda")
        buf[shift:].copy_(cent.reshape(-1))
        cent = buf[shift:].view(cent.shape)
        assert cent.data_ptr() % 16 != 0
    theta_all = torch.from_numpy(w.theta).cuda()
    tol = TOL[dtype]
    # two calls in a row: 8 queries with k = 4, then 5 other queries with k = 8 and a scalar threshold
    for (lo, n, k, use_vec) in ((0, 8, 4, True), (8, 5, 8, False)):
        q = q_all[lo:lo + n].contiguous()
        theta = theta_all[lo:lo + n].contiguous() if use_vec else 0.86
        want_idx, want_sim, want_hit = cache.lookup(q, theta, k)
        idx = torch.full((n, k), -7, dtype=torch.int32, device="cuda")
        sim = torch.zeros((n, k), dtype=torch.float32, device="cuda")
        hit = torch.full((n,), 9, dtype=torch.uint8, device="cuda")
        torch.cuda.synchronize()
        free_before, held_before = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
        siso.lookup_small_noalloc(cent, q, theta, k, idx, sim, hit, valid=valid)
        torch.cuda.synchronize()
        if lo > 0:        # the first call on a device may still load the library's kernels; the second changes nothing
            assert torch.cuda.mem_get_info()[0] == free_before and torch.cuda.memory_allocated() == held_before
        th_np = w.theta[lo:lo + n] if use_vec else np.full(n, 0.86, np.float32)
        ora = oracle.lookup(w.centroids, w.queries[lo:lo + n], th_np, k, valid.cpu().numpy())
        check_lookup((idx.cpu().numpy(), sim.cpu().numpy(), hit.cpu().numpy()), ora, w.centroids, w.queries[lo:lo + n],
                     th_np, tol, valid=valid.cpu().numpy())
        assert (sim - want_sim).abs().max().item() <= tol
        gap_ok = (want_sim[:, :-1] - want_sim[:, 1:]).min(dim=1).values >= tol     # rows without near-ties
        assert torch.equal(idx[gap_ok], want_idx[gap_ok])
        th = theta if use_vec else torch.full((n,), 0.86, device="cuda")
        clear = (want_sim[:, 0] - th).abs() >= tol
        assert torch.equal(hit[clear], want_hit[clear])
        assert (valid[idx.long().flatten()] == 1).all()
    cache.close()


def test_no_alloc_lookup_refuses_sizes_beyond_its_fixed_scratch():
    cent = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    out = (torch.zeros(9, 1, dtype=torch.int32, device="cuda"), torch.zeros(9, 1, dtype=torch.float32, device="cuda"),
           torch.zeros(9, dtype=torch.uint8, device="cuda"))
    with pytest.raises(siso.SisoError) as e:       # nine queries: one more than the scratch array holds
        siso.lookup_small_noalloc(cent, torch.zeros(9, 64, dtype=torch.bfloat16, device="cuda"), 0.5, 1, *out)
    assert e.value.status == 2
    wide = torch.zeros(8, 2048, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(siso.SisoError) as e:       # dim beyond the stated maximum
        siso.lookup_small_noalloc(wide, wide[:2].contiguous(), 0.5, 1, out[0][:2], out[1][:2], out[2][:2])
    assert e.value.status == 2
    with pytest.raises(siso.SisoError):            # k beyond the list length kept per query
        siso.lookup_small_noalloc(cent, cent[:2].contiguous(), 0.5, 9, out[0], out[1], out[2])
