"""GPU parity of lookup (similarity sweep, top-k, threshold) against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from gen import workloads as W
from util import TOL, check_lookup, to_dev

pytestmark = pytest.mark.gpu

siso = pytest.importorskip("paper_2508_18736_b200")
PATHS = {"simt": siso.PATH_SIMT, "stream": siso.PATH_STREAM, "tensor": siso.PATH_TENSOR, "auto": siso.PATH_AUTO}


def run_lookup(w, k, path, valid=None, theta=None):
    cache = siso.SisoCache(w.centroids.shape[0], w.dim, w.dtype)
    cache.set_lookup_path(PATHS[path])
    cache.insert(to_dev(w.centroids, w.dtype))
    if valid is not None:
        st = cache.export()
        cache.import_(st["master"], st["size"], st["access"], st["last"], torch.from_numpy(valid).cuda(), 0)
    th = w.theta if theta is None else theta
    th_arg = float(th[0]) if np.all(th == th[0]) else torch.from_numpy(th).cuda()
    idx, sim, hit = cache.lookup(to_dev(w.queries, w.dtype), th_arg, k)
    cache.check_status()
    res = (idx.cpu().numpy(), sim.cpu().numpy(), hit.cpu().numpy())
    cache.close()
    return res


CASES = [
    # (config, overrides, mode, k, paths)
    (1, dict(), "T", 1, ["simt", "tensor", "auto"]),
    (1, dict(n_centroids=1000, n_queries=333, dim=384), "P", 4, ["simt", "stream", "tensor"]),
    (1, dict(n_centroids=517, n_queries=130, dim=136, n_clusters=16), "L", 8, ["simt", "stream", "tensor"]),   # k = 8: CUDA cores
    (1, dict(n_centroids=3, n_queries=5, dim=8, n_clusters=2), "L", 4, ["simt", "stream", "tensor"]),
    (1, dict(n_centroids=5000, n_queries=700, dim=768, n_clusters=300), "T", 4, ["tensor"]),       # fp32 on tensor cores
    (1, dict(n_centroids=2300, n_queries=1, dim=1024, n_clusters=100), "P", 2, ["tensor"]),
    (2, dict(n_centroids=4096 + 77, n_queries=700, dim=768, n_clusters=256), "T", 1, ["simt", "tensor", "auto"]),
    (2, dict(n_centroids=3000, n_queries=257, dim=768, n_clusters=128), "P", 1, ["simt", "tensor"]),
    (4, dict(n_centroids=8192 + 5, n_queries=300, dim=1024, n_clusters=512), "T", 4, ["simt", "tensor"]),
    (4, dict(n_centroids=2049, n_queries=129, dim=1024, n_clusters=64), "L", 4, ["simt", "tensor", "stream"]),
    (4, dict(n_centroids=999, n_queries=7, dim=1024, n_clusters=64), "P", 8, ["stream", "auto"]),
    (2, dict(n_centroids=640, n_queries=64, dim=72, n_clusters=32), "P", 2, ["simt", "tensor", "stream"]),
    # largest supported dimension, a single query, three query tiles (single-CTA tensor kernel), nine (CTA pairs + padding)
    (2, dict(n_centroids=300, n_queries=33, dim=4096, n_clusters=16), "L", 8, ["simt", "tensor", "stream"]),
    (1, dict(n_centroids=300, n_queries=9, dim=4096, n_clusters=16), "L", 4, ["simt", "stream"]),
    (4, dict(n_centroids=1500, n_queries=1, dim=1024, n_clusters=64), "P", 4, ["simt", "tensor", "stream", "auto"]),
    (2, dict(n_centroids=1111, n_queries=300, dim=768, n_clusters=64), "L", 1, ["tensor"]),
    (2, dict(n_centroids=700, n_queries=1100, dim=264, n_clusters=64), "L", 4, ["tensor", "auto"]),
]


@pytest.mark.parametrize("cfg,over,mode,k,paths", CASES)
def test_lookup_matches_oracle(cfg, over, mode, k, paths):
    w = W.config(cfg, mode=mode, k=k, **over)
    ora = oracle.lookup(w.centroids, w.queries, w.theta, k)
    for path in paths:
        gpu = run_lookup(w, k, path)
        stats = check_lookup(gpu, ora, w.centroids, w.queries, w.theta, TOL[w.dtype])
        if mode == "L":    # top-2 gaps are far above the tolerance here: the comparison must be exact
            assert stats["idx_mismatch"] == 0, (path, stats)
        # cluster-level check that never excuses: the best match comes from the oracle's cluster
        lab = w.centroid_labels
        assert (lab[gpu[0][:, 0]] == lab[ora[0][:, 0]]).all() or mode != "T"


@pytest.mark.parametrize("dtype,path", [("f32", "simt"), ("f32", "stream"), ("f32", "tensor"), ("bf16", "simt"), ("bf16", "tensor"),
                                        ("bf16", "stream")])
def test_lookup_skips_empty_slots_and_pads_short_results(dtype, path):
    w = W.config(1, n_centroids=300, n_queries=40, dim=64, n_clusters=10, mode="P", dtype=dtype)
    valid = (np.random.default_rng(1).random(300) < 0.02).astype(np.uint8)      # about 6 live entries, k = 8
    valid[:2] = 1
    k = 8
    ora = oracle.lookup(w.centroids, w.queries, w.theta, k, valid)
    gpu = run_lookup(w, k, path, valid=valid)
    check_lookup(gpu, ora, w.centroids, w.queries, w.theta, TOL[dtype], valid=valid)
    assert (gpu[0][:, -1] == -1).all()
    # an empty cache misses everything
    gpu = run_lookup(w, 2, path, valid=np.zeros(300, dtype=np.uint8))
    assert (gpu[0] == -1).all() and np.isneginf(gpu[1]).all() and (gpu[2] == 0).all()


@pytest.mark.parametrize("dtype,path", [("f32", "simt"), ("f32", "tensor"), ("bf16", "tensor"), ("bf16", "stream")])
def test_exact_ties_go_to_the_lower_slot_and_threshold_is_strict(dtype, path):
    rng = np.random.default_rng(3)
    C = rng.integers(-1, 2, (200, 64)).astype(np.float32) * 0.125          # exact in bf16, exact dot products
    C[150] = C[7]
    C[90] = C[7]
    Q = C[[7, 33, 7]].copy()
    if dtype == "bf16":
        Cx, Qx = W.f32_to_bf16_bits(C), W.f32_to_bf16_bits(Q)
    else:
        Cx, Qx = C, Q
    w = W.Workload("ties", dtype, 64, Cx, Qx, None, 4, np.zeros(200, np.int32), None, {})
    self_sim = (Q.astype(np.float64) ** 2).sum(1).astype(np.float32)
    for theta in (self_sim, np.nextafter(self_sim, np.float32(-1))):
        w.theta = theta
        ora = oracle.lookup(Cx, Qx, theta, 4)
        gpu = run_lookup(w, 4, path)
        assert (gpu[0] == ora[0]).all() and (gpu[1] == ora[1].astype(np.float32)).all() and (gpu[2] == ora[2]).all()
    assert gpu[0][0, :3].tolist() == [7, 90, 150] and gpu[2].tolist() == [1, 1, 1]


def test_fp32_tensor_path_rescans_queries_it_cannot_settle():
    """The fp32 tensor-core path accepts its answer only if the k-th exact similarity clears the 8th approximate one by a
    margin.  With a dozen identical rows inside one tile that never happens: those queries must come out of the exact scan, ties to the
    lower slot; the other queries are settled by the rescoring."""
    w = W.config(1, n_centroids=900, n_queries=200, dim=72, n_clusters=40, mode="P")
    C = w.centroids.copy()
    dup = [5, 17, 30, 31, 100, 101, 120, 130, 140, 150, 160, 170]         # all in the first tile of 256 rows
    C[dup] = C[5]
    Q = w.queries.copy()
    Q[:50] = C[5]                                             # 50 queries whose 12 best rows tie exactly
    w2 = W.Workload("ties", "f32", 72, C, Q, w.theta, 4, w.centroid_labels, None, {})
    ora = oracle.lookup(C, Q, w.theta, 4)
    gpu = run_lookup(w2, 4, "tensor")
    check_lookup(gpu, ora, C, Q, w.theta, TOL["f32"])
    assert (gpu[0][:50] == np.array(dup[:4])).all()
    simt = run_lookup(w2, 4, "simt")
    assert (simt[0] == gpu[0]).all() and (simt[2] == gpu[2]).all()


def test_fp32_tensor_path_sees_every_change_of_the_vectors():
    """The fp32 tensor-core path keeps the bf16 parts of the centroids between calls; every entry point that writes
    vectors must make it split them again."""
    w = W.config(1, n_centroids=600, n_queries=64, dim=72, n_clusters=30, mode="P")
    cache = siso.SisoCache(700, 72, "f32")
    ora = oracle.OracleCache(700, 72, "f32")
    cache.set_lookup_path(siso.PATH_TENSOR)
    cache.insert(to_dev(w.centroids[:500], "f32"))
    ora.insert(w.centroids[:500])
    q, theta = to_dev(w.queries, "f32"), np.full(64, 0.85, np.float32)

    def same(what):
        got = [x.cpu().numpy() for x in cache.lookup(q, 0.85, 2)]
        check_lookup(got, ora.lookup(w.queries, theta, 2), ora.lookup_copy(), w.queries, theta, TOL["f32"], valid=ora.valid)
        return got

    same("after the first insert")
    cache.insert(to_dev(w.centroids[500:], "f32"))                       # insert
    ora.insert(w.centroids[500:])
    same("after a second insert")
    idx, sim, hit = cache.lookup(q, 0.85, 1)                              # running-mean update of the hit rows
    cache.update(q, idx, hit)
    ora.update(w.queries, idx.cpu().numpy(), hit.cpu().numpy())
    got = same("after an update")
    assert hit.cpu().numpy().sum() > 0
    mm, n = cache.merge(0.9, siso.MERGE_WEIGHTED_MEAN)                     # merge moves vectors and empties slots
    ora.merge(0.9, True)
    same("after a merge")
    st = cache.export()                                                   # import replaces everything
    rolled = torch.roll(st["master"], 1, dims=0)
    cache.import_(rolled, st["size"], st["access"], st["last"], st["valid"], 5)
    ora.load_state(rolled.cpu().numpy(), st["size"].cpu().numpy(), st["access"].cpu().numpy().view(np.uint32),
                   st["last"].cpu().numpy().view(np.uint64), st["valid"].cpu().numpy(), 5)
    same("after an import")
    cache.close()


def test_scratch_regrowth_on_a_side_stream_matches_oracle():
    """Lookups of growing size on a stream that is not torch's current one: every growth replaces the handle's scratch
    and staging buffers while kernels of the earlier calls are still queued.  Tensors allocated and overwritten on the
    current stream right after each call would land in a block that was handed back too early."""
    w = W.config(2, n_centroids=6000, n_queries=1500, dim=768, n_clusters=128, mode="P")
    cache = siso.SisoCache(6000, 768, "bf16")
    cache.insert(to_dev(w.centroids, "bf16"))
    torch.cuda.synchronize()
    q_all, th_all = to_dev(w.queries, "bf16"), torch.from_numpy(w.theta).cuda()
    side = torch.cuda.Stream()
    results, junk = [], []
    for n in (4, 130, 700, 1500, 9):
        side.wait_stream(torch.cuda.current_stream())
        results.append((n, cache.lookup(q_all[:n], th_all[:n], 4, stream=side)))
        junk.append([torch.full((1 << 22,), 255, dtype=torch.uint8, device="cuda") for _ in range(6)])
    side.synchronize()
    torch.cuda.synchronize()
    assert cache.sync_status(side) == 0
    for n, (idx, sim, hit) in results:
        ora = oracle.lookup(w.centroids, w.queries[:n], w.theta[:n], 4)
        check_lookup((idx.cpu().numpy(), sim.cpu().numpy(), hit.cpu().numpy()), ora, w.centroids, w.queries[:n],
                     w.theta[:n], TOL["bf16"])
    cache.close()


def test_a_device_wait_that_runs_out_reports_timeout_and_the_handle_stays_usable():
    """Every wait inside the tensor-core kernels is bounded.  Here the kernels' own wait routine polls a barrier that
    nothing arrives on (no copy, no tensor-core operation in flight) until its limit runs out: the status word must say
    SISO_ERR_TIMEOUT once, the kernel must have returned normally, and the next lookup must be right."""
    w = W.config(2, n_centroids=1500, n_queries=200, dim=768, n_clusters=64, mode="P")
    cache = siso.SisoCache(1500, 768, "bf16")
    cache.insert(to_dev(w.centroids, "bf16"))
    cache.check_status()
    flag = cache.selftest_wait_timeout(2048)
    assert cache.sync_status() == 6                      # SISO_ERR_TIMEOUT
    assert flag.item() == 1
    assert cache.sync_status() == 0                      # reported once, then clear
    with pytest.raises(siso.SisoError):
        cache.selftest_wait_timeout(0)
    cache.set_lookup_path(siso.PATH_TENSOR)
    idx, sim, hit = cache.lookup(to_dev(w.queries, "bf16"), torch.from_numpy(w.theta).cuda(), 4)
    check_lookup((idx.cpu().numpy(), sim.cpu().numpy(), hit.cpu().numpy()),
                 oracle.lookup(w.centroids, w.queries, w.theta, 4), w.centroids, w.queries, w.theta, TOL["bf16"])
    cache.check_status()
    tf = cache.measure_fp32_fma()
    assert 20.0 < tf < 120.0, tf                         # 148 SMs x 128 lanes x 2 flop x 1.0-2.0 GHz
    cache.close()


def test_bad_arguments_return_status_and_touch_nothing():
    cache = siso.SisoCache(64, 64, "bf16")
    q = torch.zeros(4, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(siso.SisoError):
        cache.lookup(q, 0.5, k=0)
    with pytest.raises(siso.SisoError):
        cache.lookup(q, 0.5, k=9)
    with pytest.raises(ValueError):
        cache.lookup(torch.zeros(4, 32, dtype=torch.bfloat16, device="cuda"), 0.5)
    with pytest.raises(siso.SisoError):
        siso.SisoCache(64, 60, "bf16")            # dim must be a multiple of 8
    cache.insert(torch.zeros(65, 64, dtype=torch.bfloat16, device="cuda"))      # more rows than slots
    assert cache.sync_status() == 4 and cache.sync_status() == 0               # SISO_ERR_CAPACITY, then cleared
    assert cache.stats()["occupancy"] == 0
    cache.close()
