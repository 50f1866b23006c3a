"""Host side of the centroid-sharded lookup with two gloo ranks on CPU: which rows a rank holds, the all-gather of the
packed keys into the [query, rank, k] layout, and that combining the gathered lists gives every rank the same global
answer.  The device kernels are not involved: a numpy statement of the key order stands in for them here."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def pack(sim: np.ndarray, slot: np.ndarray) -> np.ndarray:
    """(order-preserving fp32 bits << 32) | (2^32 - 1 - slot): larger = more similar, ties to the lower slot."""
    u = sim.astype(np.float32).view(np.uint32).astype(np.uint64)
    s = np.where(u >> np.uint64(31) != 0, ~u & np.uint64(0xFFFFFFFF), u | np.uint64(0x80000000))
    return (s << np.uint64(32)) | (np.uint64(0xFFFFFFFF) - slot.astype(np.uint64))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2508_18736_b200 import sharded
    total, D, B, k = 37, 8, 6, 3
    rng = np.random.default_rng(0)                                   # the same data on every rank
    C = rng.standard_normal((total, D)); C /= np.linalg.norm(C, axis=1, keepdims=True)
    Q = rng.standard_normal((B, D)); Q /= np.linalg.norm(Q, axis=1, keepdims=True)
    C[20] = C[3]                                                     # an exact tie across the two shards
    per = sharded.shard_rows(total, world)
    lo, hi = sharded.local_range(rank, total, per)
    S = (Q @ C[lo:hi].T).astype(np.float32)
    order = np.lexsort((np.broadcast_to(np.arange(hi - lo), S.shape), -S), axis=1)[:, :k]
    keys = pack(np.take_along_axis(S, order, 1), order + lo)
    gathered = sharded.gather_keys(torch.from_numpy(keys.view(np.int64)))
    g = gathered.numpy().view(np.uint64).reshape(B, world * k)
    best = np.sort(g, axis=1)[:, ::-1][:, :k]
    idx = (np.uint64(0xFFFFFFFF) - (best & np.uint64(0xFFFFFFFF))).astype(np.int64)
    out[rank] = (lo, hi, tuple(gathered.shape), idx.tolist(), [sharded.owner_of(int(i), per) for i in idx[:, 0]])
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_gather_and_agree_on_the_global_top_k():
    world = 2
    port = 31500 + os.getpid() % 2000
    with mp.get_context("spawn").Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert (res[0][0], res[0][1], res[1][0], res[1][1]) == (0, 19, 19, 37)        # 37 rows: 19 + 18
    assert res[0][2] == res[1][2] == (6, 2, 3)
    assert res[0][3] == res[1][3]                                                    # every rank has the same answer
    # and it is the answer of one process over all rows (ties to the lower global slot)
    rng = np.random.default_rng(0)
    C = rng.standard_normal((37, 8)); C /= np.linalg.norm(C, axis=1, keepdims=True)
    Q = rng.standard_normal((6, 8)); Q /= np.linalg.norm(Q, axis=1, keepdims=True)
    C[20] = C[3]
    S = (Q @ C.T).astype(np.float32)
    want = np.lexsort((np.broadcast_to(np.arange(37), S.shape), -S), axis=1)[:, :3]
    assert res[0][3] == want.tolist()
    assert res[0][4] == [(int(i) // 19, int(i) % 19) for i in want[:, 0]]


def _toy_steps(rank, value):
    """A sharded operation in the library's form: a generator that yields its exchanges."""
    all_v = yield ("gather", torch.tensor([value, rank], dtype=torch.int64))
    top = yield ("max", torch.tensor([value * 2, -rank], dtype=torch.int64))
    return all_v.tolist(), top.tolist()


def _worker_run(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2508_18736_b200 import sharded
    out[rank] = sharded.run(_toy_steps(rank, 10 + rank))
    dist.barrier()
    dist.destroy_process_group()


def test_the_two_drivers_of_a_sharded_operation_agree():
    """run() does the exchanges with torch.distributed (two gloo ranks), run_lockstep() by stacking inside one process:
    both must hand every shard the same gathered and reduced tensors."""
    world = 2
    port = 33500 + os.getpid() % 2000
    with mp.get_context("spawn").Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker_run, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    sys.path.insert(0, ROOT)
    from paper_2508_18736_b200 import sharded
    want = ([[10, 0], [11, 1]], [22, 0])
    assert res[0] == want and res[1] == want
    assert sharded.run_lockstep([_toy_steps(r, 10 + r) for r in range(2)]) == [want, want]
    # without a process group the world is this process alone
    assert sharded.run(_toy_steps(0, 5)) == ([[5, 0]], [10, 0])

    def nothing_to_do():
        return 7
        yield

    assert sharded.run(nothing_to_do()) == 7 and sharded.run_lockstep([nothing_to_do(), nothing_to_do()]) == [7, 7]


def _ring_steps(rank, world):
    """The exchange pattern of the sharded MergeCentroids: about world / 2 ring steps, each unordered pair of blocks
    assigned to exactly one of its owners."""
    block = torch.full((3,), float(rank))
    swept = []
    for t in range(1, world // 2 + 1):
        peer = yield ("ring", block, t)
        s = (rank - t) % world
        assert peer.tolist() == [float(s)] * 3, "the ring delivered another rank's block"
        if (2 * t < world) or (2 * t == world and rank < s):
            swept.append((rank, s))
    pairs = yield ("gather", torch.tensor(swept + [(-1, -1)] * (world - len(swept)), dtype=torch.int64))
    return pairs.reshape(-1, 2).tolist()


def _worker_ring(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2508_18736_b200 import sharded
    out[rank] = sharded.run(_ring_steps(rank, world))
    dist.barrier()
    dist.destroy_process_group()


def test_ring_exchange_delivers_every_pair_of_blocks_to_exactly_one_owner():
    sys.path.insert(0, ROOT)
    from paper_2508_18736_b200 import sharded
    for world in (2, 3, 4, 5, 8):                       # in one process
        res = sharded.run_lockstep([_ring_steps(r, world) for r in range(world)])
        pairs = sorted(tuple(sorted(p)) for p in res[0] if p[0] >= 0)
        assert pairs == [(a, b) for a in range(world) for b in range(a + 1, world)], world
        assert all(r == res[0] for r in res)
    world = 3                                           # and over torch.distributed (gloo, three processes)
    port = 35500 + os.getpid() % 2000
    with mp.get_context("spawn").Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker_ring, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    pairs = sorted(tuple(sorted(p)) for p in res[0] if p[0] >= 0)
    assert pairs == [(0, 1), (0, 2), (1, 2)] and res[0] == res[1] == res[2]
