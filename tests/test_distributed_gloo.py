"""The N > 1 path on CPU: two gloo ranks shard the rows of one batch with the library's own helper,
each runs all seven algorithms of the oracle on its block (standing in for the per-rank scans, which
need no data from other ranks), the concatenated outputs equal the single-process results bit for
bit, and the scalar reductions used by the benchmark (max of times, sum of units) agree."""
import os
import socket
import sys

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import oracle
    from paper_2608_17641_b200 import workloads
    from paper_2608_17641_b200.distributed import Dist, shard_batch
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from _util import ALL_ALGOS, run_oracle
    d = Dist.from_env(backend="gloo")
    ro = workloads.make_rollout(50, 37, 64)
    lo, hi, mine = shard_batch(ro, d.rank, d.world)
    assert mine.N == hi - lo and mine.rewards.shape == (hi - lo, ro.T) and mine.bootstrap.shape == (hi - lo,)
    assert mine.rewards.base is not None and mine.rewards.flags["C_CONTIGUOUS"]          # a view, still contiguous
    outs = run_oracle(oracle, mine, ALL_ALGOS, threads=1)
    d.barrier()
    t_max = d.max(10.0 + rank)                 # the slowest rank decides
    units = d.sum((hi - lo) * ro.T)
    q.put((rank, lo, hi, outs, t_max, units))
    d.close()


def test_two_gloo_ranks_shard_rows_without_exchange():
    sys.path.insert(0, ROOT)
    import oracle
    from paper_2608_17641_b200 import workloads
    oracle.build()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted((q.get(timeout=120) for _ in range(2)), key=lambda x: x[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from _util import ALL_ALGOS, run_oracle
    ro = workloads.make_rollout(50, 37, 64)
    full = run_oracle(oracle, ro, ALL_ALGOS, threads=1)
    assert got[0][1] == 0 and got[0][2] == got[1][1] and got[1][2] == ro.N
    for a in ALL_ALGOS:                         # every algorithm, every output, bit for bit
        parts = [g[3][a] for g in got]
        if isinstance(full[a], tuple):
            for i, want in enumerate(full[a]):
                assert np.array_equal(np.concatenate([p[i] for p in parts]), want), (a, i)
        else:
            assert np.array_equal(np.concatenate(parts), full[a]), a
    assert got[0][4] == got[1][4] == 11.0
    assert got[0][5] == got[1][5] == ro.N * ro.T


def test_shard_batch_cuts_every_row_indexed_tensor():
    """[N,T], [N], [N,T,A] and [N,T,D] tensors are cut along rows; scalars and parameters pass through."""
    from paper_2608_17641_b200.distributed import shard_batch
    N, T, A, D = 11, 5, 3, 4
    rng = np.random.default_rng(0)
    batch = dict(rewards=rng.standard_normal((N, T)), bootstrap=rng.standard_normal(N), probs=rng.random((N, T, A)),
                 x=rng.standard_normal((N, T, D)), truncs=None, gamma=0.99, params=dict(lam=0.95))
    seen = 0
    for world in (1, 2, 3):
        pieces = [shard_batch(batch, r, world) for r in range(world)]
        assert pieces[0][0] == 0 and pieces[-1][1] == N
        for k in ("rewards", "bootstrap", "probs", "x"):
            assert np.array_equal(np.concatenate([p[2][k] for p in pieces]), batch[k])
            assert all(p[2][k].flags["C_CONTIGUOUS"] for p in pieces)
        assert all(p[2]["truncs"] is None and p[2]["gamma"] == 0.99 and p[2]["params"] == dict(lam=0.95) for p in pieces)
        seen += 1
    assert seen == 3


def test_shard_rows_partition():
    from paper_2608_17641_b200.distributed import aggregate_throughput, shard_rows
    for N in (0, 1, 7, 64, 16384):
        for world in (1, 2, 3, 8):
            blocks = [shard_rows(N, r, world) for r in range(world)]
            assert blocks[0][0] == 0 and blocks[-1][1] == N
            assert all(blocks[i][1] == blocks[i + 1][0] for i in range(world - 1))
            sizes = [hi - lo for lo, hi in blocks]
            assert max(sizes) - min(sizes) <= 1
    assert aggregate_throughput([100, 100], [1.0, 2.0]) == 200 / 2e-3
