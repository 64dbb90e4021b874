"""The N > 1 path on CPU: two gloo ranks shard the rows of one batch, each runs the oracle on its
block (standing in for the per-rank scan, which needs no data from other ranks), and the scalar
reductions used by the benchmark (max of times, sum of units) agree with a single-process run."""
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
    from paper_2608_17641_b200.distributed import Dist, shard_rows
    d = Dist.from_env(backend="gloo")
    ro = workloads.make_rollout(50, 37, 64)
    lo, hi = shard_rows(ro.N, d.rank, d.world)
    adv, _ = oracle.gae(ro.rewards[lo:hi], ro.values[lo:hi], ro.dones[lo:hi], ro.truncs[lo:hi],
                        ro.trunc_bootstrap[lo:hi], ro.bootstrap[lo:hi], gamma=0.99, lam=0.95)
    d.barrier()
    t_max = d.max(10.0 + rank)                 # the slowest rank decides
    units = d.sum((hi - lo) * ro.T)
    q.put((rank, lo, hi, adv, t_max, units))
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
    ro = workloads.make_rollout(50, 37, 64)
    full, _ = oracle.gae(ro.rewards, ro.values, ro.dones, ro.truncs, ro.trunc_bootstrap, ro.bootstrap, gamma=0.99, lam=0.95)
    assert got[0][1] == 0 and got[0][2] == got[1][1] and got[1][2] == ro.N
    assert np.array_equal(np.concatenate([got[0][3], got[1][3]]), full)
    assert got[0][4] == got[1][4] == 11.0
    assert got[0][5] == got[1][5] == ro.N * ro.T


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
