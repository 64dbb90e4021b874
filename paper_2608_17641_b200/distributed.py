"""Multi-GPU plumbing: one process per GPU, rows (environments) are independent, so ranks share no
data -- each scans its own batch (or its own contiguous block of rows) and the only communication
is the barrier around the timed region and a max / sum of scalars.  No collective on the data path.
"""
from __future__ import annotations

import os


def shard_rows(N: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous, balanced block of rows [lo, hi) owned by `rank` (blocks differ by at most one row)."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    base, extra = divmod(N, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def shard_batch(batch, rank: int, world: int, num_envs: int | None = None):
    """This rank's block of rows of every tensor of one host (or device) batch.

    `batch` is a mapping name -> array/tensor, or an object whose public attributes are arrays (a
    workloads.Rollout); entries that are None, scalars or dicts pass through.  Every array whose
    leading dimension is num_envs -- [N, T] rollout tensors, the [N] window-edge bootstrap, [N, T, A]
    action tensors, [N, T, D] trace inputs -- is cut to rows [lo, hi) of shard_rows(); the cut is a
    view (no copy) and stays contiguous because rows are the slowest axis.  Returns (lo, hi, shard)
    with `shard` of the same kind as `batch` (dict, or a shallow copy of the object with N updated).
    Rows are independent in every algorithm of the library, so the per-rank results concatenated
    in rank order are the results of the whole batch, bit for bit, with no exchange between ranks."""
    import copy
    is_map = isinstance(batch, dict)
    items = dict(batch) if is_map else {k: v for k, v in vars(batch).items() if not k.startswith("_")}
    if num_envs is None:
        num_envs = items.get("N") if not is_map else None
        if num_envs is None:
            num_envs = next(v.shape[0] for v in items.values() if hasattr(v, "shape") and len(v.shape) >= 2)
    lo, hi = shard_rows(int(num_envs), rank, world)
    cut = lambda v: v[lo:hi] if hasattr(v, "shape") and len(v.shape) >= 1 and v.shape[0] == num_envs else v
    out = {k: cut(v) for k, v in items.items()}
    if is_map:
        return lo, hi, out
    shard = copy.copy(batch)
    for k, v in out.items():
        setattr(shard, k, v)
    if hasattr(shard, "N"):
        shard.N = hi - lo
    return lo, hi, shard


def aggregate_throughput(units_per_rank: list[int], ms_per_rank: list[float]) -> float:
    """Whole-job units per second: all units divided by the slowest rank's time."""
    return sum(units_per_rank) / (max(ms_per_rank) * 1e-3)


class Dist:
    """Thin wrapper over torch.distributed for scalar reductions and barriers."""

    def __init__(self, backend: str, device=None):
        import torch
        import torch.distributed as dist
        self.torch, self.dist, self.device = torch, dist, device
        if not dist.is_initialized():
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            dist.init_process_group(backend=backend)
        self.rank, self.world = dist.get_rank(), dist.get_world_size()

    @classmethod
    def from_env(cls, backend: str = "nccl", device=None) -> "Dist":
        return cls(backend, device)

    def _scalar(self, x: float):
        dev = self.device if self.device is not None else "cpu"
        return self.torch.tensor([float(x)], dtype=self.torch.float64, device=dev)

    def barrier(self):
        if self.device is not None and self.device.type == "cuda":
            self.dist.barrier(device_ids=[self.device.index])
        else:
            self.dist.barrier()

    def max(self, x: float) -> float:
        t = self._scalar(x)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def sum(self, x: float) -> float:
        t = self._scalar(x)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.SUM)
        return float(t.item())

    def close(self):
        if self.dist.is_initialized():
            self.dist.destroy_process_group()
