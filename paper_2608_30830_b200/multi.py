"""Multi-GPU plumbing for benchmarks: one process per GPU, rank-local pools, no data-path collective.

The path shards by request (or by KV head under tensor parallelism): every rank owns its pool, its host link and
its pinned arena, so the only exchanges are a barrier and the reduction of timings.  All ranks pin their arenas
out of the same host DRAM, which is what `fit_requests` budgets for."""
import os

import numpy as np


def env_ranks():
    """(rank, world_size, local_rank) from the launcher's environment; (0, 1, 0) when launched plainly."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def fit_requests(lengths, bytes_per_token, host_available, world_size, slack_bytes=2 << 30, fraction=0.6):
    """Scale rule: keep geometry and per-request lengths, drop requests from the end until this rank's arena fits
    in its share (`fraction` of the available host memory divided by the number of ranks).  Never drops the last one."""
    lengths = np.asarray(lengths)
    budget = int(fraction * host_available / max(world_size, 1))
    n = len(lengths)
    while n > 1 and int(lengths[:n].sum()) * bytes_per_token + slack_bytes > budget:
        n -= 1
    return n


class Group:
    """Barrier and reductions over the ranks of a benchmark job; all of them are no-ops for one rank."""

    def __init__(self, backend, device=None):
        self.rank, self.world, self.local = env_ranks()
        self.device = device
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            if not dist.is_initialized():
                kw = {"device_id": device} if (backend == "nccl" and device is not None) else {}
                dist.init_process_group(backend, **kw)
            self.dist = dist

    def _tensor(self, values):
        import torch
        return torch.tensor(list(values), dtype=torch.float64, device=self.device if self.device is not None else "cpu")

    def barrier(self):
        if self.dist:
            self.dist.barrier()

    def max(self, values):
        """Element-wise maximum over ranks (timings: the job is as slow as its slowest rank)."""
        if not self.dist:
            return [float(v) for v in values]
        t = self._tensor(values)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return t.tolist()

    def sum(self, values):
        """Element-wise sum over ranks (bytes moved by the whole job)."""
        if not self.dist:
            return [float(v) for v in values]
        t = self._tensor(values)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.SUM)
        return t.tolist()

    def close(self):
        if self.dist:
            self.dist.barrier()
            self.dist.destroy_process_group()
            self.dist = None


def job_throughput(bytes_per_rank, seconds_per_rank, group):
    """Whole-job rate: bytes of all ranks divided by the slowest rank's time."""
    total = group.sum([bytes_per_rank])[0]
    slowest = group.max([seconds_per_rank])[0]
    return total / slowest, total, slowest
