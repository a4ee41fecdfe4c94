"""One process per GPU: the rank plumbing of a multi-GPU run.

The path shards by independent problems: every rank owns a full parameter server with its own
workers and its own rows of the image pool, and no gradient or weight crosses ranks (each server
of the paper's scale experiment is one such replica group).  The only exchanges are therefore
outside the data path: a barrier on both sides of a timed region and the maximum of the ranks'
device times.  Both are here so that they can be exercised with the `gloo` backend on CPU.
"""
import os

import torch


class Ranks:
    def __init__(self, backend="nccl", device=None):
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        self.backend = backend
        self.dist = None
        self.device = device
        if self.world > 1:
            import torch.distributed as dist

            kw = {}
            if backend == "nccl":
                kw["device_id"] = torch.device("cuda", self.local)
                self.device = torch.device("cuda", self.local)
            dist.init_process_group(backend, **kw)
            self.dist = dist

    def barrier(self):
        """All ranks arrive, and this rank's device is idle, before anyone goes on."""
        if self.dist is not None:
            self.dist.barrier()
        if self.backend == "nccl" and torch.cuda.is_available():
            torch.cuda.synchronize()

    def max_over_ranks(self, v):
        """The slowest rank's time: a whole-job rate divides by this."""
        if self.dist is None:
            return float(v)
        t = torch.tensor([float(v)], dtype=torch.float64, device=self.device or "cpu")
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def batch_seed(self, t):
        """Seed of this rank's input rows at tick t; ranks draw disjoint seeds (weak scaling)."""
        return t + self.rank * 1000

    def whole_job_rate(self, units_per_rank, ms):
        """Units all ranks processed divided by the slowest rank's time (ms, already the maximum)."""
        return units_per_rank * self.world / (ms * 1e-3)

    def close(self):
        if self.dist is not None:
            self.dist.destroy_process_group()
            self.dist = None
