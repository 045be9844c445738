"""Replica plumbing for runs on several GPUs of one node.

The SSD layer has no cross-GPU step: (batch, head group) pairs are independent, so N GPUs run N
independent replicas (weak scaling).  torch.distributed is used for exactly two things, both outside
the data path: a barrier around the timed region and the maximum of a per-rank timing.  The same
code runs on the `gloo` backend (CPU) in the tests and on `nccl` in bench.py.
"""
import os

import torch


class Replicas:
    """rank/world bookkeeping + barrier + max-over-ranks; a no-op group when world == 1."""

    def __init__(self, backend=None, device=None):
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.device = device
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            if not dist.is_initialized():
                kw = {}
                if backend == "nccl" and device is not None:
                    kw["device_id"] = device
                dist.init_process_group(backend or "gloo", **kw)
            self.dist = dist

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()
        if self.device is not None and self.device.type == "cuda":
            torch.cuda.synchronize(self.device)

    def max_over_ranks(self, value: float) -> float:
        if self.dist is None:
            return float(value)
        dev = self.device if (self.device is not None and self.device.type == "cuda") else torch.device("cpu")
        t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def whole_job_rate(self, units_per_rank: float, seconds_this_rank: float) -> float:
        """Aggregate throughput of all replicas: every rank processed `units_per_rank` units and the job
        took as long as its slowest rank."""
        return self.world * units_per_rank / self.max_over_ranks(seconds_this_rank)

    def close(self):
        if self.dist is not None and self.dist.is_initialized():
            self.dist.destroy_process_group()
            self.dist = None
