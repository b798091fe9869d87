"""Multi-GPU plumbing of the benchmark: independent replicas, no data-path collective.

The compression path runs on one GPU (the N nodes are a batch dimension), so several GPUs only
run independent replicas of the same job.  What the ranks share is the timing protocol: a barrier
on both sides of the timed region, the MAXIMUM of the per-rank device times, and the whole-job
throughput (every replica's units over that time).  The backend is NCCL on GPUs and gloo in the
CPU tests; nothing here touches the CUDA library.
"""
from __future__ import annotations

import os


def env_rank():
    """(rank, local_rank, world_size) from the torchrun environment; (0, 0, 1) when launched alone."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


class Replicas:
    def __init__(self, backend="nccl", device=None):
        import torch

        self.torch = torch
        self.rank, self.local_rank, self.world = env_rank()
        self.device = device
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist

            kwargs = {}
            if backend == "nccl" and device is not None:
                kwargs["device_id"] = torch.device(device)
            dist.init_process_group(backend, **kwargs)
            self.dist = dist

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()

    def max_over_ranks(self, value):
        """The slowest rank's figure (device milliseconds): every rank returns the same number."""
        if self.dist is None:
            return float(value)
        t = self.torch.tensor([float(value)], dtype=self.torch.float64,
                              device=self.device if self.device is not None else "cpu")
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def job_throughput(self, units_per_replica_step, ms_per_step):
        """Whole-job units per second: all replicas' units over the slowest rank's step time."""
        return self.world * units_per_replica_step / (ms_per_step * 1e-3)

    def close(self):
        if self.dist is not None:
            self.dist.destroy_process_group()
            self.dist = None
