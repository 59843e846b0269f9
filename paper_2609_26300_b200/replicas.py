"""Replica plumbing for runs on several GPUs of one node.

The decode path does not shard: every (sequence, KV head) is independent and each rank runs the whole workload on
its own GPU.  All that crosses ranks is a barrier around the timed region and the maximum of the per-rank timings,
through torch.distributed (NCCL on GPUs, gloo in the CPU tests).  No data-path collective exists.
"""
from __future__ import annotations

import os
from typing import List, Optional, Sequence

import torch


class Replicas:
    def __init__(self, backend: Optional[str] = None, device: Optional[torch.device] = None):
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.device = device
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            backend = backend or ("nccl" if device is not None and device.type == "cuda" else "gloo")
            kwargs = {"device_id": device} if backend == "nccl" and device is not None else {}
            dist.init_process_group(backend, **kwargs)
            self.dist = dist

    def barrier(self) -> None:
        if self.dist is not None:
            self.dist.barrier()

    def max_over_ranks(self, values: Sequence[float]) -> List[float]:
        """Element-wise maximum over ranks (time-like quantities: the slowest rank sets the job's time)."""
        t = torch.tensor(list(values), dtype=torch.float64, device=self.device if self.device is not None else "cpu")
        if self.dist is not None:
            self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return [float(x) for x in t.tolist()]

    def aggregate_tokens_per_s(self, batch_per_rank: int, us_per_step: float) -> float:
        """Whole-job decode throughput: every rank decodes `batch_per_rank` tokens per step (weak scaling)."""
        return self.world * batch_per_rank / (us_per_step * 1e-6)

    def close(self) -> None:
        if self.dist is not None:
            self.dist.destroy_process_group()
            self.dist = None
