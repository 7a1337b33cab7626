"""Process plumbing for running N independent replicas of the path, one process per GPU.

The path never exchanges data between GPUs (every move is encoded and decoded on one device), so
N > 1 means N replicas of the same job.  The only cross-rank traffic is timing bookkeeping:
a barrier around the timed region and a max-reduction of the measured durations.  The backend is
NCCL on GPUs and gloo in the CPU tests; nothing here touches the data path.
"""
from __future__ import annotations

import os


def rank_env() -> tuple[int, int, int]:
    """(rank, local_rank, world_size) as a launcher exports them; (0, 0, 1) when run alone."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


class Replicas:
    """One rank's view of the replica group."""

    def __init__(self, backend: str = "nccl", device=None):
        self.rank, self.local_rank, self.world = rank_env()
        self.device = device
        self._dist = None
        if self.world > 1:
            import torch.distributed as dist
            kw = {"device_id": device} if (backend == "nccl" and device is not None) else {}
            dist.init_process_group(backend, **kw)
            self._dist = dist

    def barrier(self) -> None:
        if self._dist is not None:
            self._dist.barrier()
        if self.device is not None and getattr(self.device, "type", "cpu") == "cuda":
            import torch
            torch.cuda.synchronize(self.device)

    def max_over_ranks(self, x: float) -> float:
        """The slowest rank's figure: a replica job is as slow as its slowest member."""
        if self._dist is None:
            return float(x)
        import torch
        t = torch.tensor([x], dtype=torch.float64, device=self.device if self.device is not None else "cpu")
        self._dist.all_reduce(t, op=self._dist.ReduceOp.MAX)
        return float(t.item())

    def aggregate_gbs(self, bytes_per_rank: int, ms_per_step: float) -> float:
        """Whole-job throughput: every rank moved bytes_per_rank in the (max) step time."""
        return self.world * bytes_per_rank / (ms_per_step * 1e-3) / 1e9

    def close(self) -> None:
        if self._dist is not None:
            self._dist.destroy_process_group()
            self._dist = None
