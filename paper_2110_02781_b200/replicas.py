"""Plumbing for running N independent replicas of the path, one process per GPU.

The path has no exchange step between GPUs: every replica trains its own copy on its own batch, so the only
collective work is measurement: a barrier on both sides of the timed region and the maximum over ranks of the
device time.  Used by bench.py; the same code runs on CPU tensors with the gloo backend in the tests.
"""
import os


class Replicas:
    def __init__(self, backend=None, device=None):
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.device = device
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            if backend == "nccl" and device is not None:
                dist.init_process_group(backend, device_id=device)
            else:
                dist.init_process_group(backend or "gloo")
            self.dist = dist

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()

    def max_over_ranks(self, value):
        """The largest of the ranks' values (a time in ms): the job is as slow as its slowest replica."""
        if self.dist is None:
            return float(value)
        import torch
        t = torch.tensor([float(value)], dtype=torch.float64, device=self.device if self.device is not None else "cpu")
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def job_throughput(self, units_per_rank, ms):
        """Whole-job units per second: every rank processed units_per_rank units in (at most) ms milliseconds."""
        return self.world * units_per_rank / (ms * 1e-3)

    def close(self):
        if self.dist is not None:
            self.dist.destroy_process_group()
            self.dist = None
