"""Multi-GPU plumbing of the benchmark.  The training step has no exchange between GPUs on this
path (every block's parameters and batch live on one device), so N GPUs run N independent
replicas of the workload ("replicas only"): the only communication is a barrier around the timed
region and a MAX over the ranks' device times.  torch.distributed provides both (NCCL on GPUs,
gloo in the CPU tests)."""
import os


class Replicas:
    def __init__(self, backend=None, device=None):
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.dist = None
        self.device = device
        if self.world > 1:
            import torch.distributed as dist
            kw = {}
            if backend == "nccl":
                import torch
                kw["device_id"] = torch.device("cuda", self.local_rank)
            dist.init_process_group(backend, **kw)
            self.dist = dist

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()

    def max_over_ranks(self, value):
        """The slowest rank's time: what the whole job waited for."""
        if self.dist is None:
            return float(value)
        import torch
        t = torch.tensor([float(value)], dtype=torch.float64, device=self.device or "cpu")
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def whole_job_rate(self, units_per_rank_step, steps, local_ms):
        """Units all ranks processed divided by the slowest rank's time (weak scaling)."""
        ms = self.max_over_ranks(local_ms)
        return self.world * units_per_rank_step * steps / (ms * 1e-3), ms

    def close(self):
        if self.dist is not None:
            self.dist.destroy_process_group()
            self.dist = None
