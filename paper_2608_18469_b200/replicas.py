"""Multi-GPU plumbing: one process per GPU, torch.distributed for the host-side exchanges (NCCL
on GPUs, gloo in the CPU tests).

Two ways to use N GPUs.  Independent replicas: every rank trains its own copy of the workload and the
only communication is a barrier around the timed region and a MAX over the ranks' device times.
Data-parallel replicas: the ranks train ONE model on disjoint shards of the batch; the library sums
each block's gradients over the ranks right behind that block's backward (one all-reduce per block
inside the step).  For that mode this module carries the host-side part: which rows a rank
takes, how the communicator's id reaches every rank, and how the ranks agree on one schedule (the
order of the library's exchanges depends on n_streams and flags, so every rank must pass the same)."""
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

    def broadcast_object(self, obj, src=0):
        """rank src's obj on every rank (any picklable value)."""
        if self.dist is None:
            return obj
        box = [obj if self.rank == src else None]
        self.dist.broadcast_object_list(box, src=src)
        return box[0]

    def shard(self, n_rows):
        """This rank's rows of a global batch of n_rows: equal contiguous shards, in rank order."""
        if n_rows % self.world:
            raise ValueError(f"{n_rows} rows do not split evenly over {self.world} replicas")
        per = n_rows // self.world
        return slice(self.rank * per, (self.rank + 1) * per)

    def agree_on(self, choice):
        """Every rank adopts rank 0's choice (a schedule picked by a local trial may differ per rank)."""
        return self.broadcast_object(choice, src=0)

    def attach(self, model, make_id):
        """Give `model` its data-parallel communicator: rank 0 draws the id with make_id(), every rank
        receives it, then all ranks enter the collective set-up together."""
        uid = self.broadcast_object(make_id() if self.rank == 0 else None, src=0)
        if not isinstance(uid, (bytes, bytearray)) or len(uid) != 128:
            raise ValueError("the communicator id must be 128 bytes")
        model.comm_init(self.rank, self.world, bytes(uid))
        return bytes(uid)

    def close(self):
        if self.dist is not None:
            self.dist.destroy_process_group()
            self.dist = None
