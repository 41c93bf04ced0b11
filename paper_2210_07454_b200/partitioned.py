"""One optimiser iteration with the workers partitioned over several processes (one GPU each).

Every process holds a handle for its own workers and a replica of x.  Algorithms 1 and 2 couple the workers only
through sums: the mean sketch, the mean gradient on I_{t-1} and the mean exact values of the selected candidates,
which are the |S| + k + P*k floats per iteration that Section III-B counts.  The iteration is therefore three calls
into the library with one all-reduce (sum) between each pair; this module holds the two exchange buffers and does
the all-reduces through ``torch.distributed`` (NCCL between GPUs).  No arithmetic of the method happens here.
"""
import torch


class PartitionedStep:
    """Drives ``step_local`` / ``step_select`` / ``step_finish`` of a handle (``binding.SketchedAMSGrad`` created with
    ``workers_total`` = the number of workers over all processes) with the two sums in between.

    all_reduce: callable(tensor) that replaces the tensor by its sum over the processes and gives every process the
    same bits; default ``torch.distributed.all_reduce`` on ``group``.  With a single process it is the identity."""

    def __init__(self, handle, device, group=None, all_reduce=None):
        self.handle = handle
        self.exchange1 = torch.zeros(handle.exchange_floats(1), dtype=torch.float32, device=device)
        self.exchange2 = torch.zeros(handle.exchange_floats(2), dtype=torch.float32, device=device)
        if all_reduce is None:
            import torch.distributed as dist

            def all_reduce(t):
                if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
                    dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
        self.all_reduce = all_reduce

    def step(self, grads, x) -> None:
        """grads: this process's workers' gradients (n_local * d float32); x: this process's replica, in place."""
        h = self.handle
        h.step_local(grads, self.exchange1)
        self.all_reduce(self.exchange1)
        h.step_select(self.exchange1, self.exchange2)
        self.all_reduce(self.exchange2)
        h.step_finish(self.exchange2, x)

    @property
    def floats_per_step(self) -> int:
        """What one process contributes to the exchange per iteration (Section III-B's communication count)."""
        return self.exchange1.numel() + self.exchange2.numel()
