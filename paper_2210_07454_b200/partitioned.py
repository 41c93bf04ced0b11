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
    same bits; default ``torch.distributed.all_reduce`` on ``group``.  With a single process it is the identity.
    stream: a ``torch.cuda.Stream`` the handle is to launch on (installed with ``set_stream``); default: whatever stream
    the handle already uses.

    The library's phases run on the handle's stream; the collective is enqueued relative to torch's CURRENT stream.
    The two are ordered explicitly with events in both directions around every all-reduce, so the result does not
    depend on the two streams being the same one."""

    def __init__(self, handle, device, group=None, all_reduce=None, stream=None):
        self.handle = handle
        self.device = torch.device(device)
        if stream is not None:
            handle.set_stream(stream.cuda_stream)
        self._stream = stream
        self.exchange1 = torch.zeros(handle.exchange_floats(1), dtype=torch.float32, device=device)
        self.exchange2 = torch.zeros(handle.exchange_floats(2), dtype=torch.float32, device=device)
        if all_reduce is None:
            import torch.distributed as dist

            def all_reduce(t):
                if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
                    dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
        self.all_reduce = all_reduce

    def _handle_stream(self):
        if self._stream is not None:
            return self._stream
        ptr = getattr(self.handle, "stream_ptr", 0)
        return torch.cuda.ExternalStream(ptr, device=self.device) if ptr else torch.cuda.default_stream(self.device)

    def _reduce_between_phases(self, buf, hs) -> None:
        """all-reduce of `buf` after the phase that filled it (on hs) and before the phase that reads it (on hs)."""
        if self.device.type != "cuda":             # host stand-ins (tests on CPU): nothing to order
            self.all_reduce(buf)
            return
        cs = torch.cuda.current_stream(self.device)
        done = torch.cuda.Event()
        done.record(hs)
        cs.wait_event(done)                        # the collective sees the phase's output
        self.all_reduce(buf)
        reduced = torch.cuda.Event()
        reduced.record(cs)
        hs.wait_event(reduced)                     # the next phase sees the sum

    def step(self, grads, x) -> None:
        """grads: this process's workers' gradients (n_local * d float32); x: this process's replica, in place."""
        h = self.handle
        hs = self._handle_stream() if self.device.type == "cuda" else None
        if hs is not None:                         # inputs produced on torch's current stream
            ready = torch.cuda.Event()
            ready.record(torch.cuda.current_stream(self.device))
            hs.wait_event(ready)
        h.step_local(grads, self.exchange1)
        self._reduce_between_phases(self.exchange1, hs)
        h.step_select(self.exchange1, self.exchange2)
        self._reduce_between_phases(self.exchange2, hs)
        h.step_finish(self.exchange2, x)
        if hs is not None:                         # x is ready for work queued on torch's current stream
            finished = torch.cuda.Event()
            finished.record(hs)
            torch.cuda.current_stream(self.device).wait_event(finished)

    @property
    def floats_per_step(self) -> int:
        """What one process contributes to the exchange per iteration (Section III-B's communication count)."""
        return self.exchange1.numel() + self.exchange2.numel()
