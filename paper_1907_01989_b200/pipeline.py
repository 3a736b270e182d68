"""Host-buffer pipeline around one bound executable: copies of the next batch overlap the kernels of
the current one.

`gi_run` takes device buffers; a caller whose images live in (pinned) host memory pays a host-to-device
copy per batch.  Run back to back on one stream, copy and kernels add up; here the copy goes to a second
stream into one of two device input buffers, so that a step costs max(copy, kernels) instead of their sum.
Only argument marshalling, streams and events: every arithmetic step still runs in the library's kernels.
"""
from __future__ import annotations

from typing import List, Sequence


class HostPipeline:
    """Two-slot software pipeline: H2D on a copy stream, gi_run + D2H on the compute stream."""

    def __init__(self, ex, input_shapes: Sequence[Sequence[int]], output_shapes: Sequence[Sequence[int]], dtype, device="cuda:0",
                 slots: int = 2, graphs: bool = False):
        """graphs: capture each slot's gi_run once as a CUDA graph (its device buffers never change) and replay
        it per batch: one launch instead of one per kernel.  Falls back to plain launches if capture fails
        (`self.graphs` then stays empty)."""
        import torch
        self.torch = torch
        self.ex = ex
        self.slots = slots
        self.compute = torch.cuda.current_stream(device)
        self.copy = torch.cuda.Stream(device)
        self.ins = [[torch.empty(tuple(s), dtype=dtype, device=device) for s in input_shapes] for _ in range(slots)]
        self.outs = [[torch.empty(tuple(s), dtype=dtype, device=device) for s in output_shapes] for _ in range(slots)]
        self.loaded = [torch.cuda.Event() for _ in range(slots)]   # slot's inputs have arrived
        self.free = [torch.cuda.Event() for _ in range(slots)]     # slot's kernels and read-back are done
        self.used = [False] * slots
        self.n = 0
        self.graphs = []
        if graphs:
            try:
                side = torch.cuda.Stream(device)
                side.wait_stream(self.compute)
                caught = []
                with torch.cuda.stream(side):
                    for s in range(slots):
                        self.ex.run(self.ins[s], self.outs[s], side)  # warm-up: attributes, tensor maps
                    side.synchronize()
                    for s in range(slots):
                        cg = torch.cuda.CUDAGraph()
                        with torch.cuda.graph(cg, stream=side):
                            self.ex.run(self.ins[s], self.outs[s], torch.cuda.current_stream(device))
                        caught.append(cg)
                self.compute.wait_stream(side)
                torch.cuda.synchronize(device)
                self.graphs = caught
            except Exception:  # capture is an optimisation, never a requirement
                self.graphs = []

    def submit(self, host_inputs: Sequence, host_outputs: Sequence) -> None:
        """Enqueue one batch: pinned host tensors in, pinned host tensors out.  Asynchronous; results are
        complete after `synchronize()` (or after the compute stream reaches a later event)."""
        torch = self.torch
        s = self.n % self.slots
        self.n += 1
        with torch.cuda.stream(self.copy):
            if self.used[s]:
                self.copy.wait_event(self.free[s])  # the batch that used this slot before has finished
            for d, h in zip(self.ins[s], host_inputs):
                d.copy_(h, non_blocking=True)
            self.loaded[s].record(self.copy)
        self.compute.wait_event(self.loaded[s])
        with torch.cuda.stream(self.compute):
            if self.graphs:
                self.graphs[s].replay()
            else:
                self.ex.run(self.ins[s], self.outs[s], self.compute)
            for h, d in zip(host_outputs, self.outs[s]):
                h.copy_(d, non_blocking=True)
            self.free[s].record(self.compute)
        self.used[s] = True

    def synchronize(self) -> None:
        self.compute.synchronize()
        self.copy.synchronize()

    def device_buffers(self) -> List:
        return self.ins
