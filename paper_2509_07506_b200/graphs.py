"""Replaying a fixed sequence of calls from a CUDA graph.

For decode-sized batches every call of this library is bound by launch cost, not by the GPU: a
prepared call costs 2.5-3 us of host time for 1-2 us of device time.  A sequence of prepared
calls on fixed tensors (a layer's add+norm, activation and merge, say) can be captured once into a
CUDA graph and replayed with a single launch; the kernels keep their programmatic-dependent-launch
edges inside the graph, so each one's prologue (and its L2 prefetch) overlaps the previous one's tail.
torch's graph object is used for capture and replay: device plumbing, no arithmetic.
"""
from __future__ import annotations

from typing import Optional, Sequence

import torch

from .binding import PreparedCall


class CapturedCalls:
    """``CapturedCalls([call_a, call_b, ...])`` runs the prepared calls once eagerly on a side stream
    (so that lazy initialisation happens outside the capture), then captures them in order;
    ``replay()`` re-issues the whole sequence on the current stream with one launch.  The tensors the
    calls were prepared on are the graph's inputs and outputs.  The eager warm-up run has already
    executed every call once when the constructor returns (in-place calls such as fused_add_rmsnorm
    have then modified their operands), so fill the inputs after constructing, and refill them in
    place between replays."""

    def __init__(self, calls: Sequence[PreparedCall], device: Optional[torch.device] = None):
        self.calls = list(calls)
        if not self.calls:
            raise ValueError("at least one prepared call is needed")
        self.device = device if device is not None else torch.device("cuda", torch.cuda.current_device())
        side = torch.cuda.Stream(self.device)
        side.wait_stream(torch.cuda.current_stream(self.device))
        with torch.cuda.stream(side):
            for call in self.calls:       # warm-up outside the capture
                call(side)
            side.synchronize()
            self.graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(self.graph, stream=side):
                for call in self.calls:
                    call(side)
        torch.cuda.current_stream(self.device).wait_stream(side)

    def replay(self) -> None:
        self.graph.replay()
