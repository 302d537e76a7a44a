"""Pipelined processing of host-resident batches.

The three operations are independent per row, so a batch that lives in (pinned) host memory can be
cut into row chunks that are uploaded, processed and downloaded concurrently: uploads on one stream
(one copy engine), kernels on a second, downloads on a third (the other copy engine), chained by
events.  The interconnect is full duplex, so the steady state costs max(upload, download) per batch
instead of their sum.
"""
from __future__ import annotations

from typing import Callable, Dict, Hashable, Iterable, Tuple

import torch


class HostStreamer:
    """Upload -> compute -> download pipeline over three CUDA streams.

    ``submit(key, uploads, call, downloads)`` enqueues one chunk: ``uploads`` and ``downloads`` are
    (destination, source) tensor pairs copied with ``copy_(non_blocking=True)`` (host tensors
    should be pinned), ``call`` launches the kernel(s) on the current stream.  ``key`` names the
    device buffers the chunk uses: a later chunk with the same key does not start uploading before
    the earlier one has finished downloading, so device buffers can be reused across batches.
    Nothing blocks the host; call ``synchronize()`` before reading the host results.
    """

    def __init__(self, device: torch.device):
        self.device = device
        self.up = torch.cuda.Stream(device)
        self.compute = torch.cuda.Stream(device)
        self.down = torch.cuda.Stream(device)
        self._free_after: Dict[Hashable, torch.cuda.Event] = {}

    def submit(self, key: Hashable, uploads: Iterable[Tuple[torch.Tensor, torch.Tensor]],
               call: Callable[[], None], downloads: Iterable[Tuple[torch.Tensor, torch.Tensor]]) -> None:
        prev = self._free_after.get(key)
        with torch.cuda.stream(self.up):
            if prev is not None:
                self.up.wait_event(prev)
            for dst, src in uploads:
                dst.copy_(src, non_blocking=True)
            uploaded = torch.cuda.Event()
            uploaded.record(self.up)
        with torch.cuda.stream(self.compute):
            self.compute.wait_event(uploaded)
            call()
            computed = torch.cuda.Event()
            computed.record(self.compute)
        with torch.cuda.stream(self.down):
            self.down.wait_event(computed)
            for dst, src in downloads:
                dst.copy_(src, non_blocking=True)
            downloaded = torch.cuda.Event()
            downloaded.record(self.down)
        self._free_after[key] = downloaded

    def wait_for(self, stream: torch.cuda.Stream) -> None:
        """Make all three pipeline streams wait for work already enqueued on `stream`."""
        ev = torch.cuda.Event()
        ev.record(stream)
        for s in (self.up, self.compute, self.down):
            s.wait_event(ev)

    def synchronize(self) -> None:
        self.up.synchronize()
        self.compute.synchronize()
        self.down.synchronize()
