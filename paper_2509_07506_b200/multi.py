"""Host-side helpers for running on several GPUs, one process per GPU.

All three operations are independent per row (per token), so a batch is sharded by contiguous row
blocks and every rank works on its own block with no collective on the data path.  The only
communication is the timing reduction (max over ranks) that a benchmark or a scheduler needs.
"""
from __future__ import annotations

import os
from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


def shard_rows(total_rows: int, world: int, rank: int) -> Tuple[int, int]:
    """(first_row, row_count) of `rank`'s contiguous block; blocks differ by at most one row,
    cover [0, total_rows) exactly once, and are empty only when there are fewer rows than ranks."""
    if world < 1 or not 0 <= rank < world or total_rows < 0:
        raise ValueError("bad sharding arguments")
    base, extra = divmod(total_rows, world)
    count = base + (1 if rank < extra else 0)
    first = rank * base + min(rank, extra)
    return first, count


def env_rank_world() -> Tuple[int, int, int]:
    """(rank, world_size, local_rank) from the torchrun environment; (0, 1, 0) when absent."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init_process_group(backend: str, device: torch.device | None = None) -> None:
    """Rendezvous over 127.0.0.1 unless MASTER_ADDR says otherwise."""
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29500")
    if backend == "nccl" and device is not None:
        dist.init_process_group(backend, device_id=device)
    else:
        dist.init_process_group(backend)


def max_over_ranks(values: Sequence[float], device: torch.device | str = "cpu") -> List[float]:
    """Elementwise maximum of `values` over all ranks (identity without a process group)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def aggregate_rate(units_per_rank_per_step: float, world: int, steps: int, elapsed_ms: float) -> float:
    """Whole-job rate: units all ranks processed in `steps` steps divided by the (max-over-ranks) time."""
    return world * units_per_rank_per_step * steps / (elapsed_ms * 1e-3)


# ---------------------------------------------------------------------------------------------
# starting the ranks of one node without torchrun
# ---------------------------------------------------------------------------------------------

def free_port() -> int:
    import socket
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(argv: Sequence[str], world: int, timeout: float | None = None) -> int:
    """Run `argv` (a full command line) as `world` processes of one node, one per rank, with the
    environment a launcher would give them (RANK, LOCAL_RANK, WORLD_SIZE, MASTER_ADDR = 127.0.0.1 and
    a free MASTER_PORT).  Standard output and error of every rank pass through to this process's.
    Returns the largest exit code; if a rank fails the others are terminated (they would otherwise
    wait for it in their next collective)."""
    import subprocess
    import time
    if world < 1:
        raise ValueError("world must be at least 1")
    port = free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen(list(argv), env=env))
    deadline = None if timeout is None else time.time() + timeout
    worst = 0
    pending = set(range(world))
    while pending:
        for rank in sorted(pending):
            rc = procs[rank].poll()
            if rc is None:
                continue
            pending.discard(rank)
            worst = max(worst, abs(rc))
            if rc != 0:  # the others cannot finish without it
                for other in pending:
                    procs[other].terminate()
        if deadline is not None and time.time() > deadline:
            for other in pending:
                procs[other].terminate()
            worst = max(worst, 124)
            deadline = None
        if pending:
            time.sleep(0.05)
    return worst


# ---------------------------------------------------------------------------------------------
# tensor-parallel partial hidden states: who reads what in astra_fused_allreduce_add_rmsnorm
# ---------------------------------------------------------------------------------------------

def exchange_partials(local, export, open_remote, group=None) -> list:
    """Every rank of a tensor-parallel group holds one partial hidden state; the fused all-reduce
    kernel of each rank needs all of them, in rank order.  `export(local)` turns this rank's buffer
    into a picklable handle (for CUDA memory: an inter-process memory handle), the handles are
    all-gathered over the process group, and `open_remote(handle, owner_rank)` maps every other
    rank's buffer into this process.  Returns the list of buffers indexed by rank, with this rank's
    own buffer (not a re-opened copy of it) in its own slot.  Both callables are injected so that the
    ordering logic is independent of the memory system underneath."""
    if not (dist.is_available() and dist.is_initialized()):
        return [local]
    world, rank = dist.get_world_size(group), dist.get_rank(group)
    handles = [None] * world
    dist.all_gather_object(handles, export(local), group=group)
    return [local if owner == rank else open_remote(handles[owner], owner) for owner in range(world)]


def exchange_buffers(local, export, open_remote, group=None) -> list:
    """The same exchange for any per-rank buffer: the two-shot form of the fused all-reduce
    (astra_fused_allreduce_add_rmsnorm_ex) needs every rank's output buffers as well, because each rank
    stores its block of normalised rows (and of the new residual) into all of them."""
    return exchange_partials(local, export, open_remote, group)


def row_block_of_rank(total_rows: int, group=None) -> Tuple[int, int]:
    """The contiguous row block of the [total_rows, H] hidden state that this rank reduces and
    normalises (reading that block from all N partials): (first_row, row_count).  Used two ways: with
    sequence-parallel consumers the rank keeps the block for itself; in the two-shot form it stores
    the block into every rank's buffers, so that all ranks end up with all rows while each element
    crosses the links once as a partial and once as a result."""
    if not (dist.is_available() and dist.is_initialized()):
        return 0, total_rows
    return shard_rows(total_rows, dist.get_world_size(group), dist.get_rank(group))


def export_cuda_tensor(t: torch.Tensor):
    """`export` for exchange_partials when the partial is a CUDA tensor and the ranks are processes of
    one node: an inter-process memory handle in torch's picklable form.  The tensor must stay alive
    (and unchanged) for as long as any rank may read it."""
    from torch.multiprocessing.reductions import reduce_tensor
    return reduce_tensor(t)


def open_cuda_tensor(handle, owner: int) -> torch.Tensor:
    """`open_remote` for exchange_partials: maps the owner's buffer into this process and returns a
    tensor over it (no copy).  Reading it is ordinary device memory access through the mapping."""
    rebuild, args = handle
    return rebuild(*args)


class PeerEvents:
    """Stream ordering between the ranks of one node without synchronising any host with its GPU.

    The fused all-reduce kernels wait for nothing on the device; the caller must order them after
    every rank's partial has been written (and, in the two-shot form, order the consumers after every
    rank's stores).  Each rank owns one inter-process CUDA event; the handles are exchanged once.
    A phase then goes: every rank enqueues its producer work and calls ``record()``; the ranks meet
    at a host barrier (``barrier()``: hosts only, the GPUs keep running); every rank calls
    ``wait_for_all()``, which makes its stream wait for all ranks' recorded events, and enqueues the
    consumer.  The host barrier is what guarantees that each ``wait_for_all`` sees the peers' events
    already recorded: a stream wait on an event captures the event's most recent record at the time
    of the call, and a wait on an event that was never recorded returns at once.  Nothing here spins
    on the device: the waits are stream dependencies resolved by the driver."""

    def __init__(self, device: torch.device, group=None):
        self.device = device
        self.group = group
        self.mine = torch.cuda.Event(enable_timing=False, interprocess=True)
        if dist.is_available() and dist.is_initialized():
            self.rank, world = dist.get_rank(group), dist.get_world_size(group)
            with torch.cuda.device(device):
                handle = self.mine.ipc_handle()
            handles = [None] * world
            dist.all_gather_object(handles, handle, group=group)
            self.events = [self.mine if owner == self.rank else torch.cuda.Event.from_ipc_handle(device, handles[owner])
                           for owner in range(world)]
        else:
            self.rank, self.events = 0, [self.mine]

    def record(self, stream: torch.cuda.Stream | None = None) -> None:
        """Mark the point in `stream` (default: the current stream) that the peers will wait for."""
        self.mine.record(stream if stream is not None else torch.cuda.current_stream(self.device))

    def barrier(self) -> None:
        """Host-only meeting point between ``record`` and ``wait_for_all`` (no GPU synchronisation)."""
        if dist.is_available() and dist.is_initialized():
            dist.barrier(group=self.group)

    def wait_for_all(self, stream: torch.cuda.Stream | None = None) -> None:
        """Order everything enqueued on `stream` from here on after every rank's recorded event."""
        stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        for ev in self.events:
            stream.wait_event(ev)

    def phase(self, stream: torch.cuda.Stream | None = None) -> None:
        """record, host barrier, wait for all: one complete ordering step."""
        self.record(stream)
        self.barrier()
        self.wait_for_all(stream)
