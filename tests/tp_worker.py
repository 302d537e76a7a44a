"""One rank of the two-process check of astra_fused_allreduce_add_rmsnorm with partials that live in
ANOTHER PROCESS's device memory (mapped through an inter-process handle), started by
test_gpu_allreduce.py through multi.spawn_ranks.  With one GPU in the machine both ranks use it: the
kernel has no device-side wait, the ordering is two host barriers, so nothing here depends on the
two ranks' kernels running at the same time.  The two-shot form is checked the same way: each rank
stores its row block into the other rank's mapped output buffers.  Writes <outdir>/tp_gpu_ok<rank> on success."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

import oracle  # noqa: E402
import paper_2509_07506_b200 as astra  # noqa: E402
from paper_2509_07506_b200 import multi  # noqa: E402
from paper_2509_07506_b200 import workloads as wl  # noqa: E402
from parity import check_values  # noqa: E402


def main() -> int:
    out_dir = sys.argv[1]
    rank, world, local = multi.env_rank_world()
    dev = torch.device("cuda", local % torch.cuda.device_count())
    torch.cuda.set_device(dev)
    multi.init_process_group("gloo")
    try:
        T, H = 600, 4096
        inp = wl.allreduce_rmsnorm_inputs(T, H, world, wl.BF16, seed=11)   # same seed: every rank knows all partials
        mine = inp.parts[rank].to(dev)
        r, w = inp.residual.to(dev), inp.weight.to(dev)
        y = torch.empty_like(mine)
        torch.cuda.synchronize()
        parts = multi.exchange_partials(mine, multi.export_cuda_tensor, multi.open_cuda_tensor)
        assert len(parts) == world and parts[rank] is mine
        dist.barrier()                      # every partial is written before any rank reads
        first, count = multi.row_block_of_rank(T)
        # whole batch (as a tensor-parallel consumer needs it) ...
        astra.astra_fused_allreduce_add_rmsnorm(y, r, parts, w, inp.eps)
        # ... and this rank's own row block only (as a sequence-parallel consumer needs it)
        sl = slice(first, first + count)
        y2, r2 = torch.empty_like(mine[sl]), inp.residual[sl].to(dev)
        astra.astra_fused_allreduce_add_rmsnorm(y2, r2, [p[sl] for p in parts], w, inp.eps)
        torch.cuda.synchronize()
        dist.barrier()                      # nobody releases its partial while a peer may still read it
        oy, orr = oracle.fused_allreduce_add_rmsnorm([wl.bits(p) for p in inp.parts], wl.bits(inp.residual),
                                                     wl.bits(inp.weight), inp.eps, wl.BF16, nthreads=4)
        assert np.array_equal(wl.bits(r.cpu()), orr), "residual sum is not bit-exact"
        check_values(y.cpu().to(torch.float64).numpy(), oy, wl.BF16, what=f"rank {rank}: y")
        assert np.array_equal(wl.bits(r2.cpu()), orr[sl]) and torch.equal(y2, y[sl])
        for owner in range(world):          # the mapped partials are the owners' bytes
            assert torch.equal(parts[owner].cpu(), inp.parts[owner])
        # Two-shot form: every rank reduces its own row block and STORES the results into every rank's
        # buffers (its own directly, the other rank's through the mapping).
        y_all, r_all = torch.zeros_like(mine), inp.residual.to(dev)
        torch.cuda.synchronize()
        ys = multi.exchange_buffers(y_all, multi.export_cuda_tensor, multi.open_cuda_tensor)
        rs = multi.exchange_buffers(r_all, multi.export_cuda_tensor, multi.open_cuda_tensor)
        assert ys[rank] is y_all and rs[rank] is r_all
        dist.barrier()                      # every buffer exists and holds its initial contents
        astra.astra_fused_allreduce_add_rmsnorm_ex([b[sl] for b in ys], [b[sl] for b in rs], r_all[sl],
                                                   [p[sl] for p in parts], w, inp.eps)
        torch.cuda.synchronize()
        dist.barrier()                      # every rank's stores have landed before anyone reads its buffers
        assert np.array_equal(wl.bits(r_all.cpu()), orr), "two-shot: the assembled residual is not bit-exact"
        check_values(y_all.cpu().to(torch.float64).numpy(), oy, wl.BF16, what=f"rank {rank}: two-shot y")
        # The same two steps ordered by inter-process events instead of host synchronisation: the
        # partial is produced by a kernel on the stream, the ranks' streams wait for one another's
        # events, and no host waits for its GPU until the results are read back.
        ev_written, ev_read = multi.PeerEvents(dev), multi.PeerEvents(dev)
        for rep in range(3):
            # new partials every repetition (the oracle gets the same bits): a stale read would show
            scaled = [(p.to(torch.float32) * float(rep + 2)).to(p.dtype) for p in inp.parts]
            mine.copy_(scaled[rank])
            r_all.copy_(inp.residual)
            y_all.zero_()
            ev_written.phase()              # every rank's partial (and reset buffers) precede every rank's kernel
            astra.astra_fused_allreduce_add_rmsnorm_ex([b[sl] for b in ys], [b[sl] for b in rs], r_all[sl],
                                                       [p[sl] for p in parts], w, inp.eps)
            ev_read.phase()                 # every rank's kernel precedes any reuse of partials and any read of results
            got_y, got_r = y_all.cpu(), r_all.cpu()      # stream-ordered copies: they follow the waits above
            oy3, orr3 = oracle.fused_allreduce_add_rmsnorm([wl.bits(p) for p in scaled], wl.bits(inp.residual),
                                                           wl.bits(inp.weight), inp.eps, wl.BF16, nthreads=4)
            assert np.array_equal(wl.bits(got_r), orr3), f"event-ordered two-shot, repetition {rep}: residual not bit-exact"
            check_values(got_y.to(torch.float64).numpy(), oy3, wl.BF16, what=f"rank {rank}: event-ordered two-shot y")
        torch.cuda.synchronize()
        del parts, ys, rs, ev_written, ev_read
        dist.barrier()
        with open(os.path.join(out_dir, f"tp_gpu_ok{rank}"), "w") as fh:
            fh.write("ok")
    finally:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
