"""GPU parity of astra_fused_allreduce_add_rmsnorm (the all-reduce of the tensor-parallel partial
hidden states folded into add + RMSNorm) against the oracle, element by element, through the C ABI.
All partials live on the one GPU here; the kernel reads them with the same plain loads it would use
for peer-mapped memory.  The residual sum is compared bit for bit, y within the rmsnorm gate."""
import numpy as np
import pytest
import torch

import oracle
import paper_2509_07506_b200 as astra
from paper_2509_07506_b200 import workloads as wl
from parity import check_values
from test_gpu_parity import NCPU, Guarded, f64, fold, row_chunks

pytestmark = pytest.mark.gpu

BF16, FP16, FP32 = wl.BF16, wl.FP16, wl.FP32


def run_allreduce(inp: wl.AllreduceRmsnormInputs, offset=0, prepared=False):
    T, H = inp.residual.shape
    gparts = [Guarded(p, offset) for p in inp.parts]
    gr, gw = Guarded(inp.residual, offset), Guarded(inp.weight, offset)
    gy = Guarded(torch.zeros_like(inp.residual), offset)
    if prepared:
        astra.prepare_fused_allreduce_add_rmsnorm(gy.t, gr.t, [g.t for g in gparts], gw.t, inp.eps)()
    else:
        astra.astra_fused_allreduce_add_rmsnorm(gy.t, gr.t, [g.t for g in gparts], gw.t, inp.eps)
    torch.cuda.synchronize()
    for g in gparts + [gr, gw, gy]:
        g.check()
    for g, p in zip(gparts, inp.parts):
        assert torch.equal(g.host().view(torch.uint8), p.view(torch.uint8)), "a partial was modified"
    assert torch.equal(gw.host(), inp.weight)
    y, r = gy.host(), gr.host()
    stats = {}
    for sl in row_chunks(T, H):
        oy, orr = oracle.fused_allreduce_add_rmsnorm([wl.bits(p[sl]) for p in inp.parts], wl.bits(inp.residual[sl]),
                                                     wl.bits(inp.weight), inp.eps, inp.dtype, nthreads=NCPU)
        assert np.array_equal(wl.bits(r[sl]), orr), f"residual sum is not bit-exact in rows {sl.start}..{sl.stop}"
        fold(stats, check_values(f64(y[sl]), oy, inp.dtype,
                                 what=f"allreduce rmsnorm {len(inp.parts)} x {(T, H)} rows {sl.start}.."))
    return stats


@pytest.mark.parametrize("n_parts", [2, 4, 8])
@pytest.mark.parametrize("T,H", [(8192, 4096), (16, 4096), (257, 4100)])
def test_allreduce_rmsnorm_tensor_parallel_shapes(n_parts, T, H):
    stats = run_allreduce(wl.allreduce_rmsnorm_inputs(T, H, n_parts, BF16, seed=n_parts))
    assert stats["max_err_ulp"] <= 2.0


@pytest.mark.parametrize("dtype,H", [(FP16, 4096), (FP32, 2048), (BF16, 2048), (FP32, 1024)])
def test_allreduce_rmsnorm_long_streams(dtype, H):
    """From 4096 rows on, rows of 16-byte vectors with 16 units per thread take the register-capped
    instantiation of the kernel: every storage type of it, every row, against the oracle."""
    run_allreduce(wl.allreduce_rmsnorm_inputs(4096 + 5, H, 3, dtype, seed=H + 1))


@pytest.mark.parametrize("n_parts", [2, 5])
@pytest.mark.parametrize("T,H,offset", [(400, 8192, 0), (300, 16384, 0), (330, 12288, 16), (350, 1024, 0),
                                        (310, 4096, 8), (4100, 4096, 8), (320, 4100, 0)])
def test_allreduce_rmsnorm_streaming_shapes(n_parts, T, H, offset):
    """More rows than one wave.  Operands that are 32-byte aligned take 32-byte vectors (one or two per
    thread, two or four partial loads in flight, blocks of 128 to 512 threads); rows too narrow for that,
    16-byte aligned operands (offset 8; from 4096 rows on in the register-capped form) and 8-byte aligned
    rows (H = 4100) take the narrower forms."""
    run_allreduce(wl.allreduce_rmsnorm_inputs(T, H, n_parts, BF16, seed=T + n_parts), offset=offset)


@pytest.mark.parametrize("dtype", [BF16, FP16, FP32])
@pytest.mark.parametrize("n_parts", [1, 2, 3, 5, 8, 16])
def test_allreduce_rmsnorm_part_counts(dtype, n_parts):
    run_allreduce(wl.allreduce_rmsnorm_inputs(33, 5120, n_parts, dtype, seed=40 + n_parts))


@pytest.mark.parametrize("dtype", [BF16, FP32])
@pytest.mark.parametrize("n_parts", [2, 5])
@pytest.mark.parametrize("H", [1, 2, 3, 7, 8, 9, 250, 1000, 4098, 4101, 8192, 11008, 14336, 16384, 16392,
                               20500, 32768, 40000, 65538])
def test_allreduce_rmsnorm_widths(dtype, n_parts, H):
    """Every launch shape: 16-, 8-, 4- and 2-byte vectors, 1 to 8 vectors per thread, two or four
    partial loads in flight, and the two-sweep kernel for rows too wide for the registers."""
    run_allreduce(wl.allreduce_rmsnorm_inputs(5 if H < 20000 else 3, H, n_parts, dtype, seed=H))


@pytest.mark.parametrize("offset", [1, 2, 4])
@pytest.mark.parametrize("H", [4096, 4100])
def test_allreduce_rmsnorm_pointer_offsets(offset, H):
    run_allreduce(wl.allreduce_rmsnorm_inputs(7, H, 3, BF16, seed=offset), offset=offset)


@pytest.mark.parametrize("T", [64, 300, 1500])
def test_allreduce_rmsnorm_one_part_is_kernel_2(T):
    """One partial: the operation is fused_add_rmsnorm with a separate y.  The residual is identical
    bit for bit; y follows the same arithmetic but the two calls may sum a row's squares in different
    orders (different launch shapes), so both are gated against the oracle and may differ from each
    other by one unit in the last place at most."""
    inp = wl.allreduce_rmsnorm_inputs(T, 4096, 1, BF16, seed=9)
    x, r, w = inp.parts[0].cuda(), inp.residual.cuda(), inp.weight.cuda()
    y1, r1 = torch.empty_like(x), r.clone()
    astra.astra_fused_allreduce_add_rmsnorm(y1, r1, [x], w, inp.eps)
    y2, r2 = torch.empty_like(x), torch.empty_like(x)
    astra.astra_fused_add_rmsnorm_ex(y2, r2, x, r, w, inp.eps)
    assert torch.equal(r1, r2)
    oy, orr = oracle.fused_add_rmsnorm(wl.bits(inp.parts[0]), wl.bits(inp.residual), wl.bits(inp.weight), inp.eps, BF16)
    assert np.array_equal(wl.bits(r1.cpu()), orr)
    check_values(f64(y1.cpu()), oy, BF16, what="one partial")
    check_values(f64(y2.cpu()), oy, BF16, what="fused_add_rmsnorm_ex")
    steps = (wl.bits(y1.cpu()).astype(np.int32) - wl.bits(y2.cpu()).astype(np.int32))
    assert np.abs(steps).max() <= 1, "the two calls differ by more than one unit in the last place"


def test_allreduce_rmsnorm_depends_on_rank_order_as_the_oracle_does():
    """Large cancelling partials: the result depends on the order of the additions; the kernel must
    follow rank order exactly (bit-exact residual for two different orders of the same partials)."""
    T, H = 9, 4096
    g = torch.Generator().manual_seed(3)
    big = (torch.randn((T, H), generator=g) * 1000).to(torch.bfloat16)
    small = (torch.randn((T, H), generator=g) * 1e-3).to(torch.bfloat16)
    base = wl.allreduce_rmsnorm_inputs(T, H, 1, BF16, seed=1)
    for parts in ([big, -big, small], [big, small, -big], [small, big, -big]):
        run_allreduce(wl.AllreduceRmsnormInputs(parts, base.residual * 1e-3, base.weight, 1e-6, BF16))


def test_allreduce_rmsnorm_prepared_and_repeatable():
    inp = wl.allreduce_rmsnorm_inputs(700, 5120, 4, BF16, seed=77)
    a = run_allreduce(inp)
    b = run_allreduce(inp, prepared=True)
    assert a == b
    parts = [p.cuda() for p in inp.parts]
    w = inp.weight.cuda()
    ref = None
    for _ in range(6):
        y, r = torch.empty_like(parts[0]), inp.residual.cuda()
        astra.astra_fused_allreduce_add_rmsnorm(y, r, parts, w, inp.eps)
        got = (y.clone(), r.clone())
        if ref is None:
            ref = got
        assert torch.equal(ref[0], got[0]) and torch.equal(ref[1], got[1])


# ---- the two-shot form: a rank reduces its own row block and stores the results to every rank ----

def run_two_shot(inp: wl.AllreduceRmsnormInputs, world: int, rank: int, offset=0, in_place=True):
    """One rank's call of the two-shot form on one GPU: `world` full-size [T, H] destination buffers
    for y and for the residual stand for the ranks' buffers; the rank's own residual buffer (slot
    `rank`) is the residual input when in_place.  Inside the rank's row block every destination must
    hold the oracle's rows; outside it nothing may change."""
    from paper_2509_07506_b200 import multi
    T, H = inp.residual.shape
    first, count = multi.shard_rows(T, world, rank)
    sl = slice(first, first + count)
    td = inp.residual.dtype
    sentinel = torch.full((T, H), 7.0, dtype=td)
    gparts = [Guarded(p, offset) for p in inp.parts]
    gw = Guarded(inp.weight, offset)
    gys = [Guarded(sentinel, offset) for _ in range(world)]
    grs = [Guarded(inp.residual if (in_place and d == rank) else sentinel, offset) for d in range(world)]
    gin = grs[rank] if in_place else Guarded(inp.residual, offset)
    astra.astra_fused_allreduce_add_rmsnorm_ex([g.t[sl] for g in gys], [g.t[sl] for g in grs], gin.t[sl],
                                               [g.t[sl] for g in gparts], gw.t, inp.eps)
    torch.cuda.synchronize()
    for g in gparts + gys + grs + [gw, gin]:
        g.check()
    for g, p in zip(gparts, inp.parts):
        assert torch.equal(g.host().view(torch.uint8), p.view(torch.uint8)), "a partial was modified"
    if count == 0:
        oy = orr = None
    else:
        oy, orr = oracle.fused_allreduce_add_rmsnorm([wl.bits(p[sl]) for p in inp.parts], wl.bits(inp.residual[sl]),
                                                     wl.bits(inp.weight), inp.eps, inp.dtype, nthreads=NCPU)
    outside = torch.ones(T, dtype=torch.bool)
    outside[sl] = False
    stats = {}
    y0 = gys[0].host()
    for d in range(world):
        y, r = gys[d].host(), grs[d].host()
        assert torch.equal(y.view(torch.uint8), y0.view(torch.uint8)), "the y destinations differ"
        assert bool((y[outside] == 7.0).all()), "y was written outside the rank's row block"
        keep = inp.residual if (in_place and d == rank) else sentinel
        assert torch.equal(r[outside].view(torch.uint8), keep[outside].view(torch.uint8)), \
            "a residual destination was written outside the rank's row block"
        if count:
            assert np.array_equal(wl.bits(r[sl]), orr), f"destination {d}: residual sum is not bit-exact"
    if not in_place:
        assert torch.equal(gin.host().view(torch.uint8), inp.residual.view(torch.uint8)), "the residual input was modified"
    if count:
        fold(stats, check_values(f64(y0[sl]), oy, inp.dtype, what=f"two-shot rank {rank}/{world} {(T, H)}"))
    return stats


@pytest.mark.parametrize("world,rank", [(2, 1), (4, 0), (8, 5), (16, 15)])
@pytest.mark.parametrize("T,H", [(613, 4096), (64, 4100), (37, 20500)])
def test_two_shot_row_blocks(world, rank, T, H):
    stats = run_two_shot(wl.allreduce_rmsnorm_inputs(T, H, world, BF16, seed=world * 100 + rank), world, rank)
    assert stats["max_err_ulp"] <= 2.0


@pytest.mark.parametrize("dtype", [FP16, FP32])
def test_two_shot_other_storage_types_and_separate_residual_input(dtype):
    run_two_shot(wl.allreduce_rmsnorm_inputs(130, 5120, 3, dtype, seed=5), 3, 2, in_place=False)
    run_two_shot(wl.allreduce_rmsnorm_inputs(130, 5120, 3, dtype, seed=5), 3, 1, offset=2)


def test_two_shot_long_block_and_empty_block():
    """A block of 4096 rows or more takes the register-capped instantiation; a rank that is dealt no
    rows (fewer rows than ranks) launches nothing and writes nothing."""
    run_two_shot(wl.allreduce_rmsnorm_inputs(8200, 2048, 2, BF16, seed=21), 2, 1)
    run_two_shot(wl.allreduce_rmsnorm_inputs(3, 4096, 4, BF16, seed=22), 4, 3)


def test_two_shot_with_single_destinations_is_the_one_shot_call_bit_for_bit():
    inp = wl.allreduce_rmsnorm_inputs(300, 4096, 4, BF16, seed=23)
    parts, w = [p.cuda() for p in inp.parts], inp.weight.cuda()
    y1, r1 = torch.empty_like(parts[0]), inp.residual.cuda()
    astra.astra_fused_allreduce_add_rmsnorm(y1, r1, parts, w, inp.eps)
    y2, r2 = torch.empty_like(parts[0]), inp.residual.cuda()
    astra.astra_fused_allreduce_add_rmsnorm_ex([y2], [r2], r2, parts, w, inp.eps)
    assert torch.equal(y1, y2) and torch.equal(r1, r2)


def test_two_shot_all_ranks_assemble_the_whole_batch():
    """Every rank's call in turn (one GPU, so one after the other): together the row blocks fill every
    rank's buffers with the whole batch's result (the residual exactly what the one-shot call gives)."""
    world, T, H = 4, 1001, 4096
    from paper_2509_07506_b200 import multi
    inp = wl.allreduce_rmsnorm_inputs(T, H, world, BF16, seed=24)
    parts, w = [p.cuda() for p in inp.parts], inp.weight.cuda()
    y_ref, r_ref = torch.empty_like(parts[0]), inp.residual.cuda()
    astra.astra_fused_allreduce_add_rmsnorm(y_ref, r_ref, parts, w, inp.eps)
    ys = [torch.zeros_like(parts[0]) for _ in range(world)]
    rs = [inp.residual.cuda() for _ in range(world)]      # every rank holds the residual
    for rank in range(world):
        first, count = multi.shard_rows(T, world, rank)
        sl = slice(first, first + count)
        astra.astra_fused_allreduce_add_rmsnorm_ex([y[sl] for y in ys], [r[sl] for r in rs], rs[rank][sl],
                                                   [p[sl] for p in parts], w, inp.eps)
    torch.cuda.synchronize()
    # The residual is bit-exact whatever the launch shape.  y depends on the order in which a block
    # sums the squares, which differs between the launch shape of a 250-row block and that of the
    # 1001-row batch, so it is compared with the oracle (and across destinations bit for bit).
    for d in range(world):
        assert torch.equal(rs[d], r_ref) and torch.equal(ys[d], ys[0])
    oy, orr = oracle.fused_allreduce_add_rmsnorm([wl.bits(p) for p in inp.parts], wl.bits(inp.residual),
                                                 wl.bits(inp.weight), inp.eps, BF16, nthreads=NCPU)
    assert np.array_equal(wl.bits(r_ref.cpu()), orr)
    check_values(f64(ys[0].cpu()), oy, BF16, what="two-shot, assembled from four row blocks")
    check_values(f64(y_ref.cpu()), oy, BF16, what="one-shot")


def test_allreduce_rmsnorm_binding_refuses_bad_calls():
    e = lambda *shape: torch.zeros(shape, dtype=torch.bfloat16, device="cuda")  # noqa: E731
    with pytest.raises(ValueError):
        astra.astra_fused_allreduce_add_rmsnorm(e(4, 64), e(4, 64), [], e(64), 1e-6)
    with pytest.raises(ValueError):
        astra.astra_fused_allreduce_add_rmsnorm(e(4, 64), e(4, 64), [e(4, 64)] * 17, e(64), 1e-6)
    with pytest.raises(ValueError):
        astra.astra_fused_allreduce_add_rmsnorm(e(4, 64), e(4, 64), [e(4, 32)], e(64), 1e-6)
    with pytest.raises(TypeError):
        astra.astra_fused_allreduce_add_rmsnorm(e(4, 64), e(4, 64), [e(4, 64).float()], e(64), 1e-6)
    y = e(4, 64)
    with pytest.raises(astra.AstraError) as err:
        astra.astra_fused_allreduce_add_rmsnorm(y, e(4, 64), [y, e(4, 64)], e(64), 1e-6)
    assert err.value.status == 6
    with pytest.raises(ValueError):
        astra.astra_fused_allreduce_add_rmsnorm_ex([], [e(4, 64)], e(4, 64), [e(4, 64)], e(64), 1e-6)
    with pytest.raises(ValueError):
        astra.astra_fused_allreduce_add_rmsnorm_ex([e(4, 64)], [e(4, 64)] * 17, e(4, 64), [e(4, 64)], e(64), 1e-6)
    with pytest.raises(ValueError):
        astra.astra_fused_allreduce_add_rmsnorm_ex([e(4, 64)], [e(5, 64)], e(4, 64), [e(4, 64)], e(64), 1e-6)
    r = e(4, 64)
    with pytest.raises(astra.AstraError) as err:
        astra.astra_fused_allreduce_add_rmsnorm_ex([y, y], [r], r, [e(4, 64)], e(64), 1e-6)
    assert err.value.status == 6


def test_allreduce_rmsnorm_reads_partials_of_another_process(tmp_path):
    """Two ranks as two processes: each holds one partial, maps the other's through an inter-process
    memory handle, and runs the fused kernel over both; each compares with the oracle.  With one GPU
    both ranks share it (the kernel never waits on a peer; the ordering is host barriers)."""
    import os
    import sys
    from paper_2509_07506_b200 import multi
    worker = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tp_worker.py")
    rc = multi.spawn_ranks([sys.executable, worker, str(tmp_path)], 2, timeout=600)
    assert rc == 0
    assert (tmp_path / "tp_gpu_ok0").exists() and (tmp_path / "tp_gpu_ok1").exists()
