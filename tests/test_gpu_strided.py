"""GPU parity of the strided / out-of-place entry points against the fp64 oracle.

The operands are slices of wider device buffers filled with a pattern; the oracle sees the
gathered contiguous copies, and everything outside the slices must keep the pattern."""
import numpy as np
import pytest
import torch

import oracle
import paper_2509_07506_b200 as astra
from paper_2509_07506_b200 import workloads as wl
from parity import check_lse, check_values, merge_floor

pytestmark = pytest.mark.gpu

BF16, FP16 = wl.BF16, wl.FP16
PATTERN = -7.75  # exactly representable in both storage types


def f64(t):
    return t.to(torch.float64).numpy()


def pitched(host: torch.Tensor, pitch: int, col0: int):
    """Device buffer [rows, pitch] filled with PATTERN, with `host` (2-D) copied into columns
    [col0, col0 + width).  Returns (buffer, view)."""
    rows, width = host.shape
    buf = torch.full((rows, pitch), PATTERN, dtype=host.dtype, device="cuda")
    view = buf[:, col0:col0 + width]
    view.copy_(host)
    return buf, view


def untouched(buf, col0, width):
    mask = torch.ones(buf.shape[-1], dtype=torch.bool, device=buf.device)
    mask[col0:col0 + width] = False
    return bool((buf[..., mask] == PATTERN).all())


@pytest.mark.parametrize("dtype", [BF16, FP16])
@pytest.mark.parametrize("H,pitch,col0", [(4096, 4096 + 64, 0), (4096, 8192, 4096), (4100, 4100 + 12, 4),
                                          (520, 777, 3), (8192, 8192 + 8, 8), (24576, 24576 + 64, 32), (40000, 40008, 8)])
@pytest.mark.parametrize("in_place", [False, True])
def test_rmsnorm_ex_pitched(dtype, H, pitch, col0, in_place):
    T = 37
    inp = wl.rmsnorm_inputs(T, H, dtype, eps=1e-5, seed=H + col0)
    xb, xv = pitched(inp.x, pitch, col0)
    rb, rv = pitched(inp.residual, pitch + 16, col0)
    w = inp.weight.cuda()
    if in_place:
        yb, yv, rob, rov = xb, xv, rb, rv
    else:
        yb, yv = pitched(torch.zeros_like(inp.x), pitch + 32, col0)
        rob, rov = pitched(torch.zeros_like(inp.x), pitch, col0)
    astra.astra_fused_add_rmsnorm_ex(yv, rov, xv, rv, w, inp.eps)
    torch.cuda.synchronize()
    oy, orr = oracle.fused_add_rmsnorm(wl.bits(inp.x), wl.bits(inp.residual), wl.bits(inp.weight), inp.eps, dtype)
    assert np.array_equal(wl.bits(rov.cpu().contiguous()), orr), "residual sum is not bit-exact"
    check_values(f64(yv.cpu()), oy, dtype, what="rmsnorm_ex")
    for buf in (xb, rb, yb, rob):
        assert untouched(buf, col0, H)
    if not in_place:  # inputs unchanged
        assert torch.equal(xv.cpu(), inp.x) and torch.equal(rv.cpu(), inp.residual)


def test_rmsnorm_ex_equals_in_place_call():
    inp = wl.rmsnorm_inputs(300, 5120, BF16, eps=1e-5, seed=2)
    x1, r1, w = inp.x.cuda(), inp.residual.cuda(), inp.weight.cuda()
    x2, r2 = inp.x.cuda(), inp.residual.cuda()
    y2, ro2 = torch.empty_like(x2), torch.empty_like(r2)
    astra.astra_fused_add_rmsnorm(x1, r1, w, inp.eps)
    astra.astra_fused_add_rmsnorm_ex(y2, ro2, x2, r2, w, inp.eps)
    assert torch.equal(x1, y2) and torch.equal(r1, ro2)


@pytest.mark.parametrize("dtype", [BF16, FP16])
@pytest.mark.parametrize("D,pitch,col0", [(14336, 14336 + 64, 0), (4096, 3 * 4096, 4096), (1000, 1003, 1), (100, 256, 28)])
def test_silu_ex_separate_gate_and_up(dtype, D, pitch, col0):
    T = 19
    inp = wl.silu_inputs(T, D, dtype, std=2.0, seed=D)
    gate_h, up_h = inp.input[:, :D].contiguous(), inp.input[:, D:].contiguous()
    gb, gv = pitched(gate_h, pitch, col0)
    ub, uv = pitched(up_h, pitch + 8, col0)
    ob, ov = pitched(torch.zeros_like(gate_h), pitch + 24, col0)
    astra.astra_silu_and_mul_ex(ov, gv, uv)
    torch.cuda.synchronize()
    want = oracle.silu_and_mul(wl.bits(inp.input), dtype)
    check_values(f64(ov.cpu()), want, dtype, what="silu_ex")
    for buf in (gb, ub, ob):
        assert untouched(buf, col0, D)
    assert torch.equal(gv.cpu(), gate_h) and torch.equal(uv.cpu(), up_h)


def test_silu_ex_mid_size_pitched_rows():
    """Enough rows for the 32-byte-vector form, with pitches (multiples of 16 elements) that keep every
    row 32-byte aligned, and with a pitch that leaves rows only 16-byte aligned."""
    T, D = 600, 5120
    inp = wl.silu_inputs(T, D, BF16, std=2.0, seed=77)
    gate_h, up_h = inp.input[:, :D].contiguous(), inp.input[:, D:].contiguous()
    want = oracle.silu_and_mul(wl.bits(inp.input), BF16)
    for pitch in (D + 64, D + 8):
        gb, gv = pitched(gate_h, pitch, 0)
        ub, uv = pitched(up_h, pitch + 16, 0)
        ob, ov = pitched(torch.zeros_like(gate_h), pitch + 32, 0)
        astra.astra_silu_and_mul_ex(ov, gv, uv)
        torch.cuda.synchronize()
        check_values(f64(ov.cpu()), want, BF16, what=f"silu_ex mid size, pitch {pitch}")
        for buf in (gb, ub, ob):
            assert untouched(buf, 0, D)


def test_silu_ex_on_packed_rows_equals_plain_call():
    inp = wl.silu_inputs(64, 14336, BF16, seed=4)
    d = inp.input.cuda()
    o1, o2 = torch.empty((64, 14336), dtype=d.dtype, device="cuda"), torch.empty((64, 14336), dtype=d.dtype, device="cuda")
    astra.astra_silu_and_mul(o1, d)
    astra.astra_silu_and_mul_ex(o2, d[:, :14336], d[:, 14336:])
    assert torch.equal(o1, o2)


@pytest.mark.parametrize("dtype", [BF16, FP16])
@pytest.mark.parametrize("Hh,D", [(32, 128), (5, 80), (3, 7), (8, 256)])
@pytest.mark.parametrize("layout", ["head_major_scores", "sliced_values", "in_place_a"])
def test_merge_ex_strided(dtype, Hh, D, layout):
    T = 41
    inp = wl.merge_inputs(T, Hh, D, dtype, seed=Hh * 100 + D, neg_inf_frac=0.05)
    td = inp.v_a.dtype
    if layout == "head_major_scores":
        va, vb = inp.v_a.cuda(), inp.v_b.cuda()
        vo = torch.zeros_like(va)
        sa = inp.lse_a.t().contiguous().cuda().t()  # [T, Hh] view of a [Hh, T] tensor
        sb = inp.lse_b.t().contiguous().cuda().t()
        so_store = torch.full((Hh, T), 99.0, device="cuda")
        so = so_store.t()
        bufs = []
    else:
        wide = D + 24
        def slot(h):
            buf = torch.full((T, Hh, wide), PATTERN, dtype=td, device="cuda")
            buf[:, :, 8:8 + D].copy_(h)
            return buf, buf[:, :, 8:8 + D]
        ba, va = slot(inp.v_a)
        bb, vb = slot(inp.v_b)
        if layout == "in_place_a":
            bo, vo = ba, va
        else:
            bo, vo = slot(torch.zeros_like(inp.v_a))
        sa, sb = inp.lse_a.cuda(), inp.lse_b.cuda()
        so = torch.full((T, Hh), 99.0, device="cuda")
        bufs = [ba, bb, bo]
    astra.astra_merge_attn_states_lse_ex(vo, so, va, sa, vb, sb)
    torch.cuda.synchronize()
    ov, os_ = oracle.merge_attn_states_lse(wl.bits(inp.v_a), inp.lse_a.numpy(), wl.bits(inp.v_b), inp.lse_b.numpy(), dtype)
    floor = merge_floor(f64(inp.v_a), inp.lse_a.numpy(), f64(inp.v_b), inp.lse_b.numpy(), dtype)
    check_values(f64(vo.cpu()), ov, dtype, extra=floor, what="merge_ex")
    check_lse(so.cpu().numpy(), os_, what="merge_ex lse")
    for buf in bufs:
        assert untouched(buf, 8, D)


def test_merge_ex_dense_equals_plain_call():
    inp = wl.merge_inputs(257, 32, 128, BF16, seed=6)
    va, vb, sa, sb = inp.v_a.cuda(), inp.v_b.cuda(), inp.lse_a.cuda(), inp.lse_b.cuda()
    v1, s1, v2, s2 = torch.empty_like(va), torch.empty_like(sa), torch.empty_like(va), torch.empty_like(sa)
    astra.astra_merge_attn_states_lse(v1, s1, va, sa, vb, sb)
    astra.astra_merge_attn_states_lse_ex(v2, s2, va, sa, vb, sb)
    assert torch.equal(v1, v2) and torch.equal(s1.view(torch.int32), s2.view(torch.int32))


def test_rmsnorm_ex_operands_are_slices_of_one_buffer():
    """x and residual interleave row by row inside one wide buffer (no shared element)."""
    T, H = 29, 4096
    inp = wl.rmsnorm_inputs(T, H, BF16, eps=1e-5, seed=31)
    wide = torch.full((T, 2 * H + 256), PATTERN, dtype=torch.bfloat16, device="cuda")
    xv, rv = wide[:, :H], wide[:, H + 128:2 * H + 128]
    xv.copy_(inp.x); rv.copy_(inp.residual)
    astra.astra_fused_add_rmsnorm_ex(xv, rv, xv, rv, inp.weight.cuda(), inp.eps)
    oy, orr = oracle.fused_add_rmsnorm(wl.bits(inp.x), wl.bits(inp.residual), wl.bits(inp.weight), inp.eps, BF16)
    assert np.array_equal(wl.bits(rv.cpu().contiguous()), orr)
    check_values(f64(xv.cpu()), oy, BF16, what="rmsnorm_ex slices")
    assert bool((wide[:, H:H + 128] == PATTERN).all()) and bool((wide[:, 2 * H + 128:] == PATTERN).all())
