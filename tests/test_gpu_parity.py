"""GPU parity: the CUDA library (through its C ABI) against the fp64 oracle, element by element,
on the same seeded host inputs.  Every device buffer sits between guard regions that are checked
after each launch.  Gates are defined in parity.py."""
import numpy as np
import pytest
import torch

import oracle
import paper_2509_07506_b200 as astra
from paper_2509_07506_b200 import workloads as wl
from parity import check_lse, check_values, merge_floor, ulp

pytestmark = pytest.mark.gpu

BF16, FP16 = wl.BF16, wl.FP16
GUARD = 512  # bytes on each side of every device buffer
NCPU = max(1, len(__import__("os").sched_getaffinity(0)))


class Guarded:
    """A device tensor placed `offset_elems` elements past a 256-byte-aligned point, with
    pattern-filled guard regions before and after it."""

    def __init__(self, host: torch.Tensor, offset_elems: int = 0):
        host = host.contiguous()
        self.nbytes = host.numel() * host.element_size()
        off = offset_elems * host.element_size()
        self.raw = torch.full((GUARD + off + self.nbytes + GUARD,), 0xA5, dtype=torch.uint8, device="cuda")
        self.lo = GUARD + off
        inner = self.raw[self.lo:self.lo + self.nbytes]
        self.t = inner.view(host.dtype).view(host.shape)
        self.t.copy_(host)

    def check(self):
        assert bool((self.raw[:self.lo] == 0xA5).all()), "guard before the buffer was overwritten"
        assert bool((self.raw[self.lo + self.nbytes:] == 0xA5).all()), "guard after the buffer was overwritten"

    def host(self) -> torch.Tensor:
        return self.t.cpu()


def f64(t: torch.Tensor) -> np.ndarray:
    return t.to(torch.float64).numpy()


# ---------------------------------------------------------------------------------------------
# runners
# ---------------------------------------------------------------------------------------------

CHUNK_ELEMS = 1 << 24  # elements compared at a time (bounds the fp64 temporaries to a few hundred MB)


def row_chunks(rows: int, width: int):
    """Consecutive row ranges of at most CHUNK_ELEMS elements that together cover every row."""
    step = max(1, CHUNK_ELEMS // max(1, width))
    for r0 in range(0, rows, step):
        yield slice(r0, min(rows, r0 + step))


def fold(total: dict, part: dict) -> dict:
    for k, v in part.items():
        total[k] = total.get(k, 0) + v if k.startswith("beyond") else max(total.get(k, 0.0), v)
    return total


def run_rmsnorm(inp: wl.RmsnormInputs, offset=0, stream=None):
    """Runs the library on the input and compares EVERY row with the oracle (in row chunks)."""
    gx, gr, gw = Guarded(inp.x, offset), Guarded(inp.residual, offset), Guarded(inp.weight, offset)
    astra.astra_fused_add_rmsnorm(gx.t, gr.t, gw.t, inp.eps, stream=stream)
    torch.cuda.synchronize()
    for g in (gx, gr, gw):
        g.check()
    assert torch.equal(gw.host(), inp.weight)
    y, r = gx.host(), gr.host()
    T, H = inp.x.shape
    stats = {}
    for sl in row_chunks(T, H):
        oy, orr = oracle.fused_add_rmsnorm(wl.bits(inp.x[sl]), wl.bits(inp.residual[sl]), wl.bits(inp.weight),
                                           inp.eps, inp.dtype, nthreads=NCPU)
        assert np.array_equal(wl.bits(r[sl]), orr), f"residual sum is not bit-exact in rows {sl.start}..{sl.stop}"
        fold(stats, check_values(f64(y[sl]), oy, inp.dtype, what=f"rmsnorm {tuple(inp.x.shape)} rows {sl.start}.."))
    return stats


def run_silu(inp: wl.SiluInputs, offset=0):
    T, twoD = inp.input.shape
    D = twoD // 2
    gi = Guarded(inp.input, offset)
    go = Guarded(torch.zeros((T, D), dtype=inp.input.dtype), offset)
    astra.astra_silu_and_mul(go.t, gi.t)
    torch.cuda.synchronize()
    gi.check(); go.check()
    assert torch.equal(gi.host(), inp.input)
    out = go.host()
    stats = {}
    for sl in row_chunks(T, D):
        want = oracle.silu_and_mul(wl.bits(inp.input[sl]), inp.dtype, nthreads=NCPU)
        extra = 0.0
        if inp.dtype == wl.FP32:  # the exponent's argument is rounded to binary32: |a| * 2^-24 relative
            extra = 2.0 * np.abs(f64(inp.input[sl][:, :D])) * ulp(np.where(want == 0, 1.0, want), inp.dtype) * (want != 0)
        fold(stats, check_values(f64(out[sl]), want, inp.dtype, extra=extra,
                                 what=f"silu {tuple(inp.input.shape)} rows {sl.start}.."))
    return stats


def run_merge(inp: wl.MergeInputs, offset=0, in_place=None, with_lse=True):
    T, Hh, D = inp.v_a.shape
    ga, gb = Guarded(inp.v_a, offset), Guarded(inp.v_b, offset)
    gsa, gsb = Guarded(inp.lse_a, offset), Guarded(inp.lse_b, offset)
    if in_place == "a":
        go = ga
    elif in_place == "b":
        go = gb
    else:
        go = Guarded(torch.zeros_like(inp.v_a), offset)
    gso = Guarded(torch.full((T, Hh), 123.0, dtype=torch.float32), offset)
    astra.astra_merge_attn_states_lse(go.t, gso.t if with_lse else None, ga.t, gsa.t, gb.t, gsb.t)
    torch.cuda.synchronize()
    for g in (ga, gb, gsa, gsb, go, gso):
        g.check()
    # inputs untouched (bitwise: the scores may hold NaN)
    assert torch.equal(gsa.host().view(torch.int32), inp.lse_a.view(torch.int32))
    assert torch.equal(gsb.host().view(torch.int32), inp.lse_b.view(torch.int32))
    v, s = go.host(), gso.host()
    if not with_lse:
        assert bool((s == 123.0).all())
    stats = {}
    for sl in row_chunks(T, Hh * D):
        ov, os_ = oracle.merge_attn_states_lse(wl.bits(inp.v_a[sl]), inp.lse_a[sl].numpy(), wl.bits(inp.v_b[sl]),
                                               inp.lse_b[sl].numpy(), inp.dtype, nthreads=NCPU)
        floor = merge_floor(f64(inp.v_a[sl]), inp.lse_a[sl].numpy(), f64(inp.v_b[sl]), inp.lse_b[sl].numpy(), inp.dtype)
        fold(stats, check_values(f64(v[sl]), ov, inp.dtype, extra=floor,
                                 what=f"merge {tuple(inp.v_a.shape)} tokens {sl.start}.."))
        if with_lse:
            fold(stats, {"max_lse_err": check_lse(s[sl].numpy(), os_, what=f"merge lse {tuple(inp.v_a.shape)}")})
    return stats


# ---------------------------------------------------------------------------------------------
# the named configurations
# ---------------------------------------------------------------------------------------------

def test_config1_fused_add_rmsnorm():
    stats = run_rmsnorm(wl.config1())
    assert stats["max_err_ulp"] <= 2.0


def test_config2_silu_and_mul():
    stats = run_silu(wl.config2())
    assert stats["max_err_ulp"] <= 2.0


def test_config3_merge_attn_states_lse():
    inp = wl.config3()
    both = torch.isinf(inp.lse_a) & torch.isinf(inp.lse_b)
    one = torch.isinf(inp.lse_a) ^ torch.isinf(inp.lse_b)
    assert both.sum() >= 4 and one.sum() > 50
    run_merge(inp)


@pytest.mark.parametrize("dtype", [BF16, FP16])
@pytest.mark.parametrize("H", wl.SWEEP_H)
@pytest.mark.parametrize("T", wl.SWEEP_T)
def test_config4_rmsnorm_sweep(dtype, T, H):
    run_rmsnorm(wl.config4_point(dtype, T, H))  # every row, also at T = 16384


def test_config5_chain_shapes():
    """Full-size chain shapes in the launch configuration the benchmark times; every row of all
    three calls is compared with the oracle."""
    cfg = wl.config5()
    assert run_rmsnorm(cfg["rmsnorm"])["max_err_ulp"] <= 2.0
    assert run_silu(cfg["silu"])["max_err_ulp"] <= 2.0
    run_merge(cfg["merge"])  # gated inside (2 ulp plus the accumulation floor of a cancelling blend)


@pytest.mark.parametrize("dtype", [BF16, FP16])
@pytest.mark.parametrize("kernel,shape", [(k, sh) for k, sh, _, _ in wl.TABLE4])
def test_table4_shapes(dtype, kernel, shape):
    """The twelve shapes of the paper's per-shape study (Table 4), all elements."""
    inp = wl.table4_inputs(kernel, shape, dtype)
    {"merge_attn_states_lse": run_merge, "fused_add_rmsnorm": run_rmsnorm, "silu_and_mul": run_silu}[kernel](inp)


# ---------------------------------------------------------------------------------------------
# shapes: tiny, ragged, several tiles, odd alignment
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype", [BF16, FP16])
@pytest.mark.parametrize("H", [1, 2, 3, 7, 8, 9, 33, 250, 1000, 4100, 4101, 4098, 8190, 11008, 14336,
                               32768, 32776, 40000, 65538, 16392, 20500, 49152, 131072, 131080, 100000])
def test_rmsnorm_widths(dtype, H):
    # widths above 16384 exercise the cluster kernel (2, 4 or 8 blocks per row) and, beyond
    # 131072 or with narrow vectors, the two-sweep kernel; T = 3 or 5 leaves a partial wave of clusters
    T = 3 if H > 20000 else 5
    run_rmsnorm(wl.rmsnorm_inputs(T, H, dtype, eps=1e-5, seed=H))


@pytest.mark.parametrize("offset", [1, 2, 4, 8])
@pytest.mark.parametrize("H", [4096, 4100, 520])
def test_rmsnorm_pointer_offsets(offset, H):
    run_rmsnorm(wl.rmsnorm_inputs(7, H, BF16, eps=1e-6, seed=offset), offset=offset)


@pytest.mark.parametrize("offset", [0, 8, 16, 4])
@pytest.mark.parametrize("T,H", [(1033, 4096), (1024, 5120), (1100, 2048), (333, 4096), (1025, 14336), (1030, 11008),
                                 (1024, 16384), (1040, 1024)])
def test_rmsnorm_streaming_alignments(offset, T, H):
    """From 1024 rows on, rows that are 32-byte aligned take two 32-byte vectors per thread, 16-byte
    aligned ones (offset 8) four 16-byte vectors, 8-byte aligned ones (offset 4) 8-byte vectors; between
    one wave of rows and 1024 rows the 16-byte form serves both."""
    run_rmsnorm(wl.rmsnorm_inputs(T, H, BF16, eps=1e-5, seed=offset + T), offset=offset)


def test_rmsnorm_closed_forms_on_gpu():
    # constant row -> sign(c) * w ; zero row -> 0
    H = 4096
    w = wl.rmsnorm_inputs(1, H, BF16, seed=5).weight
    x = torch.full((3, H), 0.75, dtype=torch.bfloat16); r = torch.full((3, H), 1.25, dtype=torch.bfloat16)
    x[1] = -2.0; r[1] = -1.0; x[2] = 1.5; r[2] = -1.5
    gx, gr, gw = Guarded(x), Guarded(r), Guarded(w)
    astra.astra_fused_add_rmsnorm(gx.t, gr.t, gw.t, 1e-6)
    y = gx.host()
    assert torch.equal(y[0], w) and torch.equal(y[1], -w) and bool((y[2] == 0).all())
    assert bool((gr.host()[0] == 2.0).all()) and bool((gr.host()[2] == 0).all())


def test_rmsnorm_on_side_stream_and_repeatable():
    inp = wl.rmsnorm_inputs(300, 5120, BF16, eps=1e-5, seed=12)
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        a = run_rmsnorm(inp, stream=s)
    b = run_rmsnorm(inp)
    assert a == b


@pytest.mark.parametrize("dtype", [BF16, FP16])
@pytest.mark.parametrize("D", [1, 2, 7, 8, 9, 100, 1000, 4096, 5120, 12288, 14336, 14340, 14342, 14337])
def test_silu_widths(dtype, D):
    run_silu(wl.silu_inputs(5, D, dtype, std=2.0, seed=D))


@pytest.mark.parametrize("dtype", [BF16, FP16])
@pytest.mark.parametrize("T,D,offset", [(256, 14336, 0), (1024, 4096, 0), (700, 5120, 16), (700, 5120, 8), (2048, 14336, 0),
                                        (300, 11008, 0)])
def test_silu_mid_sizes(dtype, T, D, offset):
    """Between about one and ten waves of blocks the 32-byte-vector form runs where gate, up and out are
    32-byte aligned (offsets 0 and 16; D = 11008 puts the up half only 16-byte aligned), the 16-byte
    form otherwise."""
    run_silu(wl.silu_inputs(T, D, dtype, std=2.0, seed=T + D), offset=offset)


@pytest.mark.parametrize("offset", [1, 2, 4])
def test_silu_pointer_offsets(offset):
    run_silu(wl.silu_inputs(9, 4096, BF16, seed=offset), offset=offset)


def test_silu_extreme_gates():
    vals = [0.0, -0.0, 1e-30, -1e-30, 20.0, -20.0, 87.0, -87.0, 88.5, -88.5, 100.0, -100.0, 1e4, -1e4,
            3e38, -3e38, 0.5, -0.5]
    a = torch.tensor(vals, dtype=torch.float32).repeat(8)
    b = torch.linspace(-1, 1, a.numel())
    row = torch.cat([a, b]).to(torch.bfloat16).reshape(1, -1)
    run_silu(wl.SiluInputs(row, BF16))
    row16 = torch.cat([a.clamp(-6e4, 6e4), b]).to(torch.float16).reshape(1, -1)
    run_silu(wl.SiluInputs(row16, FP16))


@pytest.mark.parametrize("dtype", [BF16, FP16])
@pytest.mark.parametrize("Hh,D", [(1, 1), (3, 7), (3, 8), (2, 9), (32, 128), (40, 128), (32, 256), (5, 80),
                                  (7, 64), (3, 130), (2, 1028), (1, 4100)])
def test_merge_shapes(dtype, Hh, D):
    run_merge(wl.merge_inputs(37, Hh, D, dtype, seed=Hh * 1000 + D, neg_inf_frac=0.05))


@pytest.mark.parametrize("offset", [1, 2, 4])
def test_merge_pointer_offsets(offset):
    run_merge(wl.merge_inputs(33, 8, 128, BF16, seed=offset), offset=offset)


@pytest.mark.parametrize("in_place", ["a", "b"])
def test_merge_in_place_values(in_place):
    run_merge(wl.merge_inputs(129, 32, 128, BF16, seed=9), in_place=in_place)


def test_merge_without_lse_output():
    run_merge(wl.merge_inputs(65, 4, 128, BF16, seed=10), with_lse=False)


def test_merge_special_scores():
    """Equal scores -> mean and +ln 2; one -inf -> the other state, bit for bit, even when the empty
    side holds Inf/NaN; both -inf -> zeros and -inf; +inf / NaN scores -> NaN."""
    T, Hh, D = 8, 1, 128
    inp = wl.merge_inputs(T, Hh, D, BF16, seed=3, neg_inf_frac=0.0, forced_both_neg_inf=0)
    ninf, inf, nan = float("-inf"), float("inf"), float("nan")
    inp.lse_a[:, 0] = torch.tensor([1.5, 2.0, ninf, ninf, 3.0, inf, nan, -40.0])
    inp.lse_b[:, 0] = torch.tensor([1.5, ninf, -7.0, ninf, ninf, 0.0, 0.0, -40.0])
    inp.v_b[4, 0, :4] = torch.tensor([inf, -inf, nan, 1.0], dtype=torch.bfloat16)  # garbage on the empty side
    inp.v_a[2, 0, :2] = torch.tensor([nan, inf], dtype=torch.bfloat16)
    ga, gb = Guarded(inp.v_a), Guarded(inp.v_b)
    gsa, gsb = Guarded(inp.lse_a), Guarded(inp.lse_b)
    go, gso = Guarded(torch.zeros_like(inp.v_a)), Guarded(torch.zeros((T, Hh), dtype=torch.float32))
    astra.astra_merge_attn_states_lse(go.t, gso.t, ga.t, gsa.t, gb.t, gsb.t)
    v, s = go.host(), gso.host()
    assert torch.equal(v[1], inp.v_a[1]) and s[1, 0] == 2.0
    assert torch.equal(v[2], inp.v_b[2]) and s[2, 0] == -7.0
    assert bool((v[3] == 0).all()) and s[3, 0] == ninf
    assert torch.equal(v[4], inp.v_a[4]) and s[4, 0] == 3.0
    assert bool(v[5].isnan().all()) and bool(s[5].isnan().all())
    assert bool(v[6].isnan().all()) and bool(s[6].isnan().all())
    run_merge(inp)  # and the whole thing against the oracle


@pytest.mark.parametrize("dtype", [BF16, FP16, wl.FP32])
def test_merge_large_finite_score_gaps(dtype):
    """Finite score gaps around and beyond the point where the smaller side's binary32 weight
    underflows (a gap of about 87.3 reaches the subnormals, about 103.3 reaches exactly 0): the
    kernel then drops that side like an empty one, while the double-precision weight is still
    non-zero.  With finite payloads the two agree to far below one unit of the gate; both orders."""
    gaps = [80.0, 87.0, 88.0, 90.0, 100.0, 103.0, 103.5, 104.0, 120.0, 150.0, 200.0, 1000.0, 3e38]
    T, Hh, D = 2 * len(gaps), 3, 128
    inp = wl.merge_inputs(T, Hh, D, dtype, seed=21, neg_inf_frac=0.0, forced_both_neg_inf=0)
    for i, g in enumerate(gaps):
        base = torch.tensor([-50.0, 0.0, 7.5])
        hi = base if g < 1e30 else torch.zeros(3)
        lo = hi - g if g < 1e30 else torch.full((3,), -g)
        inp.lse_a[2 * i], inp.lse_b[2 * i] = hi, lo          # a dominates
        inp.lse_a[2 * i + 1], inp.lse_b[2 * i + 1] = lo, hi  # b dominates
    inp.v_a[:, :, :4] = torch.tensor([3.0e4, -3.0e4, 1.0, -0.0], dtype=inp.v_a.dtype)  # large finite payloads
    inp.v_b[:, :, :4] = torch.tensor([-3.0e4, 3.0e4, -1.0, 0.0], dtype=inp.v_b.dtype)
    run_merge(inp)
    # beyond the underflow point the dominated side is dropped: the other state comes back bit for bit
    va, vb = inp.v_a.cuda(), inp.v_b.cuda()
    vo, so = torch.empty_like(va), torch.empty((T, Hh), device="cuda")
    astra.astra_merge_attn_states_lse(vo, so, va, inp.lse_a.cuda(), vb, inp.lse_b.cuda())
    for i, g in enumerate(gaps):
        if g >= 104.0:
            assert torch.equal(vo[2 * i].cpu(), inp.v_a[2 * i]) and torch.equal(vo[2 * i + 1].cpu(), inp.v_b[2 * i + 1])
            assert torch.equal(so[2 * i].cpu(), inp.lse_a[2 * i]) and torch.equal(so[2 * i + 1].cpu(), inp.lse_b[2 * i + 1])


# ---------------------------------------------------------------------------------------------
# degenerate sizes and error codes through the C ABI
# ---------------------------------------------------------------------------------------------

def test_empty_inputs_launch_nothing():
    lib = astra.load_library()
    buf = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    p = buf.data_ptr()
    assert lib.astra_fused_add_rmsnorm(p, p + 32, p + 64, 0, 16, 1e-6, 0, None) == 0
    assert lib.astra_silu_and_mul(p, p + 32, 0, 8, 0, None) == 0
    assert lib.astra_merge_attn_states_lse(p, None, p, p, p, p, 0, 1, 8, 0, None) == 0
    torch.cuda.synchronize()
    assert bool((buf == 0).all())


def test_empty_batches_through_the_binding():
    """torch reports address 0 for a tensor without elements; a rank that was dealt no rows must still
    be able to make its calls."""
    for td in (torch.bfloat16, torch.float16, torch.float32):
        e = lambda *shape: torch.empty(shape, dtype=td, device="cuda")  # noqa: E731
        astra.astra_fused_add_rmsnorm(e(0, 64), e(0, 64), e(64), 1e-6)
        astra.astra_fused_add_rmsnorm_ex(e(0, 64), e(0, 64), e(0, 64), e(0, 64), e(64), 1e-6)
        astra.astra_silu_and_mul(e(0, 32), e(0, 64))
        astra.astra_silu_and_mul_ex(e(0, 32), e(0, 32), e(0, 32))
        s = lambda: torch.empty((0, 4), device="cuda")  # noqa: E731
        astra.astra_merge_attn_states_lse(e(0, 4, 16), s(), e(0, 4, 16), s(), e(0, 4, 16), s())
        astra.astra_merge_attn_states_lse_ex(e(0, 4, 16), None, e(0, 4, 16), s(), e(0, 4, 16), s())
        astra.astra_fused_allreduce_add_rmsnorm(e(0, 64), e(0, 64), [e(0, 64), e(0, 64)], e(64), 1e-6)
    torch.cuda.synchronize()


def test_prepared_calls_match_plain_calls_bit_for_bit():
    """A prepared call (validated once, re-issued with only the stream looked up) runs the same
    launch as the plain call: identical bits, also when re-issued after the inputs were refilled and
    on a side stream."""
    rms = wl.rmsnorm_inputs(48, 4096, BF16, eps=1e-5, seed=31)
    si = wl.silu_inputs(16, 12288, FP16, seed=32)
    mi = wl.merge_inputs(96, 32, 128, BF16, seed=33)
    x, r, w = rms.x.cuda(), rms.residual.cuda(), rms.weight.cuda()
    x2, r2 = x.clone(), r.clone()
    d_in = si.input.cuda(); o1, o2 = torch.empty((16, 12288), dtype=torch.float16, device="cuda"), torch.empty((16, 12288), dtype=torch.float16, device="cuda")
    va, vb, sa, sb = mi.v_a.cuda(), mi.v_b.cuda(), mi.lse_a.cuda(), mi.lse_b.cuda()
    v1, v2, l1, l2 = torch.empty_like(va), torch.empty_like(va), torch.empty_like(sa), torch.empty_like(sa)
    p_rms = astra.prepare_fused_add_rmsnorm(x2, r2, w, rms.eps)
    p_silu = astra.prepare_silu_and_mul(o2, d_in)
    p_merge = astra.prepare_merge_attn_states_lse(v2, l2, va, sa, vb, sb)
    side = torch.cuda.Stream()
    for rep in range(3):
        x.copy_(rms.x); r.copy_(rms.residual); x2.copy_(rms.x); r2.copy_(rms.residual)
        o2.zero_(); v2.zero_(); l2.zero_()
        astra.astra_fused_add_rmsnorm(x, r, w, rms.eps)
        astra.astra_silu_and_mul(o1, d_in)
        astra.astra_merge_attn_states_lse(v1, l1, va, sa, vb, sb)
        if rep == 2:
            side.wait_stream(torch.cuda.current_stream())
            p_rms(side); p_silu(side); p_merge(side)
            torch.cuda.current_stream().wait_stream(side)
        else:
            p_rms(); p_silu(); p_merge()
        torch.cuda.synchronize()
        assert torch.equal(x, x2) and torch.equal(r, r2) and torch.equal(o1, o2)
        assert torch.equal(v1, v2) and torch.equal(l1.view(torch.int32), l2.view(torch.int32))
    oy, orr = oracle.fused_add_rmsnorm(wl.bits(rms.x), wl.bits(rms.residual), wl.bits(rms.weight), rms.eps, BF16)
    assert np.array_equal(wl.bits(r2.cpu()), orr)
    check_values(f64(x2.cpu()), oy, BF16, what="prepared rmsnorm")


def test_prepared_call_routes_agree_bit_for_bit():
    """A prepared call is issued by the extension module; ``via_ctypes`` issues the same arguments
    through ctypes.  Both reach the same entry point: identical bits, on the current and a side stream."""
    rms = wl.rmsnorm_inputs(40, 5120, FP16, eps=1e-5, seed=41)
    mi = wl.merge_inputs(70, 8, 128, BF16, seed=43, neg_inf_frac=0.05)
    ar = wl.allreduce_rmsnorm_inputs(24, 4096, 3, BF16, seed=44)
    w = rms.weight.cuda()
    va, vb, sa, sb = mi.v_a.cuda(), mi.v_b.cuda(), mi.lse_a.cuda(), mi.lse_b.cuda()
    parts, aw = [p.cuda() for p in ar.parts], ar.weight.cuda()
    outs = []
    side = torch.cuda.Stream()
    for route in ("extension", "ctypes", "ctypes on a side stream"):
        x, r = rms.x.cuda(), rms.residual.cuda()
        vo, lo = torch.empty_like(va), torch.empty_like(sa)
        y, rr = torch.empty_like(parts[0]), ar.residual.cuda()
        calls = [astra.prepare_fused_add_rmsnorm(x, r, w, rms.eps), astra.prepare_merge_attn_states_lse(vo, lo, va, sa, vb, sb),
                 astra.prepare_fused_allreduce_add_rmsnorm(y, rr, parts, aw, ar.eps)]
        if route == "extension":
            for c in calls:
                c()
        elif route == "ctypes":
            for c in calls:
                c.via_ctypes()
        else:
            side.wait_stream(torch.cuda.current_stream())
            for c in calls:
                c.via_ctypes(side)
            torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        outs.append((x, r, vo, lo.view(torch.int32), y, rr))
    for other in outs[1:]:
        for a, b in zip(outs[0], other):
            assert torch.equal(a, b)
    oy, orr = oracle.fused_add_rmsnorm(wl.bits(rms.x), wl.bits(rms.residual), wl.bits(rms.weight), rms.eps, FP16)
    assert np.array_equal(wl.bits(outs[0][1].cpu()), orr)
    check_values(f64(outs[0][0].cpu()), oy, FP16, what="prepared rmsnorm, extension route")


def test_decode_chain_replayed_from_a_graph_matches_the_oracle():
    """The three calls at a decode-sized batch, captured once and replayed with new inputs: every
    replay's outputs are compared with the oracle (and are bit-identical to the eager calls')."""
    T, H, D, Hh, Dh = 16, 4096, 14336, 32, 128
    dev = "cuda"
    x = torch.empty((T, H), dtype=torch.bfloat16, device=dev); r = torch.empty_like(x)
    w = torch.empty((H,), dtype=torch.bfloat16, device=dev)
    si = torch.empty((T, 2 * D), dtype=torch.bfloat16, device=dev); so = torch.empty((T, D), dtype=torch.bfloat16, device=dev)
    va = torch.empty((T, Hh, Dh), dtype=torch.bfloat16, device=dev); vb = torch.empty_like(va); vo = torch.empty_like(va)
    sa = torch.empty((T, Hh), device=dev); sb = torch.empty_like(sa); lo = torch.empty_like(sa)
    chain = astra.CapturedCalls([astra.prepare_fused_add_rmsnorm(x, r, w, 1e-5), astra.prepare_silu_and_mul(so, si),
                                 astra.prepare_merge_attn_states_lse(vo, lo, va, sa, vb, sb)])
    for seed in (101, 102, 103):
        rms = wl.rmsnorm_inputs(T, H, BF16, eps=1e-5, seed=seed)
        sil = wl.silu_inputs(T, D, BF16, seed=seed)
        mer = wl.merge_inputs(T, Hh, Dh, BF16, seed=seed, neg_inf_frac=0.05)
        x.copy_(rms.x); r.copy_(rms.residual); w.copy_(rms.weight); si.copy_(sil.input)
        va.copy_(mer.v_a); vb.copy_(mer.v_b); sa.copy_(mer.lse_a); sb.copy_(mer.lse_b)
        so.zero_(); vo.zero_(); lo.zero_()
        chain.replay()
        torch.cuda.synchronize()
        oy, orr = oracle.fused_add_rmsnorm(wl.bits(rms.x), wl.bits(rms.residual), wl.bits(rms.weight), 1e-5, BF16)
        assert np.array_equal(wl.bits(r.cpu()), orr)
        check_values(f64(x.cpu()), oy, BF16, what="graph replay: rmsnorm")
        check_values(f64(so.cpu()), oracle.silu_and_mul(wl.bits(sil.input), BF16), BF16, what="graph replay: silu")
        ov, ol = oracle.merge_attn_states_lse(wl.bits(mer.v_a), mer.lse_a.numpy(), wl.bits(mer.v_b), mer.lse_b.numpy(), BF16)
        check_values(f64(vo.cpu()), ov, BF16, extra=merge_floor(f64(mer.v_a), mer.lse_a.numpy(), f64(mer.v_b), mer.lse_b.numpy(), BF16),
                     what="graph replay: merge")
        check_lse(lo.cpu().numpy(), ol, what="graph replay: merge lse")
        # the same inputs through eager calls: identical bits
        x2, r2 = rms.x.cuda(), rms.residual.cuda()
        so2, vo2, lo2 = torch.empty_like(so), torch.empty_like(vo), torch.empty_like(lo)
        astra.astra_fused_add_rmsnorm(x2, r2, w, 1e-5)
        astra.astra_silu_and_mul(so2, si)
        astra.astra_merge_attn_states_lse(vo2, lo2, va, sa, vb, sb)
        assert torch.equal(x, x2) and torch.equal(r, r2) and torch.equal(so, so2) and torch.equal(vo, vo2)
        assert torch.equal(lo.view(torch.int32), lo2.view(torch.int32))


def test_a_pending_runtime_error_of_the_caller_survives_a_library_call():
    """An error that some other code left pending in the caller's CUDA runtime (here: a call the
    runtime refuses on the host, nothing reaches the GPU) must still be there after a successful
    library call: the library neither reads nor clears the caller's last-error state."""
    import ctypes
    try:
        rt = ctypes.CDLL("libcudart.so.12")   # the runtime torch has loaded
    except OSError:
        pytest.skip("the shared CUDA runtime torch uses cannot be opened by name")
    rt.cudaPeekAtLastError.restype = ctypes.c_int
    rt.cudaGetLastError.restype = ctypes.c_int
    rt.cudaSetDevice.restype = ctypes.c_int
    inp = wl.silu_inputs(8, 1024, BF16, seed=3)
    d_in = inp.input.cuda()
    out = torch.empty((8, 1024), dtype=torch.bfloat16, device="cuda")
    call = astra.prepare_silu_and_mul(out, d_in)
    torch.cuda.synchronize()
    assert rt.cudaPeekAtLastError() == 0
    refused = rt.cudaSetDevice(9999)          # no such device: refused on the host
    try:
        assert refused != 0 and rt.cudaPeekAtLastError() == refused
        call()                                 # a successful launch through the C ABI
        assert rt.cudaPeekAtLastError() == refused, "the library consumed the caller's pending error"
    finally:
        assert rt.cudaGetLastError() == refused    # take it out again
    assert rt.cudaPeekAtLastError() == 0
    torch.cuda.synchronize()
    check_values(f64(out.cpu()), oracle.silu_and_mul(wl.bits(inp.input), BF16), BF16, what="silu after a pending error")


def test_binding_rejects_wrong_arguments():
    x = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(TypeError):
        astra.astra_fused_add_rmsnorm(x.cpu(), x, x[0], 1e-6)
    with pytest.raises(ValueError):
        astra.astra_fused_add_rmsnorm(x, x[:, :32], x[0], 1e-6)
    with pytest.raises(TypeError):
        astra.astra_silu_and_mul(x[:, :32].contiguous().float(), x)
    with pytest.raises(astra.AstraError) as e:
        astra.astra_fused_add_rmsnorm(x, x, x[0].clone(), 1e-6)
    assert e.value.status == 6


def test_host_streamer_pipeline_matches_oracle():
    """Host-resident batches processed in row chunks over three streams, device buffers reused
    for a second batch: results of both batches match the oracle."""
    from paper_2509_07506_b200.hoststream import HostStreamer
    dev = torch.device("cuda", torch.cuda.current_device())
    T, D, chunk = 96, 1000, 32
    pipe = HostStreamer(dev)
    d_in = torch.empty((T, 2 * D), dtype=torch.bfloat16, device=dev)
    d_out = torch.empty((T, D), dtype=torch.bfloat16, device=dev)
    batches = [wl.silu_inputs(T, D, BF16, seed=s) for s in (41, 42)]
    host_in = [b.input.pin_memory() for b in batches]
    host_out = [torch.empty((T, D), dtype=torch.bfloat16).pin_memory() for _ in batches]
    for hin, hout in zip(host_in, host_out):
        for r0 in range(0, T, chunk):
            sl = slice(r0, r0 + chunk)
            pipe.submit(("silu", r0), [(d_in[sl], hin[sl])],
                        lambda sl=sl: astra.astra_silu_and_mul(d_out[sl], d_in[sl]),
                        [(hout[sl], d_out[sl])])
    pipe.synchronize()
    for b, hout in zip(batches, host_out):
        check_values(f64(hout), oracle.silu_and_mul(wl.bits(b.input), BF16), BF16, what="host streamer")


def test_results_are_bitwise_repeatable():
    """No atomics and a fixed reduction order: repeated launches on the same inputs, back to back and
    interleaved with other launches, give bit-identical outputs (a cheap race detector)."""
    rms = wl.rmsnorm_inputs(700, 5120, BF16, eps=1e-5, seed=77)
    si = wl.silu_inputs(300, 14336, BF16, seed=78)
    mi = wl.merge_inputs(900, 32, 128, BF16, seed=79)
    w = rms.weight.cuda()
    d_si = si.input.cuda(); va, vb = mi.v_a.cuda(), mi.v_b.cuda(); sa, sb = mi.lse_a.cuda(), mi.lse_b.cuda()
    ref = None
    for it in range(12):
        x, r = rms.x.cuda(), rms.residual.cuda()
        so = torch.empty((300, 14336), dtype=torch.bfloat16, device="cuda")
        vo, lo = torch.empty_like(va), torch.empty_like(sa)
        astra.astra_fused_add_rmsnorm(x, r, w, rms.eps)
        astra.astra_silu_and_mul(so, d_si)
        astra.astra_merge_attn_states_lse(vo, lo, va, sa, vb, sb)
        got = [t.clone() for t in (x, r, so, vo)] + [lo.view(torch.int32).clone()]
        if ref is None:
            ref = got
        else:
            for a, b in zip(ref, got):
                assert torch.equal(a, b), f"iteration {it} differs"
