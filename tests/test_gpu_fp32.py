"""GPU parity for fp32 storage (ASTRA_FP32): same kernels, two 16-bit units per element, no rounding
at the store.  The residual sum is bit-exact (one binary32 add); values are gated at 16 fp32 ulp
(plus the documented argument-rounding term for silu and the blend floor for merge)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2509_07506_b200 as astra
from paper_2509_07506_b200 import workloads as wl
from parity import check_lse, check_values, merge_floor
from test_gpu_parity import run_merge, run_rmsnorm, run_silu

pytestmark = pytest.mark.gpu
FP32 = wl.FP32


@pytest.mark.parametrize("T,H", [(16, 4096), (64, 8192), (5, 4100), (5, 4098), (3, 250), (2, 33), (3, 1), (4, 5120),
                                 (3, 11008), (2, 14336), (2, 40000), (3, 8200), (2, 65536), (2, 70000)])
def test_rmsnorm_fp32(T, H):
    run_rmsnorm(wl.rmsnorm_inputs(T, H, FP32, eps=1e-5, seed=H))


@pytest.mark.parametrize("T,H", [(1100, 4096), (1024, 2048), (1500, 1024), (700, 4096)])
def test_rmsnorm_fp32_streaming_sizes(T, H):
    """More rows than one wave of blocks: 32-byte vectors (two per thread) where the rows allow it,
    16-byte vectors otherwise; every row against the oracle."""
    run_rmsnorm(wl.rmsnorm_inputs(T, H, FP32, eps=1e-5, seed=T))


@pytest.mark.parametrize("offset", [1, 2, 4])
def test_rmsnorm_fp32_pointer_offsets(offset):
    run_rmsnorm(wl.rmsnorm_inputs(7, 4096, FP32, eps=1e-6, seed=offset), offset=offset)


@pytest.mark.parametrize("T,D", [(128, 14336), (5, 1000), (3, 7), (2, 1), (4, 4098), (9, 4096)])
def test_silu_fp32(T, D):
    run_silu(wl.silu_inputs(T, D, FP32, std=2.0, seed=D))


@pytest.mark.parametrize("T,Hh,D", [(512, 32, 128), (37, 5, 80), (9, 3, 7), (5, 1, 1), (11, 8, 256), (7, 2, 130)])
def test_merge_fp32(T, Hh, D):
    run_merge(wl.merge_inputs(T, Hh, D, FP32, seed=T + D, neg_inf_frac=0.05))


def test_merge_fp32_in_place_and_offsets():
    run_merge(wl.merge_inputs(65, 8, 128, FP32, seed=5), in_place="a")
    run_merge(wl.merge_inputs(33, 8, 128, FP32, seed=6), offset=1)


def test_fp32_pitched_and_out_of_place():
    T, H, pitch = 21, 520, 777
    inp = wl.rmsnorm_inputs(T, H, FP32, eps=1e-5, seed=9)
    xb = torch.full((T, pitch), -7.75, device="cuda"); rb = torch.full((T, pitch + 4), -7.75, device="cuda")
    xv, rv = xb[:, 3:3 + H], rb[:, 3:3 + H]
    xv.copy_(inp.x); rv.copy_(inp.residual)
    y = torch.zeros((T, H), device="cuda"); ro = torch.zeros((T, H), device="cuda")
    astra.astra_fused_add_rmsnorm_ex(y, ro, xv, rv, inp.weight.cuda(), inp.eps)
    oy, orr = oracle.fused_add_rmsnorm(wl.bits(inp.x), wl.bits(inp.residual), wl.bits(inp.weight), inp.eps, FP32)
    assert np.array_equal(wl.bits(ro.cpu()), orr)
    check_values(y.cpu().double().numpy(), oy, FP32, what="rmsnorm_ex fp32")
    assert bool((xb[:, :3] == -7.75).all()) and bool((xb[:, 3 + H:] == -7.75).all())
    # head-major scores with fp32 values
    mi = wl.merge_inputs(19, 4, 64, FP32, seed=10)
    va, vb = mi.v_a.cuda(), mi.v_b.cuda()
    sa, sb = mi.lse_a.t().contiguous().cuda().t(), mi.lse_b.t().contiguous().cuda().t()
    vo = torch.zeros_like(va); so = torch.zeros((4, 19), device="cuda").t()
    astra.astra_merge_attn_states_lse_ex(vo, so, va, sa, vb, sb)
    ov, os_ = oracle.merge_attn_states_lse(wl.bits(mi.v_a), mi.lse_a.numpy(), wl.bits(mi.v_b), mi.lse_b.numpy(), FP32)
    floor = merge_floor(mi.v_a.double().numpy(), mi.lse_a.numpy(), mi.v_b.double().numpy(), mi.lse_b.numpy(), FP32)
    check_values(vo.cpu().double().numpy(), ov, FP32, extra=floor, what="merge_ex fp32")
    check_lse(so.cpu().numpy(), os_, what="merge_ex fp32")
