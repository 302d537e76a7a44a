"""GPU parity of the ablation library (the paper's baseline / optimised design pairs) against the
fp64 oracle, on the value distributions of the named configurations.  Both designs of every pair
must meet the same gates as the library's own kernels, so that their timings compare like with like."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_07506_b200 import ablation
from paper_2509_07506_b200 import workloads as wl
from parity import check_lse, check_values, merge_floor

pytestmark = pytest.mark.gpu
BF16, FP16 = wl.BF16, wl.FP16


def f64(t):
    return t.to(torch.float64).numpy()


@pytest.mark.parametrize("design", [0, 1])
@pytest.mark.parametrize("dtype", [BF16, FP16])
@pytest.mark.parametrize("T,H", [(16, 4096), (33, 5120), (5, 4100), (3, 250), (2, 11008)])
def test_ablation_rmsnorm(design, dtype, T, H):
    inp = wl.rmsnorm_inputs(T, H, dtype, eps=1e-6, seed=H)
    x, r, w = inp.x.cuda(), inp.residual.cuda(), inp.weight.cuda()
    ablation.astra_ablation_fused_add_rmsnorm(design, x, r, w, inp.eps)
    oy, orr = oracle.fused_add_rmsnorm(wl.bits(inp.x), wl.bits(inp.residual), wl.bits(inp.weight), inp.eps, dtype)
    assert np.array_equal(wl.bits(r.cpu()), orr)
    check_values(f64(x.cpu()), oy, dtype, what=f"ablation rmsnorm design {design}")


@pytest.mark.parametrize("design", [0, 1])
@pytest.mark.parametrize("dtype", [BF16, FP16])
@pytest.mark.parametrize("T,D", [(128, 14336), (7, 4096), (3, 250), (5, 1002)])
def test_ablation_silu(design, dtype, T, D):
    inp = wl.silu_inputs(T, D, dtype, std=2.0, seed=D)
    d = inp.input.cuda()
    out = torch.zeros((T, D), dtype=d.dtype, device="cuda")
    ablation.astra_ablation_silu_and_mul(design, out, d)
    check_values(f64(out.cpu()), oracle.silu_and_mul(wl.bits(inp.input), dtype), dtype,
                 what=f"ablation silu design {design}")


@pytest.mark.parametrize("design", [0, 1])
@pytest.mark.parametrize("dtype", [BF16, FP16])
@pytest.mark.parametrize("T,Hh,D", [(512, 32, 128), (37, 5, 80), (9, 3, 256), (11, 2, 34)])
def test_ablation_merge(design, dtype, T, Hh, D):
    inp = wl.merge_inputs(T, Hh, D, dtype, seed=T + D)
    va, vb, sa, sb = inp.v_a.cuda(), inp.v_b.cuda(), inp.lse_a.cuda(), inp.lse_b.cuda()
    vo, so = torch.zeros_like(va), torch.zeros_like(sa)
    ablation.astra_ablation_merge_attn_states_lse(design, vo, so, va, sa, vb, sb)
    ov, os_ = oracle.merge_attn_states_lse(wl.bits(inp.v_a), inp.lse_a.numpy(), wl.bits(inp.v_b), inp.lse_b.numpy(), dtype)
    floor = merge_floor(f64(inp.v_a), inp.lse_a.numpy(), f64(inp.v_b), inp.lse_b.numpy(), dtype)
    check_values(f64(vo.cpu()), ov, dtype, extra=floor, what=f"ablation merge design {design}")
    check_lse(so.cpu().numpy(), os_, what=f"ablation merge design {design}")
