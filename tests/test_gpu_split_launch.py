"""Inputs with more than 2^31-1 vectors (or rows) are processed by several launches.  That cannot be
reached with real sizes in a test, so the library is rebuilt with the two per-launch limits lowered
(a few thousand vectors, 7 rows) and the same parity checks run through the C ABI of that build."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2509_07506_b200 import build as astra_build
from paper_2509_07506_b200 import workloads as wl
from parity import check_lse, check_values, merge_floor

pytestmark = pytest.mark.gpu
BF16 = wl.BF16


@pytest.fixture(scope="module")
def small_limits_lib(tmp_path_factory):
    path = str(tmp_path_factory.mktemp("split") / "libastra_small_limits.so")
    astra_build.build_variant(path, {"ASTRA_MAX_VECS_PER_LAUNCH": 3000, "ASTRA_MAX_ROWS_PER_LAUNCH": 7})
    lib = ctypes.CDLL(path)
    vp, i64, i32, f32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_float
    lib.astra_fused_add_rmsnorm.argtypes = [vp, vp, vp, i64, i64, f32, i32, vp]
    lib.astra_silu_and_mul.argtypes = [vp, vp, i64, i64, i32, vp]
    lib.astra_merge_attn_states_lse.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, i32, vp]
    lib.astra_merge_attn_states_lse_ex.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64,
                                                   ctypes.POINTER(ctypes.c_int64), i32, vp]
    return lib


def f64(t):
    return t.to(torch.float64).numpy()


def test_rmsnorm_rows_split_over_launches(small_limits_lib):
    inp = wl.rmsnorm_inputs(40, 520, BF16, eps=1e-5, seed=1)           # 40 rows, 7 per launch
    x, r, w = inp.x.cuda(), inp.residual.cuda(), inp.weight.cuda()
    assert small_limits_lib.astra_fused_add_rmsnorm(x.data_ptr(), r.data_ptr(), w.data_ptr(), 40, 520, 1e-5, 0, None) == 0
    oy, orr = oracle.fused_add_rmsnorm(wl.bits(inp.x), wl.bits(inp.residual), wl.bits(inp.weight), 1e-5, BF16)
    assert np.array_equal(wl.bits(r.cpu()), orr)
    check_values(f64(x.cpu()), oy, BF16, what="rmsnorm split")


def test_silu_vectors_split_over_launches(small_limits_lib):
    T, D = 101, 1000                                                    # 125 vectors per row, 24 rows per launch
    inp = wl.silu_inputs(T, D, BF16, seed=2)
    d = inp.input.cuda()
    out = torch.zeros((T, D), dtype=torch.bfloat16, device="cuda")
    assert small_limits_lib.astra_silu_and_mul(out.data_ptr(), d.data_ptr(), T, D, 0, None) == 0
    check_values(f64(out.cpu()), oracle.silu_and_mul(wl.bits(inp.input), BF16), BF16, what="silu split")


@pytest.mark.parametrize("strided", [False, True])
def test_merge_rows_split_over_launches(small_limits_lib, strided):
    T, Hh, D = 53, 6, 128                                               # 318 rows; 8 or 16 vectors per row
    inp = wl.merge_inputs(T, Hh, D, BF16, seed=3, neg_inf_frac=0.05)
    va, vb, sa, sb = inp.v_a.cuda(), inp.v_b.cuda(), inp.lse_a.cuda(), inp.lse_b.cuda()
    vo = torch.zeros_like(va)
    if strided:
        so_store = torch.zeros((Hh, T), device="cuda")
        so = so_store.t()
        strides = (ctypes.c_int64 * 12)(Hh * D, D, Hh * D, D, Hh * D, D, Hh, 1, Hh, 1, 1, T)
        st = small_limits_lib.astra_merge_attn_states_lse_ex(vo.data_ptr(), so.data_ptr(), va.data_ptr(), sa.data_ptr(),
                                                             vb.data_ptr(), sb.data_ptr(), T, Hh, D, strides, 0, None)
    else:
        so = torch.zeros_like(sa)
        st = small_limits_lib.astra_merge_attn_states_lse(vo.data_ptr(), so.data_ptr(), va.data_ptr(), sa.data_ptr(),
                                                          vb.data_ptr(), sb.data_ptr(), T, Hh, D, 0, None)
    assert st == 0
    ov, os_ = oracle.merge_attn_states_lse(wl.bits(inp.v_a), inp.lse_a.numpy(), wl.bits(inp.v_b), inp.lse_b.numpy(), BF16)
    floor = merge_floor(f64(inp.v_a), inp.lse_a.numpy(), f64(inp.v_b), inp.lse_b.numpy(), BF16)
    check_values(f64(vo.cpu()), ov, BF16, extra=floor, what="merge split")
    check_lse(so.cpu().numpy(), os_, what="merge split")
