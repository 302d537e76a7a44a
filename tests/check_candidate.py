"""Deterministic core of the paper's Testing and Profiling agents, as a test tool (Algorithm 1:
Validate and Profile; Section 3.1: max-discrepancy correctness and geometric-mean performance).

Given any shared library that exports the C ABI of include/astra.h, it
  1. validates the three entry points against the fp64 oracle on a suite of diverse shapes
     (the named configurations, ragged and tiny shapes, both 16-bit storage types) with the same
     gates as the parity tests, and
  2. profiles them with the paper's protocol (20 warm-up launches, 100 timed) on the Table 4 shapes,
and prints one log record per call: (round, candidate, correct, worst discrepancy, per-shape times,
geometric-mean time), i.e. the tuple Algorithm 1 appends to its log.

    python tests/check_candidate.py --lib path/to/libcandidate.so [--round 3] [--baseline other.so]

With --baseline the record also carries the geometric-mean speedup over that library.  This is test
infrastructure (it calls the oracle); it is not part of the product path.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import math
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
for p in (ROOT, os.path.join(ROOT, "tests")):
    if p not in sys.path:
        sys.path.insert(0, p)

import numpy as np  # noqa: E402
import torch  # noqa: E402

import oracle  # noqa: E402
from paper_2509_07506_b200 import workloads as wl  # noqa: E402
from parity import check_lse, check_values, merge_floor  # noqa: E402


def load(path: str) -> ctypes.CDLL:
    lib = ctypes.CDLL(path)
    vp, i64, i32, f32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_float
    lib.astra_fused_add_rmsnorm.argtypes = [vp, vp, vp, i64, i64, f32, i32, vp]
    lib.astra_silu_and_mul.argtypes = [vp, vp, i64, i64, i32, vp]
    lib.astra_merge_attn_states_lse.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, i32, vp]
    for f in (lib.astra_fused_add_rmsnorm, lib.astra_silu_and_mul, lib.astra_merge_attn_states_lse):
        f.restype = i32
    return lib


def _f64(t):
    return t.to(torch.float64).numpy()


def validate(lib) -> dict:
    """max_i d(S'(x_i), y_i) <= eps over the suite; returns {'correct': bool, 'worst_ulp': float, ...}."""
    worst, failures, cases = 0.0, [], 0
    stream = None

    def attempt(name, fn):
        nonlocal worst, cases
        cases += 1
        try:
            worst = max(worst, fn())
        except AssertionError as e:
            failures.append(f"{name}: {str(e)[:200]}")

    def rms(T, H, dtype, eps):
        inp = wl.rmsnorm_inputs(T, H, dtype, eps=eps, seed=T * 7 + H)
        x, r, w = inp.x.cuda(), inp.residual.cuda(), inp.weight.cuda()
        st = lib.astra_fused_add_rmsnorm(x.data_ptr(), r.data_ptr(), w.data_ptr(), T, H, eps, dtype, stream)
        assert st == 0, f"status {st}"
        oy, orr = oracle.fused_add_rmsnorm(wl.bits(inp.x), wl.bits(inp.residual), wl.bits(inp.weight), eps, dtype)
        assert np.array_equal(wl.bits(r.cpu()), orr), "residual sum is not bit-exact"
        return check_values(_f64(x.cpu()), oy, dtype)["max_err_ulp"]

    def silu(T, D, dtype):
        inp = wl.silu_inputs(T, D, dtype, std=2.0, seed=T + D)
        d = inp.input.cuda()
        out = torch.zeros((T, D), dtype=d.dtype, device="cuda")
        st = lib.astra_silu_and_mul(out.data_ptr(), d.data_ptr(), T, D, dtype, stream)
        assert st == 0, f"status {st}"
        return check_values(_f64(out.cpu()), oracle.silu_and_mul(wl.bits(inp.input), dtype), dtype)["max_err_ulp"]

    def merge(T, Hh, D, dtype):
        inp = wl.merge_inputs(T, Hh, D, dtype, seed=T + Hh + D, neg_inf_frac=0.02)
        va, vb, sa, sb = inp.v_a.cuda(), inp.v_b.cuda(), inp.lse_a.cuda(), inp.lse_b.cuda()
        vo, so = torch.zeros_like(va), torch.zeros_like(sa)
        st = lib.astra_merge_attn_states_lse(vo.data_ptr(), so.data_ptr(), va.data_ptr(), sa.data_ptr(),
                                             vb.data_ptr(), sb.data_ptr(), T, Hh, D, dtype, stream)
        assert st == 0, f"status {st}"
        ov, os_ = oracle.merge_attn_states_lse(wl.bits(inp.v_a), inp.lse_a.numpy(), wl.bits(inp.v_b),
                                               inp.lse_b.numpy(), dtype)
        floor = merge_floor(_f64(inp.v_a), inp.lse_a.numpy(), _f64(inp.v_b), inp.lse_b.numpy(), dtype)
        u = check_values(_f64(vo.cpu()), ov, dtype, extra=floor)["max_err_ulp"]
        check_lse(so.cpu().numpy(), os_)
        return u

    for dtype in (wl.BF16, wl.FP16):
        for T, H in ((16, 4096), (1, 8192), (33, 5120), (5, 4100), (3, 33), (256, 4096), (128, 11008)):
            attempt(f"rmsnorm[{T},{H}]/{dtype}", lambda: rms(T, H, dtype, 1e-6))
        for T, D in ((128, 14336), (16, 4096), (5, 1001), (3, 7), (64, 8192)):
            attempt(f"silu[{T},{D}]/{dtype}", lambda: silu(T, D, dtype))
        for T, Hh, D in ((512, 32, 128), (37, 5, 80), (9, 3, 7), (64, 40, 128), (16, 32, 256)):
            attempt(f"merge[{T},{Hh},{D}]/{dtype}", lambda: merge(T, Hh, D, dtype))
    torch.cuda.synchronize()
    return {"correct": not failures, "cases": cases, "worst_ulp": round(worst, 3), "failures": failures[:5]}


def profile(lib, warmup: int = 20, reps: int = 100) -> dict:
    """us per call on the Table 4 shapes (fp16), 20 warm-up + 100 timed launches per shape."""
    td, code = torch.float16, wl.FP16
    times = {}
    st = torch.cuda.current_stream().cuda_stream
    for kernel, shape, _, _ in wl.TABLE4:
        if kernel == "merge_attn_states_lse":
            T, Hh, D = shape
            va = torch.randn(shape, device="cuda").to(td); vb = torch.randn(shape, device="cuda").to(td)
            vo = torch.empty_like(va)
            sa = torch.rand((T, Hh), device="cuda") * 20 - 5; sb = torch.rand((T, Hh), device="cuda") * 20 - 5
            so = torch.empty_like(sa)
            call = lambda: lib.astra_merge_attn_states_lse(vo.data_ptr(), so.data_ptr(), va.data_ptr(), sa.data_ptr(),  # noqa: E731
                                                           vb.data_ptr(), sb.data_ptr(), T, Hh, D, code, st)
        elif kernel == "fused_add_rmsnorm":
            T, H = shape
            x = torch.randn(shape, device="cuda").to(td); r = torch.randn(shape, device="cuda").to(td)
            w = torch.ones((H,), device="cuda", dtype=td)
            call = lambda: lib.astra_fused_add_rmsnorm(x.data_ptr(), r.data_ptr(), w.data_ptr(), T, H, 1e-6, code, st)  # noqa: E731
        else:
            T, D = shape
            inp = torch.randn((T, 2 * D), device="cuda").to(td); out = torch.empty((T, D), device="cuda", dtype=td)
            call = lambda: lib.astra_silu_and_mul(out.data_ptr(), inp.data_ptr(), T, D, code, st)  # noqa: E731
        for _ in range(warmup):
            call()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(reps):
            call()
        b.record()
        torch.cuda.synchronize()
        times[f"{kernel}{list(shape)}"] = round(a.elapsed_time(b) * 1e3 / reps, 3)
    geo = math.exp(sum(math.log(v) for v in times.values()) / len(times))
    return {"us_per_call": times, "geomean_us": round(geo, 3)}


def main(argv=None) -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--lib", required=True)
    ap.add_argument("--baseline", default=None)
    ap.add_argument("--round", type=int, default=0)
    ap.add_argument("--oracle-lib", default=None,
                    help="use this build of the oracle instead of the stock one (the tool's own tests pass a "
                         "deliberately wrong copy to see validation fail)")
    args = ap.parse_args(argv)
    oracle.build()
    if args.oracle_lib:
        oracle._lib = oracle.declare(ctypes.CDLL(args.oracle_lib))
    lib = load(args.lib)
    rec = {"round": args.round, "candidate": os.path.basename(args.lib)}
    rec.update(validate(lib))
    rec["performance"] = profile(lib)
    if args.baseline:
        base = profile(load(args.baseline))
        ratios = [base["us_per_call"][k] / rec["performance"]["us_per_call"][k] for k in base["us_per_call"]]
        rec["geomean_speedup_over_baseline"] = round(math.exp(sum(math.log(v) for v in ratios) / len(ratios)), 3)
    print(json.dumps(rec))
    return 0 if rec["correct"] else 1


if __name__ == "__main__":
    sys.exit(main())
