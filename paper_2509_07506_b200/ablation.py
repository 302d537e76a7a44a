"""The paper's case-study design pairs on B200: binding of ``include/astra_ablation.h`` and a runner
that reproduces the paper's headline quantity, the speedup of the optimised design over the
baseline design per shape and as a geometric mean (Section 3.1), with this library's own kernels
timed beside them.

    python -m paper_2509_07506_b200.ablation [--dtype fp16|bf16] [--json]

Shapes: the twelve of the paper's per-shape study (Table 4) plus the three large chain shapes.
Times are device microseconds from a CUDA graph of 100 launches (cold: cycling through enough
buffer sets to exceed L2), so host launch cost does not blur the comparison.
"""
from __future__ import annotations

import ctypes
import json
import math
import os
import statistics
import sys
from typing import Optional

import torch

from . import binding
from . import workloads as wl

ABLATION_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libastra_ablation.so")
EXPORTED_SYMBOLS = (
    "astra_ablation_merge_attn_states_lse",
    "astra_ablation_fused_add_rmsnorm",
    "astra_ablation_silu_and_mul",
)
DESIGN_BASELINE = 0
DESIGN_OPTIMISED = 1

_lib = None


def load_library() -> ctypes.CDLL:
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(ABLATION_LIB_PATH):
        raise ImportError(f"{ABLATION_LIB_PATH} is missing: build it with `python -m paper_2509_07506_b200.build`")
    lib = ctypes.CDLL(ABLATION_LIB_PATH)
    vp, i64, i32, f32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_float
    lib.astra_ablation_merge_attn_states_lse.argtypes = [i32, vp, vp, vp, vp, vp, vp, i64, i64, i64, i32, vp]
    lib.astra_ablation_merge_attn_states_lse.restype = i32
    lib.astra_ablation_fused_add_rmsnorm.argtypes = [i32, vp, vp, vp, i64, i64, f32, i32, vp]
    lib.astra_ablation_fused_add_rmsnorm.restype = i32
    lib.astra_ablation_silu_and_mul.argtypes = [i32, vp, vp, i64, i64, i32, vp]
    lib.astra_ablation_silu_and_mul.restype = i32
    _lib = lib
    return lib


def _code16(t: torch.Tensor, name: str) -> int:
    """dtype code of a 16-bit tensor (the design pairs are built for the 16-bit storage types only)."""
    if t.dtype not in (torch.bfloat16, torch.float16):
        raise TypeError(f"{name} must be bfloat16 or float16, got {t.dtype}")
    return binding._code(t, name)


def _raise(st: int, where: str) -> None:
    if st != binding.ASTRA_OK:
        raise binding.AstraError(st, where)


def _stream(t: torch.Tensor, stream: Optional[torch.cuda.Stream]) -> int:
    return (stream if stream is not None else torch.cuda.current_stream(t.device)).cuda_stream


def astra_ablation_fused_add_rmsnorm(design: int, x, residual, weight, eps: float, stream=None) -> None:
    for t in (x, residual, weight):
        if not (t.is_cuda and t.is_contiguous() and t.dtype == x.dtype):
            raise TypeError("contiguous CUDA tensors of one dtype expected")
    T, H = x.shape
    _raise(load_library().astra_ablation_fused_add_rmsnorm(
        int(design), x.data_ptr(), residual.data_ptr(), weight.data_ptr(), T, H, float(eps),
        _code16(x, "x"), _stream(x, stream)), "astra_ablation_fused_add_rmsnorm")


def astra_ablation_silu_and_mul(design: int, out, input, stream=None) -> None:
    for t in (out, input):
        if not (t.is_cuda and t.is_contiguous() and t.dtype == input.dtype):
            raise TypeError("contiguous CUDA tensors of one dtype expected")
    T, D = input.shape[0], input.shape[1] // 2
    _raise(load_library().astra_ablation_silu_and_mul(
        int(design), out.data_ptr(), input.data_ptr(), T, D, _code16(input, "input"),
        _stream(input, stream)), "astra_ablation_silu_and_mul")


def astra_ablation_merge_attn_states_lse(design: int, v_out, lse_out, v_a, lse_a, v_b, lse_b, stream=None) -> None:
    for t in (v_out, lse_out, v_a, lse_a, v_b, lse_b):
        if not (t.is_cuda and t.is_contiguous()):
            raise TypeError("contiguous CUDA tensors expected")
    T, Hh, D = v_a.shape
    _raise(load_library().astra_ablation_merge_attn_states_lse(
        int(design), v_out.data_ptr(), lse_out.data_ptr(), v_a.data_ptr(), lse_a.data_ptr(), v_b.data_ptr(),
        lse_b.data_ptr(), T, Hh, D, _code16(v_a, "v_a"), _stream(v_a, stream)),
        "astra_ablation_merge_attn_states_lse")


# ---- runner -----------------------------------------------------------------------------------

L2_BYTES = 126 * 1024 * 1024


def _graph_us(call, sets, launches=100) -> float:
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for i in range(3):
            call(sets[i % len(sets)])
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for i in range(launches):
                call(sets[i % len(sets)])
        out = []
        for _ in range(7):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(side)
            graph.replay()
            b.record(side)
            side.synchronize()
            out.append(a.elapsed_time(b) * 1e3 / launches)
    torch.cuda.current_stream().wait_stream(side)
    return statistics.median(out[2:])


def _sets(make, nbytes):
    """Independent buffer sets to cycle through so that no launch finds its own bytes in L2: one if a
    single launch streams eight L2 sizes, otherwise at least two and enough to cover eight L2 sizes
    (this part's L2 keeps lines far longer than strict LRU eviction would)."""
    n = 1 if nbytes >= 8 * L2_BYTES else max(2, min(64, -(-8 * L2_BYTES // max(1, nbytes))))
    return [make() for _ in range(n)]


def geomean(values) -> float:
    values = list(values)
    return math.exp(sum(math.log(v) for v in values) / len(values))


def run(dtype_name: str = "fp16", dev: Optional[torch.device] = None) -> dict:
    """Times design 0, design 1 and this library's kernel on every shape; returns the table and the
    geometric-mean speedups per kernel and overall."""
    from . import astra_fused_add_rmsnorm, astra_merge_attn_states_lse, astra_silu_and_mul
    dev = dev or torch.device("cuda", torch.cuda.current_device())
    td = {"fp16": torch.float16, "bf16": torch.bfloat16}[dtype_name]
    shapes = [(k, tuple(sh), base, opt) for k, sh, base, opt in wl.TABLE4]
    shapes += [("merge_attn_states_lse", (wl.CHAIN_T, wl.CHAIN_HEADS, wl.CHAIN_HEAD_DIM), None, None),
               ("fused_add_rmsnorm", (wl.CHAIN_T, wl.CHAIN_H), None, None),
               ("silu_and_mul", (wl.CHAIN_T, wl.CHAIN_D), None, None)]
    rows = []
    for kernel, shape, h100_base, h100_opt in shapes:
        if kernel == "merge_attn_states_lse":
            T, Hh, Dh = shape
            nbytes = wl.merge_bytes(T, Hh, Dh)
            make = lambda: (torch.empty((T, Hh, Dh), device=dev, dtype=td), torch.empty((T, Hh), device=dev),  # noqa: E731
                            torch.randn((T, Hh, Dh), device=dev).to(td), torch.rand((T, Hh), device=dev) * 20 - 5,
                            torch.randn((T, Hh, Dh), device=dev).to(td), torch.rand((T, Hh), device=dev) * 20 - 5)
            calls = [lambda b, d=d: astra_ablation_merge_attn_states_lse(d, *b) for d in (0, 1)]
            calls.append(lambda b: astra_merge_attn_states_lse(*b))
        elif kernel == "fused_add_rmsnorm":
            T, H = shape
            nbytes = wl.rmsnorm_bytes(T, H)
            make = lambda: (torch.randn((T, H), device=dev).to(td), torch.randn((T, H), device=dev).to(td),  # noqa: E731
                            torch.ones((H,), device=dev, dtype=td))
            calls = [lambda b, d=d: astra_ablation_fused_add_rmsnorm(d, b[0], b[1], b[2], 1e-6) for d in (0, 1)]
            calls.append(lambda b: astra_fused_add_rmsnorm(b[0], b[1], b[2], 1e-6))
        else:
            T, D = shape
            nbytes = wl.silu_bytes(T, D)
            make = lambda: (torch.empty((T, D), device=dev, dtype=td), (2 * torch.randn((T, 2 * D), device=dev)).to(td))  # noqa: E731
            calls = [lambda b, d=d: astra_ablation_silu_and_mul(d, b[0], b[1]) for d in (0, 1)]
            calls.append(lambda b: astra_silu_and_mul(b[0], b[1]))
        sets = _sets(make, nbytes)
        us = [_graph_us(c, sets) for c in calls]
        rows.append({"kernel": kernel, "shape": list(shape), "dtype": dtype_name,
                     "us_baseline_design": round(us[0], 2), "us_optimised_design": round(us[1], 2),
                     "us_this_library": round(us[2], 2),
                     "speedup_optimised_over_baseline": round(us[0] / us[1], 3),
                     "speedup_this_library_over_baseline": round(us[0] / us[2], 3),
                     "paper_h100_us_base": h100_base, "paper_h100_us_opt": h100_opt,
                     "paper_h100_speedup": round(h100_base / h100_opt, 3) if h100_base else None})
        del sets
    summary = {}
    for k in ("merge_attn_states_lse", "fused_add_rmsnorm", "silu_and_mul"):
        sel = [r for r in rows if r["kernel"] == k]
        summary[k] = {
            "geomean_speedup_optimised_over_baseline": round(geomean(r["speedup_optimised_over_baseline"] for r in sel), 3),
            "geomean_speedup_this_library_over_baseline": round(geomean(r["speedup_this_library_over_baseline"] for r in sel), 3),
            "paper_h100_geomean_speedup_table4": round(geomean(r["paper_h100_speedup"] for r in sel if r["paper_h100_speedup"]), 3),
        }
    summary["all"] = {
        "geomean_speedup_optimised_over_baseline": round(geomean(r["speedup_optimised_over_baseline"] for r in rows), 3),
        "geomean_speedup_this_library_over_baseline": round(geomean(r["speedup_this_library_over_baseline"] for r in rows), 3),
    }
    return {"rows": rows, "summary": summary,
            "timing": "device us/call from a CUDA graph of 100 launches, cold L2 (rotating buffer sets), median of 5 replays"}


def main(argv=None) -> int:
    argv = list(sys.argv[1:] if argv is None else argv)
    dtype = "bf16" if "--dtype" in argv and argv[argv.index("--dtype") + 1] == "bf16" else "fp16"
    res = run(dtype)
    if "--json" in argv:
        print(json.dumps(res))
        return 0
    print(f"{'kernel':24s} {'shape':18s} {'base':>8s} {'opt':>8s} {'ours':>8s} {'opt/base':>9s} {'ours/base':>10s} {'paper':>7s}")
    for r in res["rows"]:
        print(f"{r['kernel']:24s} {str(r['shape']):18s} {r['us_baseline_design']:8.2f} {r['us_optimised_design']:8.2f} "
              f"{r['us_this_library']:8.2f} {r['speedup_optimised_over_baseline']:9.2f} "
              f"{r['speedup_this_library_over_baseline']:10.2f} {str(r['paper_h100_speedup']):>7s}")
    for k, v in res["summary"].items():
        print(k, v)
    return 0


if __name__ == "__main__":
    sys.exit(main())
