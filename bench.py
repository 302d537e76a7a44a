#!/usr/bin/env python
"""Benchmark of the three memory-bound kernels on the Llama-3-8B prefill-shaped chain.

One step = fused_add_rmsnorm [T,4096] -> silu_and_mul [T,2*14336] -> merge_attn_states_lse
[T,32,128] at T = 8192, bf16, issued back to back on one stream (a timing sequence; no data flows
between the three).  The metric is achieved HBM bandwidth: algorithmic (minimum) bytes of the step
divided by device time over K back-to-back steps.  Per-kernel microseconds and GB/s come from K
back-to-back launches of each kernel alone (CUDA events on the launching stream), and the roofline
fraction is taken against the measured copy bandwidth of the GPU.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl astra|reference] [--no-sweep]

N > 1 (under torchrun, or started plainly, in which case the N ranks are spawned here): every rank runs its own T = 8192 batch (weak scaling; the operations are
independent per row, so there is no collective on the data path); time is the max over ranks.
`--impl reference` times the fp64 CPU oracle on the host cores instead (rank 0 only).
Exactly one JSON line is printed on stdout by rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2509_07506_b200 import multi  # noqa: E402
from paper_2509_07506_b200 import workloads as wl  # noqa: E402

METRIC = "achieved_hbm_bandwidth_llama3_8b_prefill_chain"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 7700.0   # HGX B200 data-sheet figure
HBM3E_SPEC_GBS = 8000.0    # 3996 MHz x 2 x 8192 bit: the interface's own ceiling
FALLBACK_HBM_GBS = 6650.0
L2_BYTES = 126 * 1024 * 1024
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_traffic_T4096.txt")


def ncu_traffic(kernel: str, tokens: int):
    """Per-launch memory traffic of `kernel` at `tokens` rows from the profiler counters kept beside
    the profile summaries: DRAM bytes read plus the bytes the SMs wrote into L2 (all of which reach
    DRAM, a part of them only after the launch has ended, which is why the DRAM write counter of a
    single profiled launch falls short).  The capture was taken at a smaller row count; traffic is
    proportional to rows.  None when the counters are missing (for instance after a kernel changed)."""
    try:
        with open(TRAFFIC_FILE) as fh:
            rec = json.load(fh)
        k = rec["kernels"][kernel]
        return round((k["dram_read_bytes"] + k["l2_write_bytes_from_sm"]) * tokens / rec["tokens"])
    except Exception:
        return None


def fractions(gbs: float, peak: float) -> dict:
    """A bandwidth against the three denominators in use: the copy bandwidth measured on this machine
    (the roofline the benchmark reports against), the data-sheet figure and the interface ceiling."""
    return {"frac_of_measured_peak": round(gbs / peak, 4), "frac_of_nominal_7700": round(gbs / NOMINAL_HBM_GBS, 4),
            "frac_of_hbm3e_spec_8000": round(gbs / HBM3E_SPEC_GBS, 4)}


def chain_bytes(T: int) -> dict:
    return {
        "fused_add_rmsnorm": wl.rmsnorm_bytes(T, wl.CHAIN_H),
        "silu_and_mul": wl.silu_bytes(T, wl.CHAIN_D),
        "merge_attn_states_lse": wl.merge_bytes(T, wl.CHAIN_HEADS, wl.CHAIN_HEAD_DIM),
    }


def measured_peak() -> tuple[float, str]:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, device copy)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (earlier copy measurement on this pool)"


# ---------------------------------------------------------------------------------------------
# clocks: nvidia-smi sampled in a child process while the timed regions run (read-only queries)
# ---------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.lines = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "25"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self, windows) -> dict:
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, line in self.lines:
            if not any(a <= ts <= b for a, b in windows):
                continue
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); smax.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {
            "sm_mhz": statistics.median(sm) if sm else None,
            "sm_max_mhz": max(smax) if smax else None,
            "reasons": sorted(reasons),
            "samples": len(sm),
        }


# ---------------------------------------------------------------------------------------------
# the CUDA arm
# ---------------------------------------------------------------------------------------------
def device_chain(T: int, seed_offset: int, dev):
    """Host (pinned) and device copies of one rank's chain inputs and outputs."""
    cfg = wl.config5(T) if seed_offset == 0 else _config5_seeded(T, 4 + 1000 * seed_offset)
    rms, silu, merge = cfg["rmsnorm"], cfg["silu"], cfg["merge"]
    host_in = {
        "x": rms.x, "residual": rms.residual, "weight": rms.weight, "silu_in": silu.input,
        "v_a": merge.v_a, "v_b": merge.v_b, "lse_a": merge.lse_a, "lse_b": merge.lse_b,
    }
    host_in = {k: v.pin_memory() for k, v in host_in.items()}
    d = {k: v.to(dev) for k, v in host_in.items()}
    d["silu_out"] = torch.empty((T, wl.CHAIN_D), dtype=torch.bfloat16, device=dev)
    d["v_out"] = torch.empty_like(d["v_a"])
    d["lse_out"] = torch.empty_like(d["lse_a"])
    host_out = {k: torch.empty(d[k].shape, dtype=d[k].dtype).pin_memory()
                for k in ("x", "residual", "silu_out", "v_out", "lse_out")}
    return cfg, host_in, d, host_out


def _config5_seeded(T, seed):
    g = torch.Generator(device="cpu"); g.manual_seed(seed)
    return {"rmsnorm": wl.rmsnorm_inputs(T, wl.CHAIN_H, wl.BF16, eps=1e-5, g=g),
            "silu": wl.silu_inputs(T, wl.CHAIN_D, wl.BF16, std=1.0, g=g),
            "merge": wl.merge_inputs(T, wl.CHAIN_HEADS, wl.CHAIN_HEAD_DIM, wl.BF16, -10.0, 20.0, 0.0, 0, g=g)}


def run_astra(args, rank: int, world: int, local_rank: int) -> dict | None:
    import paper_2509_07506_b200 as astra
    import torch.distributed as dist

    dev = torch.device("cuda", local_rank % torch.cuda.device_count())
    torch.cuda.set_device(dev)
    from paper_2509_07506_b200 import build as astra_build
    if rank == 0:
        astra_build.ensure_built()  # no-op when the library matches its sources; a missing or stale library is rebuilt or fatal
    if world > 1:
        dist.barrier()
    astra.load_library()  # fails loudly if the CUDA library is missing
    T = args.tokens
    eps = 1e-5
    cfg, host_in, d, host_out = device_chain(T, rank, dev)
    nbytes = chain_bytes(T)
    step_bytes = sum(nbytes.values())

    def step():
        astra.astra_fused_add_rmsnorm(d["x"], d["residual"], d["weight"], eps)
        astra.astra_silu_and_mul(d["silu_out"], d["silu_in"])
        astra.astra_merge_attn_states_lse(d["v_out"], d["lse_out"], d["v_a"], d["lse_a"], d["v_b"], d["lse_b"])

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(dev.index) if (rank == 0 and not args.no_clocks) else None
    K, W = args.steps, args.warmup
    for _ in range(W):
        step()
    barrier()

    # ---- device-resident timed region: K chain steps back to back, one event at each end ---------
    # (no events between the kernels: a stream marker between two launches would stop the next
    # kernel's launch from overlapping the previous kernel's drain)
    c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_wall0 = time.time()
    c0.record()
    for _ in range(K):
        step()
    c1.record()
    barrier()
    total_ms = c0.elapsed_time(c1)

    # ---- per-kernel timed regions: K back-to-back launches of each kernel alone ---------------------
    # Consecutive launches cycle through independent buffer sets covering eight L2 sizes (four sets for
    # the rmsnorm, five for the merge, two for silu), so no launch finds any of its own bytes in L2.
    def copies(keys, nbytes_one):
        return [{k: (d[k] if i == 0 else d[k].clone()) for k in keys} for i in range(n_cold_sets(nbytes_one))]

    rms_sets = copies(("x", "residual"), nbytes["fused_add_rmsnorm"])
    silu_sets = copies(("silu_out", "silu_in"), nbytes["silu_and_mul"])
    merge_sets = copies(("v_out", "lse_out", "v_a", "lse_a", "v_b", "lse_b"), nbytes["merge_attn_states_lse"])
    calls = {
        "fused_add_rmsnorm": (rms_sets, lambda b: astra.astra_fused_add_rmsnorm(b["x"], b["residual"], d["weight"], eps)),
        "silu_and_mul": (silu_sets, lambda b: astra.astra_silu_and_mul(b["silu_out"], b["silu_in"])),
        "merge_attn_states_lse": (merge_sets, lambda b: astra.astra_merge_attn_states_lse(
            b["v_out"], b["lse_out"], b["v_a"], b["lse_a"], b["v_b"], b["lse_b"])),
    }
    names = list(calls)
    kernel_ms = {}
    for n in names:
        sets, fn = calls[n]
        for i in range(W):
            fn(sets[i % len(sets)])
        k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        k0.record()
        for i in range(K):
            fn(sets[i % len(sets)])
        k1.record()
        torch.cuda.synchronize()
        kernel_ms[n] = k0.elapsed_time(k1) / K
    per_kernel_sets = {n: len(calls[n][0]) for n in names}
    del rms_sets, silu_sets, merge_sets, calls
    barrier()
    t_wall1 = time.time()

    # ---- end-to-end: pinned host -> device, three calls, device -> pinned host, every step --------
    Ke = max(1, min(K, args.e2e_steps))
    h2d = sum(v.numel() * v.element_size() for v in host_in.values())
    d2h = sum(v.numel() * v.element_size() for v in host_out.values())

    # Host-resident batch through the public API: the rows are cut into chunks that are uploaded,
    # processed and downloaded concurrently on three streams (HostStreamer); every step copies all of
    # its inputs from pinned host memory and all of its outputs back.
    from paper_2509_07506_b200.hoststream import HostStreamer
    pipe = HostStreamer(dev)
    chunk = max(1, min(T, args.e2e_chunk_rows))

    def e2e_step():
        for r0 in range(0, T, chunk):
            r1 = min(T, r0 + chunk)
            sl = slice(r0, r1)
            pipe.submit(("rmsnorm", r0),
                        [(d["x"][sl], host_in["x"][sl]), (d["residual"][sl], host_in["residual"][sl])]
                        + ([(d["weight"], host_in["weight"])] if r0 == 0 else []),
                        lambda sl=sl: astra.astra_fused_add_rmsnorm(d["x"][sl], d["residual"][sl], d["weight"], eps),
                        [(host_out["x"][sl], d["x"][sl]), (host_out["residual"][sl], d["residual"][sl])])
        for r0 in range(0, T, chunk):
            r1 = min(T, r0 + chunk)
            sl = slice(r0, r1)
            pipe.submit(("silu", r0), [(d["silu_in"][sl], host_in["silu_in"][sl])],
                        lambda sl=sl: astra.astra_silu_and_mul(d["silu_out"][sl], d["silu_in"][sl]),
                        [(host_out["silu_out"][sl], d["silu_out"][sl])])
        for r0 in range(0, T, chunk):
            r1 = min(T, r0 + chunk)
            sl = slice(r0, r1)
            pipe.submit(("merge", r0),
                        [(d[k][sl], host_in[k][sl]) for k in ("v_a", "v_b", "lse_a", "lse_b")],
                        lambda sl=sl: astra.astra_merge_attn_states_lse(d["v_out"][sl], d["lse_out"][sl], d["v_a"][sl],
                                                                        d["lse_a"][sl], d["v_b"][sl], d["lse_b"][sl]),
                        [(host_out["v_out"][sl], d["v_out"][sl]), (host_out["lse_out"][sl], d["lse_out"][sl])])

    pipe.wait_for(torch.cuda.current_stream())
    for _ in range(min(2, W)):
        e2e_step()
    pipe.synchronize()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_wall2 = time.time()
    e0.record(pipe.up)
    for _ in range(Ke):
        e2e_step()
    pipe.down.wait_stream(pipe.up)
    pipe.down.wait_stream(pipe.compute)
    e1.record(pipe.down)
    pipe.synchronize()
    barrier()
    t_wall3 = time.time()
    e2e_ms = e0.elapsed_time(e1)

    # ---- max over ranks -------------------------------------------------------------------------
    times = multi.max_over_ranks([total_ms, e2e_ms] + [kernel_ms[n] for n in names],
                                 device=dev if args.backend == "nccl" else "cpu")
    total_ms, e2e_ms = float(times[0]), float(times[1])
    kernel_ms = {n: float(times[2 + j]) for j, n in enumerate(names)}

    if sampler is not None:
        sampler.stop()
    if rank != 0:
        return None

    peak, peak_source = measured_peak()
    value = multi.aggregate_rate(step_bytes, world, K, total_ms) / 1e9
    per_kernel = {}
    for n in names:
        gbs = nbytes[n] / (kernel_ms[n] * 1e-3) / 1e9
        per_kernel[n] = {"us_per_call": round(kernel_ms[n] * 1e3, 2), "algorithmic_bytes": nbytes[n],
                         "gbs": round(gbs, 1), **fractions(gbs, peak), "ncu_traffic_bytes": ncu_traffic(n, T)}
    dominant = max(names, key=lambda n: kernel_ms[n])
    dom_gbs = nbytes[dominant] / (kernel_ms[dominant] * 1e-3) / 1e9
    result = {
        "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": round(total_ms / K, 5), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "storage_dtype": "bf16", "data": "synthetic",
        "config": {
            "workload": chain_workload_name(T),
            "tokens_per_gpu": T, "seed": 4,
            "l2_policy": "inputs larger than L2: each step touches %.0f MB (L2 is 126 MB) and every kernel's "
                         "own working set exceeds L2, so nothing is re-used across launches" % (step_bytes / 1e6),
            "parallelism": "rows sharded across GPUs, no collective" if world > 1 else "single GPU",
        },
        "per_kernel": per_kernel,
        "per_kernel_how": f"each kernel alone: {K} back-to-back launches between two CUDA events, after the chain region, "
                          f"cycling through {per_kernel_sets} independent buffer sets (the cycle covers eight L2 sizes)",
        "roofline": {"bound": "hbm", "kernel": dominant, "achieved": round(dom_gbs, 1), "peak": peak,
                     "unit": "GB/s", "frac": round(dom_gbs / peak, 4), "traffic": ncu_traffic(dominant, T),
                     "traffic_how": "ncu, per launch: dram__bytes_read.sum + bytes written into L2 by the SMs "
                                    "(lts__t_sectors_srcunit_tex_op_write.sum x 32), captured at T=4096 and scaled by rows",
                     "peak_source": peak_source, "algorithmic_bytes_per_launch": nbytes[dominant],
                     "frac_of_hbm3e_spec_8000": round(dom_gbs / HBM3E_SPEC_GBS, 4),
                     "frac_of_nominal_7700": round(dom_gbs / NOMINAL_HBM_GBS, 4)},
        "e2e": {"value": round(world * step_bytes * Ke / (e2e_ms * 1e-3) / 1e9, 2), "unit": UNIT,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": Ke,
                "ms_per_step": round(e2e_ms / Ke, 3),
                "how": f"pinned host -> device, kernels, device -> pinned host for every tensor of every step, in "
                       f"{chunk}-row chunks pipelined over three streams (upload / compute / download)"},
        "gpu_launches": 6 * K + 3 * Ke * (-(-T // chunk)),  # chain + per-kernel regions + chunked end-to-end steps
        "launcher": os.environ.get("ASTRA_BENCH_LAUNCHER", "external launcher" if world > 1 else "single process"),
        "clocks": sampler.summary([(t_wall0, t_wall1), (t_wall2, t_wall3)]) if sampler else None,
    }
    if world == 1 and not args.no_sweep:
        result["shape_sweep"] = shape_sweep(astra, dev, peak)
        result["table4"] = table4_sweep(astra, dev, peak)
        result["strided_variants"] = strided_variants(astra, dev, peak)
        result["decode_chain"] = decode_chain(astra, dev)
        result["fp32_variants"] = fp32_variants(astra, dev, peak)
        result["rmsnorm_cost_model"] = rmsnorm_cost_model(astra, dev, peak)
        result["allreduce_rmsnorm"] = allreduce_variants(astra, dev, peak)
    if world == 1 and not args.no_ablation:
        from paper_2509_07506_b200 import ablation
        astra_build.ensure_built(ablation=True)
        abl = ablation.run("fp16", dev)
        result["ablation"] = {"what": "the paper's baseline/optimised design pairs (Section 5.3) rebuilt for sm_100a, "
                                      "timed beside this library on the Table 4 shapes and the three chain shapes",
                              "summary": abl["summary"], "rows": abl["rows"], "timing": abl["timing"]}
    if world == 1 and not args.no_cpu:
        result["cpu_baseline"] = oracle_baseline(cfg, rows=min(args.cpu_rows, T))
        result["cpu_baseline"]["gpu_vs_oracle"] = oracle_agreement(astra, cfg, dev, rows=min(256, T))
    return result


def _time_launches(fn, reps=100, warmup=20):
    """Paper protocol: 20 warm-up launches, 100 timed, back to back; median of 5 batches (us/call)."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    out = []
    for _ in range(5):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        out.append(a.elapsed_time(b) * 1e3 / reps)
    return statistics.median(out)


COLD_FOOTPRINT = 8 * L2_BYTES


def n_cold_sets(nbytes: int) -> int:
    """Buffer sets to cycle through so that no launch finds anything of its own in L2: one when a single
    launch already streams eight L2 sizes, otherwise at least two and enough that the cycle covers
    eight L2 sizes (at most 64 sets, so the smallest shapes stay partly L2-resident; they are
    latency-bound either way).  The L2 of this part does not evict in strict LRU order: with a cycle of
    only 2-3 L2 sizes, lines written 250 MB earlier were still found there ([8192, 4096] in place ran
    at 36.4 us on one 268 MB set, 40.2 us on two, 40.8 us on four); from a cycle of about 8 L2 sizes on
    the times stop changing."""
    if nbytes >= COLD_FOOTPRINT:
        return 1
    return max(2, min(64, -(-COLD_FOOTPRINT // max(1, nbytes))))


def _rotating(make, nbytes: int):
    """Independent buffer sets for L2-cold timing (see n_cold_sets)."""
    return [make() for _ in range(n_cold_sets(nbytes))]


def _time_sets(call, sets):
    """us/call, cycling through the buffer sets (one set: L2-hot; several: every launch misses L2)."""
    state = {"i": 0}

    def fn():
        call(sets[state["i"] % len(sets)])
        state["i"] += 1
    return _time_launches(fn)


def _time_graph(call, sets, launches=100):
    """us/call on the device alone: `launches` calls captured into one CUDA graph (cycling through the
    buffer sets), replayed; removes the host's per-call cost, which dominates the small shapes."""
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


def shape_sweep(astra, dev, peak) -> list:
    """us/call for configs[0..2] and every point of the fused_add_rmsnorm sweep (configs[3]).
    `us_hot` repeats one buffer set (it stays in L2 when it fits); `us_cold` cycles through enough
    sets to defeat L2 (n_cold_sets); `*_graph` are the same launches replayed from a CUDA graph (device
    time only).  Shapes that stream more than two L2 sizes carry the roofline fraction of their L2-cold
    time; the small ones are launch-latency bound and are reported in us only."""
    rows = []

    def add(kernel, dtype, shape, nbytes, make, call):
        one = [make()]
        big = nbytes >= COLD_FOOTPRINT
        many = one if big else _rotating(make, nbytes)
        hot = _time_sets(call, one)
        cold = hot if big else _time_sets(call, many)
        row = {"kernel": kernel, "dtype": wl.DTYPE_NAME[dtype], "shape": shape, "algorithmic_bytes": nbytes,
               "us_hot": round(hot, 2), "us_cold": round(cold, 2)}
        if not big:  # device time without the host's launch cost
            row["us_hot_graph"] = round(_time_graph(call, one), 2)
            row["us_cold_graph"] = round(_time_graph(call, many), 2)
        best = cold if big else row["us_cold_graph"]
        gbs = nbytes / (best * 1e-6) / 1e9
        row["gbs_cold"] = round(gbs, 1)
        if nbytes > 2 * L2_BYTES:      # streaming sizes carry the roofline fraction (of the L2-cold time)
            row.update(fractions(gbs, peak))
        else:
            row["frac_of_measured_peak"] = None
        rows.append(row)

    def rms(dtype, T, H):
        td = wl.torch_dtype(dtype)
        make = lambda: (torch.randn((T, H), device=dev).to(td), torch.randn((T, H), device=dev).to(td),  # noqa: E731
                        torch.ones((H,), device=dev, dtype=td))
        add("fused_add_rmsnorm", dtype, [T, H], wl.rmsnorm_bytes(T, H), make,
            lambda b: astra.astra_fused_add_rmsnorm(b[0], b[1], b[2], 1e-5))

    rms(wl.BF16, 16, 4096)                                            # configs[0]
    T, D = 128, wl.CHAIN_D                                            # configs[1]
    add("silu_and_mul", wl.BF16, [T, 2 * D], wl.silu_bytes(T, D),
        lambda: (torch.empty((T, D), device=dev, dtype=torch.bfloat16),
                 (2 * torch.randn((T, 2 * D), device=dev)).to(torch.bfloat16)),
        lambda b: astra.astra_silu_and_mul(b[0], b[1]))
    T, Hh, Dh = 512, 32, 128                                          # configs[2]
    add("merge_attn_states_lse", wl.BF16, [T, Hh, Dh], wl.merge_bytes(T, Hh, Dh),
        lambda: (torch.empty((T, Hh, Dh), device=dev, dtype=torch.bfloat16), torch.empty((T, Hh), device=dev),
                 torch.randn((T, Hh, Dh), device=dev).to(torch.bfloat16), torch.rand((T, Hh), device=dev) * 20 - 5,
                 torch.randn((T, Hh, Dh), device=dev).to(torch.bfloat16), torch.rand((T, Hh), device=dev) * 20 - 5),
        lambda b: astra.astra_merge_attn_states_lse(b[0], b[1], b[2], b[3], b[4], b[5]))
    for dtype in wl.SWEEP_DTYPES:                                     # configs[3]
        for T in wl.SWEEP_T:
            for H in wl.SWEEP_H:
                rms(dtype, T, H)
    return rows


def decode_chain(astra, dev) -> list:
    """The three-call chain at decode-sized token counts (launch-latency bound): us per chain step
    through the binding call by call, and replayed from a CUDA graph of 20 steps (device time; the
    kernels' dependent-launch hooks let each launch overlap the previous kernel's drain)."""
    rows = []
    bf = torch.bfloat16
    H, D, Hh, Dh = wl.CHAIN_H, wl.CHAIN_D, wl.CHAIN_HEADS, wl.CHAIN_HEAD_DIM
    for T in (1, 16, 64, 256):
        x = torch.randn((T, H), device=dev).to(bf); r = torch.randn((T, H), device=dev).to(bf)
        w = torch.ones((H,), device=dev, dtype=bf)
        si = torch.randn((T, 2 * D), device=dev).to(bf); so = torch.empty((T, D), device=dev, dtype=bf)
        va = torch.randn((T, Hh, Dh), device=dev).to(bf); vb = torch.randn((T, Hh, Dh), device=dev).to(bf)
        vo = torch.empty_like(va)
        sa = torch.rand((T, Hh), device=dev) * 30 - 10; sb = torch.rand((T, Hh), device=dev) * 30 - 10
        lo = torch.empty_like(sa)

        def step(_=None):
            astra.astra_fused_add_rmsnorm(x, r, w, 1e-5)
            astra.astra_silu_and_mul(so, si)
            astra.astra_merge_attn_states_lse(vo, lo, va, sa, vb, sb)

        prepared = [astra.prepare_fused_add_rmsnorm(x, r, w, 1e-5), astra.prepare_silu_and_mul(so, si),
                    astra.prepare_merge_attn_states_lse(vo, lo, va, sa, vb, sb)]

        def step_prepared(_=None):
            for call in prepared:
                call()

        eager = _time_launches(step)
        ready = _time_launches(step_prepared)
        graph = _time_graph(step, [None], launches=20)
        rows.append({"tokens": T, "us_per_step_eager": round(eager, 2), "us_per_step_prepared": round(ready, 2),
                     "us_per_step_graph": round(graph, 2)})
    return rows


def rmsnorm_cost_model(astra, dev, peak) -> list:
    """fused_add_rmsnorm, bf16: device time (CUDA graph of 100 launches, L2-cold) at seven token counts
    per hidden size, and the least-squares fit t = t0 + bytes / BW over them.  t0 is the fixed cost of
    a launch (ramp-up and drain of the grid, with the launch itself overlapped by the previous kernel's
    tail); BW is the streaming rate once the grid is in flight.  A mid-size shape's fraction of the
    peak is bytes / (t0 + bytes / BW) / peak: what is lost there is t0, not streaming rate."""
    td = torch.bfloat16
    out = []
    for H in wl.SWEEP_H:
        pts = []
        for T in (256, 512, 1024, 2048, 4096, 8192, 16384):
            nbytes = wl.rmsnorm_bytes(T, H)
            make = lambda: (torch.randn((T, H), device=dev).to(td), torch.randn((T, H), device=dev).to(td),  # noqa: E731
                            torch.ones((H,), device=dev, dtype=td))
            sets = _rotating(make, nbytes)
            us = _time_graph(lambda b: astra.astra_fused_add_rmsnorm(b[0], b[1], b[2], 1e-5), sets)
            pts.append((T, nbytes, us))
            del sets
        n = len(pts)
        sx = sum(p[1] for p in pts); sy = sum(p[2] for p in pts)
        sxx = sum(p[1] * p[1] for p in pts); sxy = sum(p[1] * p[2] for p in pts)
        slope = (n * sxy - sx * sy) / (n * sxx - sx * sx)      # us per byte
        t0 = (sy - slope * sx) / n
        bw = 1e-3 / slope                                      # GB/s
        out.append({"H": H, "t0_us": round(t0, 2), "bw_gbs": round(bw, 1), "bw_frac_of_measured_peak": round(bw / peak, 4),
                    "points": [{"T": T, "us": round(us, 2), "gbs": round(b / us / 1e3, 1),
                                "frac_of_measured_peak": round(b / us / 1e3 / peak, 4),
                                "model_us": round(t0 + slope * b, 2)} for T, b, us in pts]})
    return out


def allreduce_variants(astra, dev, peak) -> list:
    """astra_fused_allreduce_add_rmsnorm (the partial hidden states of N tensor-parallel ranks summed
    inside add + RMSNorm) with all partials in this GPU's memory: (N + 3) * T * H * 2 algorithmic bytes
    against the HBM roofline at the prefill shape, device microseconds at decode shapes, and beside each
    the separate-kernels route it replaces on one GPU (N - 1 torch adds, then astra_fused_add_rmsnorm).
    Over NVLink the partials of the other ranks would arrive at link speed instead; not measured here."""
    td = torch.bfloat16
    rows = []
    H = wl.CHAIN_H
    for T in (wl.CHAIN_T, 1024, 16):
        for n in (2, 4, 8):
            nbytes = wl.allreduce_rmsnorm_bytes(T, H, n)
            make = lambda: ([torch.randn((T, H), device=dev).to(td) for _ in range(n)], torch.randn((T, H), device=dev).to(td),  # noqa: E731
                            torch.empty((T, H), device=dev, dtype=td), torch.ones((H,), device=dev, dtype=td))
            big = nbytes > 2 * L2_BYTES   # carries a roofline fraction
            sets = _rotating(make, nbytes)
            fused = lambda b: astra.astra_fused_allreduce_add_rmsnorm(b[2], b[1], b[0], b[3], 1e-5)  # noqa: E731

            def separate(b):
                acc = b[2]
                torch.add(b[0][0], b[0][1], out=acc)
                for p in b[0][2:]:
                    acc.add_(p)
                astra.astra_fused_add_rmsnorm(acc, b[1], b[3], 1e-5)

            us = _time_graph(fused, sets)
            us_sep = _time_graph(separate, sets)
            gbs = nbytes / us / 1e3
            row = {"shape": [T, H], "n_parts": n, "algorithmic_bytes": nbytes, "us_device": round(us, 2),
                   "gbs": round(gbs, 1), "us_device_separate_kernels": round(us_sep, 2),
                   "speedup_over_separate_kernels": round(us_sep / us, 2)}
            if big:
                row.update(fractions(gbs, peak))
            rows.append(row)
            del sets
    # Two-shot form: one rank's call on its block of T / N rows, the results stored to N destinations
    # each (all of them in this GPU's memory here; over NVLink N - 1 of the N would be peer stores).
    T = wl.CHAIN_T
    for n in (2, 4, 8):
        Tb = T // n
        nbytes = wl.two_shot_rmsnorm_bytes(Tb, H, n, n, n)
        make = lambda: ([torch.randn((Tb, H), device=dev).to(td) for _ in range(n)], torch.randn((Tb, H), device=dev).to(td),  # noqa: E731
                        [torch.empty((Tb, H), device=dev, dtype=td) for _ in range(n)],
                        [torch.empty((Tb, H), device=dev, dtype=td) for _ in range(n - 1)], torch.ones((H,), device=dev, dtype=td))
        sets = _rotating(make, nbytes)
        call = lambda b: astra.astra_fused_allreduce_add_rmsnorm_ex(b[2], [b[1]] + b[3], b[1], b[0], b[4], 1e-5)  # noqa: E731
        us = _time_graph(call, sets)
        gbs = nbytes / us / 1e3
        rows.append({"form": "two-shot: one rank's row block, results stored to every rank's buffers",
                     "shape": [Tb, H], "of_batch": [T, H], "n_parts": n, "n_destinations": n,
                     "algorithmic_bytes": nbytes, "us_device": round(us, 2), "gbs": round(gbs, 1),
                     **(fractions(gbs, peak) if nbytes > 2 * L2_BYTES else {})})
        del sets
    return rows


def _variant_row(name, nbytes, make, call, peak) -> dict:
    """us/call (paper protocol, through the binding) cycling through L2-cold buffer sets."""
    sets = _rotating(make, nbytes)
    us = _time_sets(call, sets)
    gbs = nbytes / (us * 1e-6) / 1e9
    return {"call": name, "us_per_call": round(us, 2), "gbs": round(gbs, 1), "buffer_sets": len(sets),
            **fractions(gbs, peak)}


def strided_variants(astra, dev, peak) -> list:
    """The strided / out-of-place entry points at the chain shapes (T = 8192, bf16); each moves the
    same algorithmic bytes as its plain counterpart, so the same roofline applies."""
    T, H, D, Hh, Dh = wl.CHAIN_T, wl.CHAIN_H, wl.CHAIN_D, wl.CHAIN_HEADS, wl.CHAIN_HEAD_DIM
    bf = torch.bfloat16
    w = torch.ones((H,), device=dev, dtype=bf)
    rows = []
    rn = lambda *shape: torch.randn(shape, device=dev).to(bf)  # noqa: E731
    rows.append(_variant_row(
        "astra_fused_add_rmsnorm_ex out-of-place [8192,4096]", wl.rmsnorm_bytes(T, H),
        lambda: (torch.empty((T, H), device=dev, dtype=bf), torch.empty((T, H), device=dev, dtype=bf), rn(T, H), rn(T, H)),
        lambda b: astra.astra_fused_add_rmsnorm_ex(b[0], b[1], b[2], b[3], w, 1e-5), peak))

    def slices():
        wide = rn(T, 2 * H + 256)
        return wide[:, :H], wide[:, H + 128:2 * H + 128]
    rows.append(_variant_row(
        "astra_fused_add_rmsnorm_ex in place on slices of a [8192, 8448] buffer", wl.rmsnorm_bytes(T, H), slices,
        lambda b: astra.astra_fused_add_rmsnorm_ex(b[0], b[1], b[0], b[1], w, 1e-5), peak))
    rows.append(_variant_row(
        "astra_silu_and_mul_ex separate gate and up tensors [8192,14336]", wl.silu_bytes(T, D),
        lambda: (torch.empty((T, D), device=dev, dtype=bf), rn(T, D), rn(T, D)),
        lambda b: astra.astra_silu_and_mul_ex(b[0], b[1], b[2]), peak))
    rows.append(_variant_row(
        "astra_merge_attn_states_lse_ex head-major scores [8192,32,128]", wl.merge_bytes(T, Hh, Dh),
        lambda: (torch.empty((T, Hh, Dh), device=dev, dtype=bf), torch.empty((Hh, T), device=dev).t(), rn(T, Hh, Dh),
                 (torch.rand((Hh, T), device=dev) * 30 - 10).t(), rn(T, Hh, Dh), (torch.rand((Hh, T), device=dev) * 30 - 10).t()),
        lambda b: astra.astra_merge_attn_states_lse_ex(b[0], b[1], b[2], b[3], b[4], b[5]), peak))
    return rows


def fp32_variants(astra, dev, peak) -> list:
    """The three operations on fp32 storage at the chain shapes (twice the bytes of the bf16 calls)."""
    T, H, D, Hh, Dh = wl.CHAIN_T, wl.CHAIN_H, wl.CHAIN_D, wl.CHAIN_HEADS, wl.CHAIN_HEAD_DIM
    w = torch.ones((H,), device=dev)
    rn = lambda *shape: torch.randn(shape, device=dev)  # noqa: E731
    rows = [
        _variant_row("astra_fused_add_rmsnorm fp32 [8192,4096]", wl.rmsnorm_bytes(T, H, 4),
                     lambda: (rn(T, H), rn(T, H)),
                     lambda b: astra.astra_fused_add_rmsnorm(b[0], b[1], w, 1e-5), peak),
        _variant_row("astra_silu_and_mul fp32 [8192,2*14336]", wl.silu_bytes(T, D, 4),
                     lambda: (torch.empty((T, D), device=dev), rn(T, 2 * D)),
                     lambda b: astra.astra_silu_and_mul(b[0], b[1]), peak),
        _variant_row("astra_merge_attn_states_lse fp32 [8192,32,128]", wl.merge_bytes(T, Hh, Dh, 4),
                     lambda: (torch.empty((T, Hh, Dh), device=dev), torch.empty((T, Hh), device=dev), rn(T, Hh, Dh),
                              torch.rand((T, Hh), device=dev) * 30 - 10, rn(T, Hh, Dh), torch.rand((T, Hh), device=dev) * 30 - 10),
                     lambda b: astra.astra_merge_attn_states_lse(b[0], b[1], b[2], b[3], b[4], b[5]), peak),
    ]
    return rows


def table4_sweep(astra, dev, peak) -> list:
    """The paper's Table 4 shapes, fp16 (the type its fragments use): us/call through the binding
    (`us_eager`: every argument checked and converted per call; `us_prepared`: a prepared call
    re-issued), device us/call from a CUDA graph, L2-hot and L2-cold, beside the paper's H100 figures
    (measured inside a serving framework on another machine: context only)."""
    rows = []
    td = torch.float16
    for kernel, shape, h100_base, h100_opt in wl.TABLE4:
        if kernel == "merge_attn_states_lse":
            T, Hh, Dh = shape
            nbytes = wl.merge_bytes(T, Hh, Dh)
            make = lambda: (torch.empty((T, Hh, Dh), device=dev, dtype=td), torch.empty((T, Hh), device=dev),  # noqa: E731
                            torch.randn((T, Hh, Dh), device=dev).to(td), torch.rand((T, Hh), device=dev) * 20 - 5,
                            torch.randn((T, Hh, Dh), device=dev).to(td), torch.rand((T, Hh), device=dev) * 20 - 5)
            call = lambda b: astra.astra_merge_attn_states_lse(b[0], b[1], b[2], b[3], b[4], b[5])  # noqa: E731
            prep = lambda b: astra.prepare_merge_attn_states_lse(b[0], b[1], b[2], b[3], b[4], b[5])  # noqa: E731
        elif kernel == "fused_add_rmsnorm":
            T, H = shape
            nbytes = wl.rmsnorm_bytes(T, H)
            make = lambda: (torch.randn((T, H), device=dev).to(td), torch.randn((T, H), device=dev).to(td),  # noqa: E731
                            torch.ones((H,), device=dev, dtype=td))
            call = lambda b: astra.astra_fused_add_rmsnorm(b[0], b[1], b[2], 1e-6)  # noqa: E731
            prep = lambda b: astra.prepare_fused_add_rmsnorm(b[0], b[1], b[2], 1e-6)  # noqa: E731
        else:
            T, D = shape
            nbytes = wl.silu_bytes(T, D)
            make = lambda: (torch.empty((T, D), device=dev, dtype=td), (2 * torch.randn((T, 2 * D), device=dev)).to(td))  # noqa: E731
            call = lambda b: astra.astra_silu_and_mul(b[0], b[1])  # noqa: E731
            prep = lambda b: astra.prepare_silu_and_mul(b[0], b[1])  # noqa: E731
        one = [make()]
        many = _rotating(make, nbytes)
        ready = prep(one[0])
        rows.append({"kernel": kernel, "dtype": "fp16", "shape": list(shape), "algorithmic_bytes": nbytes,
                     "us_eager": round(_time_sets(call, one), 2),
                     "us_prepared": round(_time_launches(ready), 2),
                     "us_hot_graph": round(_time_graph(call, one), 2),
                     "us_cold_graph": round(_time_graph(call, many), 2),
                     "paper_h100_us_base": h100_base, "paper_h100_us_opt": h100_opt})
    return rows


# ---------------------------------------------------------------------------------------------
# the CPU arm: the oracle, as it stands, on the host cores
# ---------------------------------------------------------------------------------------------
def _oracle_pass(cfg, rows: int, nthreads: int) -> float:
    """One pass of the three oracle functions over the first `rows` rows/tokens; seconds."""
    import oracle
    rms, silu, merge = cfg["rmsnorm"], cfg["silu"], cfg["merge"]
    xb, rb, wb = wl.bits(rms.x[:rows]), wl.bits(rms.residual[:rows]), wl.bits(rms.weight)
    sb = wl.bits(silu.input[:rows])
    va, vb = wl.bits(merge.v_a[:rows]), wl.bits(merge.v_b[:rows])
    la, lb = merge.lse_a[:rows].numpy(), merge.lse_b[:rows].numpy()
    t0 = time.perf_counter()
    oracle.fused_add_rmsnorm(xb, rb, wb, rms.eps, rms.dtype, nthreads=nthreads)
    oracle.silu_and_mul(sb, silu.dtype, nthreads=nthreads)
    oracle.merge_attn_states_lse(va, la, vb, lb, merge.dtype, nthreads=nthreads)
    return time.perf_counter() - t0


def oracle_baseline(cfg, rows: int) -> dict:
    import oracle
    oracle.build()
    cores = len(os.sched_getaffinity(0))
    _oracle_pass(cfg, min(rows, 64), cores)  # load the library, touch the pages
    sec = min(_oracle_pass(cfg, rows, cores) for _ in range(2))
    b = sum(chain_bytes(rows).values())
    # the same oracle on one core, on a smaller sample (it is ~cores times slower)
    rows1 = max(1, min(rows, 512))
    sec1 = _oracle_pass(cfg, rows1, 1)
    single = {"value": round(sum(chain_bytes(rows1).values()) / sec1 / 1e9, 3), "unit": UNIT, "cores": 1,
              "sample": f"first {rows1} rows/tokens, one pass, {sec1:.2f} s"}
    return {"value": round(b / sec / 1e9, 3), "unit": UNIT, "cores": cores, "kind": "oracle", "single_thread": single,
            "sample": f"first {rows} rows/tokens of each of the three chain calls, best of 2 passes, "
                      f"{sec:.2f} s per pass, OpenMP over rows on all {cores} host cores",
            "seconds": round(sec, 3)}


def oracle_agreement(astra, cfg, dev, rows: int) -> dict:
    """Part of the CPU-baseline leg: the library's outputs on the first `rows` rows of the three chain
    calls against the oracle's, as the largest error in units of the storage type's spacing at the
    oracle's value (bf16 here; 0.5 is a correctly rounded result), the score error in absolute terms,
    and whether the residual sum agrees bit for bit."""
    import numpy as np
    import oracle
    rms, silu, merge = cfg["rmsnorm"], cfg["silu"], cfg["merge"]

    def spacing(v):
        _, e = np.frexp(np.abs(v))
        return np.ldexp(1.0, np.maximum(e - 1, -126) - 7)

    def worst(gpu, want):
        gpu = gpu.cpu().to(torch.float64).numpy()
        nz = want != 0
        return round(float(np.max(np.abs(gpu - want)[nz] / spacing(want[nz]))), 3)

    x, r, w = rms.x[:rows].to(dev), rms.residual[:rows].to(dev), rms.weight.to(dev)
    astra.astra_fused_add_rmsnorm(x, r, w, rms.eps)
    oy, orr = oracle.fused_add_rmsnorm(wl.bits(rms.x[:rows]), wl.bits(rms.residual[:rows]), wl.bits(rms.weight),
                                       rms.eps, rms.dtype)
    si = silu.input[:rows].to(dev)
    so = torch.empty((rows, si.shape[1] // 2), dtype=si.dtype, device=dev)
    astra.astra_silu_and_mul(so, si)
    osilu = oracle.silu_and_mul(wl.bits(silu.input[:rows]), silu.dtype)
    va, vb = merge.v_a[:rows].to(dev), merge.v_b[:rows].to(dev)
    sa, sb = merge.lse_a[:rows].to(dev), merge.lse_b[:rows].to(dev)
    vo, lo = torch.empty_like(va), torch.empty_like(sa)
    astra.astra_merge_attn_states_lse(vo, lo, va, sa, vb, sb)
    ov, ol = oracle.merge_attn_states_lse(wl.bits(merge.v_a[:rows]), merge.lse_a[:rows].numpy(),
                                          wl.bits(merge.v_b[:rows]), merge.lse_b[:rows].numpy(), merge.dtype)
    torch.cuda.synchronize()
    return {"rows": rows, "max_err_ulp": {"fused_add_rmsnorm": worst(x, oy), "silu_and_mul": worst(so, osilu),
                                          "merge_attn_states_lse": worst(vo, ov)},
            "residual_sum_bit_exact": bool(np.array_equal(wl.bits(r.cpu()), orr)),
            "max_lse_abs_err": float(np.max(np.abs(lo.cpu().to(torch.float64).numpy() - ol)))}


def chain_workload_name(T: int) -> str:
    return (f"configs[4]: Llama-3-8B prefill-shaped chain, T={T} per GPU, bf16: "
            f"fused_add_rmsnorm [{T},4096] -> silu_and_mul [{T},2*14336] -> "
            f"merge_attn_states_lse [{T},32,128]")


def run_reference(args, rank: int, world: int) -> dict | None:
    if rank != 0:
        return None
    import oracle
    oracle.build()
    cores = len(os.sched_getaffinity(0))
    probe_rows = 32
    cfg = wl.config5(wl.CHAIN_T) if args.cpu_rows > 1024 else wl.config5(1024)
    max_rows = min(cfg["rmsnorm"].x.shape[0], args.cpu_rows)
    _oracle_pass(cfg, probe_rows, cores)
    t_probe = min(_oracle_pass(cfg, probe_rows, cores) for _ in range(3))
    budget = 90.0  # seconds for the whole K + W run
    rows = int(budget / max(1, args.steps + args.warmup) / (t_probe / probe_rows))
    rows = max(1, min(rows, max_rows))
    for _ in range(args.warmup):
        _oracle_pass(cfg, rows, cores)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        _oracle_pass(cfg, rows, cores)
    sec = time.perf_counter() - t0
    b = sum(chain_bytes(rows).values())
    value = round(b * args.steps / sec / 1e9, 3)
    sample = (f"each step = the fp64 oracle over the first {rows} of {wl.CHAIN_T} rows/tokens of the three chain calls, "
              f"OpenMP over rows on {cores} host cores")
    return {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": max(args.gpus, world),
        "launcher": os.environ.get("ASTRA_BENCH_LAUNCHER", "external launcher" if world > 1 else "single process"),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(sec / args.steps * 1e3, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": chain_workload_name(wl.CHAIN_T), "sample": sample, "seed": 4},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


def main() -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", choices=["astra", "reference"], default="astra")
    ap.add_argument("--e2e-steps", type=int, default=10, help="steps of the host-to-host timed region")
    ap.add_argument("--e2e-chunk-rows", type=int, default=2048, help="rows per upload/compute/download chunk")
    ap.add_argument("--cpu-rows", type=int, default=8192, help="rows of the chain the CPU baseline covers")
    ap.add_argument("--no-sweep", action="store_true", help="skip the per-shape timings of configs[0..3]")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU (oracle) baseline leg")
    ap.add_argument("--no-ablation", action="store_true", help="skip the design-pair ablation timings")
    ap.add_argument("--no-clocks", action="store_true", help="do not sample clocks with nvidia-smi")
    ap.add_argument("--backend", choices=["nccl", "gloo"], default="nccl",
                    help="process-group backend for the timing reduction when WORLD_SIZE > 1 (gloo allows a "
                         "functional check of the multi-rank path with several ranks sharing one GPU)")
    ap.add_argument("--tokens", type=int, default=wl.CHAIN_T,
                    help="tokens per GPU; the benchmark's workload is the default (8192), smaller values "
                         "are for profiler captures")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3

    # `python bench.py --gpus N` without a launcher: start the N ranks of this node here (one process
    # per GPU, rendezvous over 127.0.0.1); under torchrun the ranks already exist.
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        if args.impl == "astra" and args.backend == "nccl" and torch.cuda.device_count() < args.gpus:
            print(f"bench.py: --gpus {args.gpus} needs {args.gpus} GPUs, this machine has {torch.cuda.device_count()}",
                  file=sys.stderr)
            return 1
        os.environ["ASTRA_BENCH_LAUNCHER"] = "self-spawned ranks"
        return multi.spawn_ranks([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], args.gpus)

    rank, world, local_rank = multi.env_rank_world()

    if args.impl == "reference":
        res = run_reference(args, rank, world)
        if res is not None:
            print(json.dumps(res), flush=True)
        return 0

    if not torch.cuda.is_available():
        print("bench.py: no CUDA device; the CUDA library has no CPU fallback", file=sys.stderr)
        return 1
    if world > 1:
        multi.init_process_group(args.backend, torch.device("cuda", local_rank % torch.cuda.device_count()))
    try:
        res = run_astra(args, rank, world, local_rank)
    finally:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
    if res is not None:
        print(json.dumps(res), flush=True)
    return 0


if __name__ == "__main__":
    sys.exit(main())
