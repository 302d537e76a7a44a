"""The C ABI used the way a C or C++ serving runtime would use it: `c_consumer.c`, a plain C program
with only the CUDA runtime beside it (no Python, no torch in that process), runs one call of each
operation on inputs read from files; its outputs are compared with the oracle here, element by
element, with the same gates as the tests that go through the Python binding."""
import os
import subprocess

import numpy as np
import pytest
import torch

import oracle
from paper_2509_07506_b200 import build as astra_build
from paper_2509_07506_b200 import workloads as wl
from parity import check_lse, check_values, merge_floor, ulp

pytestmark = pytest.mark.gpu

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CUDA_HOME = os.environ.get("CUDA_HOME", "/usr/local/cuda")


@pytest.fixture(scope="module")
def consumer(tmp_path_factory):
    lib = astra_build.build()
    libdir = os.path.dirname(lib)
    exe = tmp_path_factory.mktemp("c_consumer") / "c_consumer"
    subprocess.check_call(["gcc", "-std=c99", "-O1", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"),
                           "-I", os.path.join(CUDA_HOME, "include"), os.path.join(HERE, "c_consumer.c"), "-o", str(exe),
                           "-L", libdir, "-lastra", f"-Wl,-rpath,{libdir}",
                           "-L", os.path.join(CUDA_HOME, "lib64"), "-lcudart", f"-Wl,-rpath,{os.path.join(CUDA_HOME, 'lib64')}"])
    return str(exe)


def load(path, dtype: int, shape) -> torch.Tensor:
    raw = np.fromfile(path, dtype=np.uint32 if dtype == wl.FP32 else np.uint16)
    return wl.from_bits(raw.reshape(shape), dtype)


@pytest.mark.parametrize("dtype", [wl.BF16, wl.FP16, wl.FP32])
def test_c_program_matches_the_oracle(consumer, tmp_path, dtype):
    T, H, D, Hh, Dh, N = 67, 4100, 1536, 5, 128, 3
    rms = wl.rmsnorm_inputs(T, H, dtype, eps=1e-5, seed=61)
    sil = wl.silu_inputs(T, D, dtype, seed=62)
    mer = wl.merge_inputs(T, Hh, Dh, dtype, seed=63, neg_inf_frac=0.05)
    ar = wl.allreduce_rmsnorm_inputs(T, H, N, dtype, eps=1e-5, seed=64)
    d = str(tmp_path)
    for name, t in (("x", rms.x), ("r", rms.residual), ("w", rms.weight), ("silu_in", sil.input), ("va", mer.v_a),
                    ("vb", mer.v_b), ("ar_r", ar.residual), *[(f"part{i}", p) for i, p in enumerate(ar.parts)]):
        wl.bits(t).tofile(os.path.join(d, name + ".bin"))
    mer.lse_a.numpy().tofile(os.path.join(d, "sa.bin"))
    mer.lse_b.numpy().tofile(os.path.join(d, "sb.bin"))
    run = subprocess.run([consumer, d, str(dtype), str(T), str(H), str(D), str(Hh), str(Dh), str(N)],
                         capture_output=True, text=True, timeout=300)
    assert run.returncode == 0 and run.stdout.strip() == "ok", (run.returncode, run.stdout, run.stderr)

    f64 = lambda t: t.to(torch.float64).numpy()  # noqa: E731
    oy, orr = oracle.fused_add_rmsnorm(wl.bits(rms.x), wl.bits(rms.residual), wl.bits(rms.weight), 1e-5, dtype)
    assert np.array_equal(wl.bits(load(os.path.join(d, "r_out.bin"), dtype, (T, H))), orr)
    check_values(f64(load(os.path.join(d, "y.bin"), dtype, (T, H))), oy, dtype, what="C caller: fused_add_rmsnorm")

    # the weight row of the all-reduce call is the rmsnorm's (the program passes the same buffer)
    oy, orr = oracle.fused_allreduce_add_rmsnorm([wl.bits(p) for p in ar.parts], wl.bits(ar.residual), wl.bits(rms.weight),
                                                 1e-5, dtype)
    assert np.array_equal(wl.bits(load(os.path.join(d, "ar_r_out.bin"), dtype, (T, H))), orr)
    check_values(f64(load(os.path.join(d, "ar_y.bin"), dtype, (T, H))), oy, dtype, what="C caller: fused_allreduce_add_rmsnorm")

    want = oracle.silu_and_mul(wl.bits(sil.input), dtype)
    extra = 0.0
    if dtype == wl.FP32:  # the exponent's argument is rounded to binary32: |a| * 2^-24 relative (as in test_gpu_fp32)
        extra = 2.0 * np.abs(f64(sil.input[:, :D])) * ulp(np.where(want == 0, 1.0, want), dtype) * (want != 0)
    check_values(f64(load(os.path.join(d, "silu_out.bin"), dtype, (T, D))), want, dtype, extra=extra, what="C caller: silu_and_mul")

    ov, os_ = oracle.merge_attn_states_lse(wl.bits(mer.v_a), mer.lse_a.numpy(), wl.bits(mer.v_b), mer.lse_b.numpy(), dtype)
    floor = merge_floor(f64(mer.v_a), mer.lse_a.numpy(), f64(mer.v_b), mer.lse_b.numpy(), dtype)
    check_values(f64(load(os.path.join(d, "vo.bin"), dtype, (T, Hh, Dh))), ov, dtype, extra=floor, what="C caller: merge")
    check_lse(np.fromfile(os.path.join(d, "so.bin"), dtype=np.float32).reshape(T, Hh), os_, what="C caller: merge lse")
