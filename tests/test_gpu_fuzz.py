"""Seeded random shapes around the launch-shape thresholds of the library, every element against the
oracle.  The entry points choose among many kernels and block shapes by row count, width, alignment
and (for the all-reduce form) the number of partials; the fixed parametrisations elsewhere name the
shapes their authors thought of, this file draws the rest: row counts at and next to every threshold,
widths at and next to every block-size limit, pointer offsets of every alignment class."""
import random

import pytest

from paper_2509_07506_b200 import workloads as wl
from test_gpu_allreduce import run_allreduce
from test_gpu_parity import run_merge, run_rmsnorm, run_silu

pytestmark = pytest.mark.gpu

BF16, FP16, FP32 = wl.BF16, wl.FP16, wl.FP32
MAX_ELEMS = 6_000_000     # per tensor, so that the oracle stays at a second or two per case

ROWS = [1, 2, 15, 16, 17, 31, 33, 63, 64, 65, 127, 128, 129, 148, 149, 295, 296, 297, 511, 512, 513, 1023, 1024, 1025,
        2047, 2048, 4095, 4096, 4097]
WIDTHS = [64, 250, 512, 1000, 1008, 1024, 1040, 2032, 2048, 2064, 3072, 4096, 4100, 4104, 4112, 5120, 6144, 7168, 7184,
          8192, 8208, 9216, 10240, 11008, 12288, 14336, 14352, 16384, 16400, 20480]
OFFSETS = [0, 0, 0, 16, 8, 4, 2, 1]   # elements: 32-byte aligned three times as often as each other class


def cases(seed: int, count: int, widths=WIDTHS):
    rng = random.Random(seed)
    out = []
    while len(out) < count:
        T, H = rng.choice(ROWS), rng.choice(widths)
        if T * H > MAX_ELEMS:
            continue
        out.append((T, H, rng.choice([BF16, BF16, FP16, FP32]), rng.choice(OFFSETS), rng.randrange(1 << 30)))
    return out


@pytest.mark.parametrize("T,H,dtype,offset,seed", cases(1, 120))
def test_fuzz_fused_add_rmsnorm(T, H, dtype, offset, seed):
    run_rmsnorm(wl.rmsnorm_inputs(T, H, dtype, eps=1e-5, seed=seed), offset=offset)


@pytest.mark.parametrize("T,D,dtype,offset,seed", cases(2, 90))
def test_fuzz_silu_and_mul(T, D, dtype, offset, seed):
    if 2 * T * D > MAX_ELEMS:
        T = max(1, MAX_ELEMS // (2 * D))
    run_silu(wl.silu_inputs(T, D, dtype, std=2.0, seed=seed), offset=offset)


@pytest.mark.parametrize("T,HD,dtype,offset,seed", cases(3, 60, widths=[64, 80, 128, 192, 256, 1024, 2560, 4096, 5120, 8192]))
def test_fuzz_merge_attn_states_lse(T, HD, dtype, offset, seed):
    rng = random.Random(seed)
    D = rng.choice([d for d in (16, 64, 80, 128, 256) if HD % d == 0])
    run_merge(wl.merge_inputs(T, HD // D, D, dtype, seed=seed, neg_inf_frac=0.03), offset=offset)


@pytest.mark.parametrize("T,H,dtype,offset,seed", cases(4, 120))
def test_fuzz_fused_allreduce_add_rmsnorm(T, H, dtype, offset, seed):
    n_parts = random.Random(seed).choice([1, 2, 3, 4, 5, 8, 9, 16])
    while T * H * n_parts > 3 * MAX_ELEMS:
        T = max(1, T // 2)
    run_allreduce(wl.allreduce_rmsnorm_inputs(T, H, n_parts, dtype, seed=seed), offset=offset)
