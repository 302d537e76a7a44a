"""Tolerances and comparison helpers for the GPU-vs-oracle parity tests.

Gates (oracle values are fp64; GPU values are the exact values of its 16-bit outputs):
  - residual sum: bit-for-bit.
  - bf16 outputs: |gpu - oracle| <= 2 * ulp_bf16(|oracle|), ulp_bf16(v) = 2^(floor(log2 v) - 7)
    (floored at the subnormal quantum 2^-133); oracle == 0 requires gpu == +-0.
  - fp16 outputs: |gpu - oracle| <= max(1e-3, 2 * ulp_fp16(|oracle|)), ulp_fp16(v) = 2^(floor(log2 v) - 10)
    (floored at 2^-24).  The plain 1e-3 cannot hold above |y| = 4, where half an fp16 ulp already
    exceeds it; the count of elements beyond the literal 1e-3 is returned for reporting.
  - fp32 outputs (storage without rounding, arithmetic with the GPU's approximate exp2,
    reciprocal and rsqrt, each good to about 2 ulp): |gpu - oracle| <= 16 * ulp_fp32(|oracle|) for
    rmsnorm and merge (plus the merge floor below).  For silu the exponent's argument |a|*log2(e)/2
    is rounded to binary32 before exp2, which costs |a| * 2^-24 relative: the gate there is
    (16 + 2*|a|) ulp, passed in through `extra`.
  - merge values: the blend a*Va + b*Vb can cancel, so the binary32 accumulation floor
    2^-22 * (|a*Va| + |b*Vb|) is added to the gate (4 times that for fp32 storage, where the
    weights' own few binary32 ulp are no longer hidden by the store's rounding).  `merge_floor` is
    the one definition of that term; every merge comparison in the repository uses it.
  - merged score: |gpu - oracle| <= 1e-5; -inf must be -inf.
"""
from __future__ import annotations

import numpy as np

BF16, FP16, FP32 = 0, 1, 2
_FRAC = {BF16: 7, FP16: 10, FP32: 23}
_EMIN = {BF16: -126, FP16: -14, FP32: -126}
_GATE_ULPS = {BF16: 2.0, FP16: 2.0, FP32: 16.0}


def ulp(v: np.ndarray, dtype: int) -> np.ndarray:
    """Spacing of the storage format at |v| (v != 0 finite); the subnormal quantum below the normals."""
    a = np.abs(np.asarray(v, dtype=np.float64))
    _, e = np.frexp(a)                      # a = m * 2^e with m in [0.5, 1): floor(log2 a) = e - 1, exactly
    e = np.maximum(e - 1, _EMIN[dtype])
    return np.ldexp(1.0, e - _FRAC[dtype])


def merge_floor(v_a, lse_a, v_b, lse_b, dtype: int) -> np.ndarray:
    """binary32 accumulation floor of the two-term blend, 2^-22 * (|a*Va| + |b*Vb|) with (a, b) =
    softmax([Sa, Sb]) in double precision (4 times that for fp32 storage).  v_*: [..., D] arrays of the
    inputs' exact values, lse_*: [...] scores.  An empty side (-inf score) has weight 0 and its payload,
    which may be Inf or NaN garbage, does not count; rows outside the domain (+inf or NaN scores) get 0."""
    sa = np.asarray(lse_a, dtype=np.float64)[..., None]
    sb = np.asarray(lse_b, dtype=np.float64)[..., None]
    with np.errstate(invalid="ignore", over="ignore"):
        m = np.maximum(sa, sb)
        m = np.where(np.isfinite(m), m, 0.0)
        ea, eb = np.exp(sa - m), np.exp(sb - m)
        a, b = ea / (ea + eb), eb / (ea + eb)
    a = np.nan_to_num(a, nan=0.0, posinf=0.0, neginf=0.0)
    b = np.nan_to_num(b, nan=0.0, posinf=0.0, neginf=0.0)
    va = np.nan_to_num(np.asarray(v_a, dtype=np.float64), nan=0.0, posinf=0.0, neginf=0.0)
    vb = np.nan_to_num(np.asarray(v_b, dtype=np.float64), nan=0.0, posinf=0.0, neginf=0.0)
    floor = 2.0 ** -22 * (np.abs(a * va) + np.abs(b * vb))
    return 4.0 * floor if dtype == FP32 else floor


def value_gate(oracle: np.ndarray, dtype: int, extra: np.ndarray | float = 0.0) -> np.ndarray:
    tol = _GATE_ULPS[dtype] * ulp(oracle, dtype)
    if dtype == FP16:
        tol = np.maximum(tol, 1e-3)
    tol = np.where(oracle == 0.0, 0.0, tol)
    return tol + extra


def check_values(gpu: np.ndarray, oracle: np.ndarray, dtype: int, extra=0.0, what: str = "") -> dict:
    """Assert the gate elementwise; returns summary statistics."""
    gpu = np.asarray(gpu, dtype=np.float64)
    oracle = np.asarray(oracle, dtype=np.float64)
    assert gpu.shape == oracle.shape, (gpu.shape, oracle.shape)
    nan_o = np.isnan(oracle)
    assert np.array_equal(np.isnan(gpu), nan_o), f"{what}: NaN pattern differs"
    fin = ~nan_o
    err = np.zeros_like(oracle)
    with np.errstate(invalid="ignore"):
        err[fin] = np.where(gpu[fin] == oracle[fin], 0.0, np.abs(gpu[fin] - oracle[fin]))
    tol = value_gate(np.where(fin, oracle, 1.0), dtype, extra)
    bad = fin & ~(err <= tol)
    if bad.any():
        i = np.flatnonzero(bad)[0]
        raise AssertionError(
            f"{what}: {bad.sum()} of {bad.size} elements outside the gate; first at flat index {i}: "
            f"gpu={gpu.ravel()[i]!r} oracle={oracle.ravel()[i]!r} err={err.ravel()[i]:.3e} "
            f"tol={np.broadcast_to(tol, oracle.shape).ravel()[i]:.3e}")
    u = ulp(np.where(fin & (oracle != 0), oracle, 1.0), dtype)
    return {
        "max_err_ulp": float(np.max(np.where(fin & (oracle != 0), err / u, 0.0))) if oracle.size else 0.0,
        "max_abs_err": float(err.max()) if oracle.size else 0.0,
        "beyond_literal_1e-3": int((err > 1e-3).sum()),
    }


def check_lse(gpu: np.ndarray, oracle: np.ndarray, what: str = "") -> float:
    gpu = np.asarray(gpu, dtype=np.float64)
    oracle = np.asarray(oracle, dtype=np.float64)
    assert gpu.shape == oracle.shape
    nan_o = np.isnan(oracle)
    assert np.array_equal(np.isnan(gpu), nan_o), f"{what}: NaN pattern differs"
    inf_o = np.isinf(oracle)
    assert np.array_equal(gpu[inf_o], oracle[inf_o]), f"{what}: infinite scores differ"
    fin = ~(nan_o | inf_o)
    err = np.abs(gpu[fin] - oracle[fin])
    assert np.all(err <= 1e-5), f"{what}: max score error {err.max():.3e} > 1e-5"
    return float(err.max()) if err.size else 0.0
