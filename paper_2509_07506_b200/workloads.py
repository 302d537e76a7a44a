"""Seeded synthetic inputs for the three operations (no arithmetic of the operations here).

Every tensor is drawn on the host from ``torch.Generator(device="cpu")`` in fp32, in a fixed
order, then cast (round-to-nearest-even) to the storage dtype.  The same host tensors feed the
CPU oracle (as 16-bit patterns) and are uploaded for the CUDA library, so both sides see
identical bits.  Shapes follow the Llama-family dimensions the paper draws its shapes from
(hidden 4096/5120/8192, intermediate 14336, 32 heads of 128).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, Optional

import numpy as np
import torch

BF16 = 0
FP16 = 1
FP32 = 2

_TORCH_DTYPE = {BF16: torch.bfloat16, FP16: torch.float16, FP32: torch.float32}
DTYPE_NAME = {BF16: "bf16", FP16: "fp16", FP32: "fp32"}
ELEM_BYTES = {BF16: 2, FP16: 2, FP32: 4}


def torch_dtype(dtype: int) -> torch.dtype:
    return _TORCH_DTYPE[dtype]


def bits(t: torch.Tensor) -> np.ndarray:
    """The storage patterns of a host tensor: uint16 for bf16/fp16, uint32 for fp32."""
    assert t.device.type == "cpu"
    if t.dtype == torch.float32:
        return t.contiguous().view(torch.int32).numpy().view(np.uint32)
    assert t.dtype in (torch.bfloat16, torch.float16)
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def from_bits(a: np.ndarray, dtype: int) -> torch.Tensor:
    """Inverse of :func:`bits`."""
    if dtype == FP32:
        return torch.from_numpy(np.ascontiguousarray(a).view(np.int32)).view(torch.float32)
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(_TORCH_DTYPE[dtype])


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    return g


def _randn(g, shape, dtype, mean=0.0, std=1.0) -> torch.Tensor:
    t = torch.randn(shape, generator=g, dtype=torch.float32)
    if std != 1.0:
        t.mul_(std)
    if mean != 0.0:
        t.add_(mean)
    return t.to(_TORCH_DTYPE[dtype])


@dataclass
class RmsnormInputs:
    x: torch.Tensor         # [T, H]
    residual: torch.Tensor  # [T, H]
    weight: torch.Tensor    # [H]
    eps: float
    dtype: int


@dataclass
class SiluInputs:
    input: torch.Tensor     # [T, 2D]: columns [0, D) gate, [D, 2D) up
    dtype: int


@dataclass
class MergeInputs:
    v_a: torch.Tensor       # [T, Hh, D]
    v_b: torch.Tensor       # [T, Hh, D]
    lse_a: torch.Tensor     # [T, Hh] fp32, natural log
    lse_b: torch.Tensor     # [T, Hh] fp32
    dtype: int


def rmsnorm_inputs(T: int, H: int, dtype: int = BF16, eps: float = 1e-6, seed: int = 0,
                   g: Optional[torch.Generator] = None) -> RmsnormInputs:
    """x, residual ~ N(0,1); weight ~ N(1, 0.1); drawn in that order."""
    g = g if g is not None else _gen(seed)
    x = _randn(g, (T, H), dtype)
    r = _randn(g, (T, H), dtype)
    w = _randn(g, (H,), dtype, mean=1.0, std=0.1)
    return RmsnormInputs(x, r, w, eps, dtype)


@dataclass
class AllreduceRmsnormInputs:
    parts: list             # n_parts tensors [T, H], rank order
    residual: torch.Tensor  # [T, H]
    weight: torch.Tensor    # [H]
    eps: float
    dtype: int


def allreduce_rmsnorm_inputs(T: int, H: int, n_parts: int, dtype: int = BF16, eps: float = 1e-5, seed: int = 6,
                             g: Optional[torch.Generator] = None) -> AllreduceRmsnormInputs:
    """The per-rank partial hidden states ~ N(0, 1/n_parts) each (so their sum is ~ N(0,1), as the
    hidden state of the one-GPU operation), then residual ~ N(0,1) and weight ~ N(1, 0.1); drawn in
    that order."""
    g = g if g is not None else _gen(seed)
    parts = [_randn(g, (T, H), dtype, std=float(n_parts) ** -0.5) for _ in range(n_parts)]
    r = _randn(g, (T, H), dtype)
    w = _randn(g, (H,), dtype, mean=1.0, std=0.1)
    return AllreduceRmsnormInputs(parts, r, w, eps, dtype)


def silu_inputs(T: int, D: int, dtype: int = BF16, std: float = 2.0, seed: int = 1,
                g: Optional[torch.Generator] = None) -> SiluInputs:
    """input [T, 2D] ~ N(0, std^2)."""
    g = g if g is not None else _gen(seed)
    return SiluInputs(_randn(g, (T, 2 * D), dtype, std=std), dtype)


def merge_inputs(T: int, Hh: int, D: int, dtype: int = BF16, lse_lo: float = -5.0,
                 lse_hi: float = 15.0, neg_inf_frac: float = 0.01, forced_both_neg_inf: int = 4,
                 seed: int = 2, g: Optional[torch.Generator] = None) -> MergeInputs:
    """v_a, v_b ~ N(0,1); lse_a, lse_b ~ U(lse_lo, lse_hi); then two independent masks with
    probability ``neg_inf_frac`` set entries to -inf; then ``forced_both_neg_inf`` fixed
    positions (evenly spaced) get -inf on both sides so that case is always present."""
    g = g if g is not None else _gen(seed)
    v_a = _randn(g, (T, Hh, D), dtype)
    v_b = _randn(g, (T, Hh, D), dtype)
    lse_a = torch.rand((T, Hh), generator=g, dtype=torch.float32) * (lse_hi - lse_lo) + lse_lo
    lse_b = torch.rand((T, Hh), generator=g, dtype=torch.float32) * (lse_hi - lse_lo) + lse_lo
    if neg_inf_frac > 0.0:
        mask_a = torch.rand((T, Hh), generator=g, dtype=torch.float32) < neg_inf_frac
        mask_b = torch.rand((T, Hh), generator=g, dtype=torch.float32) < neg_inf_frac
        lse_a[mask_a] = float("-inf")
        lse_b[mask_b] = float("-inf")
    n = T * Hh
    k = min(forced_both_neg_inf, n) if neg_inf_frac > 0.0 else 0
    for i in range(k):
        pos = (i * n) // k + (n // (2 * k))
        pos = min(pos, n - 1)
        lse_a.view(-1)[pos] = float("-inf")
        lse_b.view(-1)[pos] = float("-inf")
    return MergeInputs(v_a, v_b, lse_a, lse_b, dtype)


# ---- the five named configurations -------------------------------------------------------

SWEEP_T = (1, 64, 1024, 16384)
SWEEP_H = (4096, 5120, 8192, 4100)
SWEEP_DTYPES = (BF16, FP16)

CHAIN_T = 8192
CHAIN_H = 4096
CHAIN_D = 14336
CHAIN_HEADS = 32
CHAIN_HEAD_DIM = 128


def config1() -> RmsnormInputs:
    """fused_add_rmsnorm bf16 [16, 4096], eps 1e-6, seed 0."""
    return rmsnorm_inputs(16, 4096, BF16, eps=1e-6, seed=0)


def config2() -> SiluInputs:
    """silu_and_mul bf16 [128, 2*14336] ~ N(0, 2^2), seed 1."""
    return silu_inputs(128, 14336, BF16, std=2.0, seed=1)


def config3() -> MergeInputs:
    """merge_attn_states_lse bf16 [512, 32, 128], lse ~ U(-5, 15) with 1% -inf, seed 2."""
    return merge_inputs(512, 32, 128, BF16, -5.0, 15.0, 0.01, 4, seed=2)


def config4_point(dtype: int, T: int, H: int) -> RmsnormInputs:
    """One point of the fused_add_rmsnorm sweep; eps 1e-5; generator reseeded (3) per point."""
    return rmsnorm_inputs(T, H, dtype, eps=1e-5, seed=3)


def config5(T: int = CHAIN_T) -> Dict[str, object]:
    """Llama-3-8B prefill-shaped chain, bf16, one generator seeded 4 for all three calls.
    The three calls are a timing sequence; no data flows between them (the shapes differ)."""
    g = _gen(4)
    rms = rmsnorm_inputs(T, CHAIN_H, BF16, eps=1e-5, g=g)
    silu = silu_inputs(T, CHAIN_D, BF16, std=1.0, g=g)
    merge = merge_inputs(T, CHAIN_HEADS, CHAIN_HEAD_DIM, BF16, -10.0, 20.0, 0.0, 0, g=g)
    return {"rmsnorm": rms, "silu": silu, "merge": merge}


# ---- the twelve shapes of the paper's Table 4 (per-shape study) -----------------------------
# (kernel, shape, paper's H100 time of its baseline kernel in us, of its optimised kernel in us).
# The paper does not state the precision of these runs; its code fragments use 16-bit floats.
# Shapes are [seq_len, heads, head_dim] for the merge and [batch, hidden] for the other two; for
# silu_and_mul, hidden is read as the output width D (the input row is 2*D wide).
TABLE4 = (
    ("merge_attn_states_lse", (512, 32, 256), 32.9, 22.6),
    ("merge_attn_states_lse", (512, 40, 128), 32.4, 20.6),
    ("merge_attn_states_lse", (768, 32, 256), 32.5, 32.5),
    ("merge_attn_states_lse", (512, 64, 128), 32.0, 28.2),
    ("fused_add_rmsnorm", (256, 4096), 24.3, 18.3),
    ("fused_add_rmsnorm", (1024, 4096), 34.0, 28.3),
    ("fused_add_rmsnorm", (128, 11008), 25.0, 19.4),
    ("fused_add_rmsnorm", (512, 14336), 46.1, 43.0),
    ("silu_and_mul", (16, 4096), 20.9, 14.2),
    ("silu_and_mul", (32, 5120), 20.3, 13.7),
    ("silu_and_mul", (64, 8192), 20.3, 13.5),
    ("silu_and_mul", (16, 12288), 20.4, 13.6),
)


def table4_inputs(kernel: str, shape, dtype: int = BF16, seed: int = 5):
    """Seeded inputs for one Table 4 shape (same value distributions as configs[0..2])."""
    if kernel == "merge_attn_states_lse":
        return merge_inputs(shape[0], shape[1], shape[2], dtype, seed=seed)
    if kernel == "fused_add_rmsnorm":
        return rmsnorm_inputs(shape[0], shape[1], dtype, eps=1e-6, seed=seed)
    if kernel == "silu_and_mul":
        return silu_inputs(shape[0], shape[1], dtype, std=2.0, seed=seed)
    raise ValueError(kernel)


# ---- algorithmic (minimum) bytes per call -------------------------------------------------

def rmsnorm_bytes(T: int, H: int, elem: int = 2) -> int:
    """Read x and r, write y and r', read the weight once."""
    return 4 * T * H * elem + H * elem


def allreduce_rmsnorm_bytes(T: int, H: int, n_parts: int, elem: int = 2) -> int:
    """Read the n_parts partials and r, write y and r', read the weight once."""
    return (n_parts + 3) * T * H * elem + H * elem


def two_shot_rmsnorm_bytes(T_block: int, H: int, n_parts: int, n_y: int, n_r: int, elem: int = 2) -> int:
    """The two-shot form on a block of rows: read the n_parts partials and r, write y to n_y
    destinations and r' to n_r, read the weight once."""
    return (n_parts + 1 + n_y + n_r) * T_block * H * elem + H * elem


def silu_bytes(T: int, D: int, elem: int = 2) -> int:
    """Read gate and up, write out."""
    return 3 * T * D * elem


def merge_bytes(T: int, Hh: int, D: int, elem: int = 2) -> int:
    """Read v_a and v_b, write v_out; read two fp32 scores and write one per (token, head)."""
    return 3 * T * Hh * D * elem + 3 * T * Hh * 4
