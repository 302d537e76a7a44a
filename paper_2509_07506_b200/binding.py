"""Python binding of the C ABI in ``include/astra.h`` (argument marshalling only).

Each function takes torch CUDA tensors, checks what the C side cannot see (device, dtype,
contiguity, shapes that agree), passes raw device pointers and the current stream to
``libastra.so`` and raises :class:`AstraError` on a non-zero status.  All arithmetic happens in
the CUDA kernels; there is no fallback of any kind: if the shared library is missing, importing
this module's functions raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libastra.so")

ASTRA_BF16 = 0
ASTRA_FP16 = 1

ASTRA_OK = 0
ASTRA_ERR_NULL_POINTER = 1
ASTRA_ERR_BAD_SHAPE = 2
ASTRA_ERR_BAD_DTYPE = 3
ASTRA_ERR_MISALIGNED = 4
ASTRA_ERR_CUDA = 5
ASTRA_ERR_OVERLAP = 6

EXPORTED_SYMBOLS = (
    "astra_fused_add_rmsnorm",
    "astra_silu_and_mul",
    "astra_merge_attn_states_lse",
    "astra_status_string",
)

_DTYPE_CODE = {torch.bfloat16: ASTRA_BF16, torch.float16: ASTRA_FP16}


class AstraError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({status_string(status)})")


_lib = None


def load_library() -> ctypes.CDLL:
    """dlopen ``libastra.so`` from the package directory and declare the prototypes."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2509_07506_b200.build` "
            "(there is no fallback implementation)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i64, i32, f32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_float
    lib.astra_fused_add_rmsnorm.argtypes = [vp, vp, vp, i64, i64, f32, i32, vp]
    lib.astra_fused_add_rmsnorm.restype = i32
    lib.astra_silu_and_mul.argtypes = [vp, vp, i64, i64, i32, vp]
    lib.astra_silu_and_mul.restype = i32
    lib.astra_merge_attn_states_lse.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, i32, vp]
    lib.astra_merge_attn_states_lse.restype = i32
    lib.astra_status_string.argtypes = [i32]
    lib.astra_status_string.restype = ctypes.c_char_p
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().astra_status_string(int(status)).decode()


def _check(t: torch.Tensor, name: str, dtype=None, shape=None) -> None:
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must have dtype {dtype}, got {t.dtype}")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} must have shape {tuple(shape)}, got {tuple(t.shape)}")


def _code(t: torch.Tensor, name: str) -> int:
    if t.dtype not in _DTYPE_CODE:
        raise TypeError(f"{name} must be bfloat16 or float16, got {t.dtype}")
    return _DTYPE_CODE[t.dtype]


def _stream(t: torch.Tensor, stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream(t.device)
    return s.cuda_stream


class _on_device:
    """Make the tensor's device current for the duration of the call (the C side launches on the
    current device); a no-op, and cheap, when it already is."""

    __slots__ = ("idx", "prev")

    def __init__(self, t: torch.Tensor):
        self.idx = t.device.index
        self.prev = None

    def __enter__(self):
        cur = torch.cuda.current_device()
        if self.idx is not None and self.idx != cur:
            self.prev = cur
            torch.cuda.set_device(self.idx)

    def __exit__(self, *exc):
        if self.prev is not None:
            torch.cuda.set_device(self.prev)
        return False


def astra_fused_add_rmsnorm(x: torch.Tensor, residual: torch.Tensor, weight: torch.Tensor,
                            eps: float, stream: Optional[torch.cuda.Stream] = None) -> None:
    """In place: residual <- x + residual, x <- RMSNorm(x + residual) * weight.  x, residual [T, H]."""
    _check(x, "x")
    code = _code(x, "x")
    if x.dim() != 2:
        raise ValueError("x must be [T, H]")
    T, H = x.shape
    _check(residual, "residual", x.dtype, (T, H))
    _check(weight, "weight", x.dtype, (H,))
    with _on_device(x):
        st = load_library().astra_fused_add_rmsnorm(
            x.data_ptr(), residual.data_ptr(), weight.data_ptr(), T, H, float(eps), code,
            _stream(x, stream))
    if st != ASTRA_OK:
        raise AstraError(st, "astra_fused_add_rmsnorm")


def astra_silu_and_mul(out: torch.Tensor, input: torch.Tensor,
                       stream: Optional[torch.cuda.Stream] = None) -> None:
    """out[T, D] <- SiLU(input[:, :D]) * input[:, D:]."""
    _check(input, "input")
    code = _code(input, "input")
    if input.dim() != 2 or input.shape[1] % 2:
        raise ValueError("input must be [T, 2*D]")
    T, D = input.shape[0], input.shape[1] // 2
    _check(out, "out", input.dtype, (T, D))
    with _on_device(input):
        st = load_library().astra_silu_and_mul(out.data_ptr(), input.data_ptr(), T, D, code,
                                               _stream(input, stream))
    if st != ASTRA_OK:
        raise AstraError(st, "astra_silu_and_mul")


def astra_merge_attn_states_lse(v_out: torch.Tensor, lse_out: Optional[torch.Tensor],
                                v_a: torch.Tensor, lse_a: torch.Tensor,
                                v_b: torch.Tensor, lse_b: torch.Tensor,
                                stream: Optional[torch.cuda.Stream] = None) -> None:
    """v_out, lse_out <- merge of (v_a, lse_a) and (v_b, lse_b).  v_* [T, Hh, D]; lse_* [T, Hh] fp32."""
    _check(v_a, "v_a")
    code = _code(v_a, "v_a")
    if v_a.dim() != 3:
        raise ValueError("v_a must be [T, Hh, D]")
    T, Hh, D = v_a.shape
    _check(v_b, "v_b", v_a.dtype, (T, Hh, D))
    _check(v_out, "v_out", v_a.dtype, (T, Hh, D))
    _check(lse_a, "lse_a", torch.float32, (T, Hh))
    _check(lse_b, "lse_b", torch.float32, (T, Hh))
    if lse_out is not None:
        _check(lse_out, "lse_out", torch.float32, (T, Hh))
    with _on_device(v_a):
        st = load_library().astra_merge_attn_states_lse(
            v_out.data_ptr(), lse_out.data_ptr() if lse_out is not None else None,
            v_a.data_ptr(), lse_a.data_ptr(), v_b.data_ptr(), lse_b.data_ptr(),
            T, Hh, D, code, _stream(v_a, stream))
    if st != ASTRA_OK:
        raise AstraError(st, "astra_merge_attn_states_lse")
