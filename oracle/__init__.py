"""fp64 CPU oracle (test infrastructure only).

Thin ctypes loader for ``astra_oracle.c``: plain double-precision definitions of
fused_add_rmsnorm, silu_and_mul and merge_attn_states_lse (Astra paper, Table 1).
Only the tests, the smoke check and the CPU-baseline leg of the benchmark may
import this package; the CUDA library and its Python binding never do, and this
package imports nothing from them.

Arrays are numpy: storage patterns as ``uint16`` (bf16, fp16) or ``uint32`` (fp32), scores as ``float32``,
results as ``float64`` (and ``uint16`` for the bit-exact residual).
"""
from __future__ import annotations

import ctypes
import hashlib
import os
import re
import subprocess

import numpy as np

BF16 = 0
FP16 = 1
FP32 = 2

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "astra_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def _source_hash(src: str) -> str:
    with open(src, "rb") as fh:
        return hashlib.sha256(fh.read()).hexdigest()


def compile_source(src: str, out: str) -> str:
    """gcc command used for the oracle (no fast-math, no contraction).  The hash of the source is
    compiled in, so that a built library can be matched to the source beside it by content."""
    subprocess.check_call(
        ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
         "-ffp-contract=off", "-fno-fast-math", f'-DORACLE_BUILD_ID="{_source_hash(src)}"', "-o", out, src, "-lm"]
    )
    return out


def _embedded_hash(lib: str):
    try:
        with open(lib, "rb") as fh:
            m = re.search(rb"oracle-build-id:([0-9a-f]{64})", fh.read())
    except OSError:
        return None
    return m.group(1).decode() if m else None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc unless the built library already matches the source; returns the
    path of the shared object."""
    stale = _embedded_hash(_LIB) != _source_hash(_SRC)
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        compile_source(_SRC, tmp)
        os.replace(tmp, _LIB)
    return _LIB


def declare(lib):
    """Attach the C prototypes to a loaded oracle library (also used by the tests that load
    deliberately broken copies of the source)."""
    u16p = ctypes.c_void_p  # value tensors: uint16 patterns (bf16, fp16) or uint32 patterns (fp32)
    f32p = ctypes.POINTER(ctypes.c_float)
    f64p = ctypes.POINTER(ctypes.c_double)
    i64 = ctypes.c_int64
    lib.oracle_widen.argtypes = [ctypes.c_uint16, ctypes.c_int]
    lib.oracle_widen.restype = ctypes.c_double
    lib.oracle_round_to_storage.argtypes = [ctypes.c_double, ctypes.c_int]
    lib.oracle_round_to_storage.restype = ctypes.c_uint16
    lib.oracle_fused_add_rmsnorm.argtypes = [u16p, u16p, u16p, i64, i64, ctypes.c_float,
                                             ctypes.c_int, f64p, u16p, ctypes.c_int]
    lib.oracle_fused_add_rmsnorm.restype = None
    lib.oracle_fused_allreduce_add_rmsnorm.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.c_int, u16p, u16p, i64,
                                                       i64, ctypes.c_float, ctypes.c_int, f64p, u16p, ctypes.c_int]
    lib.oracle_fused_allreduce_add_rmsnorm.restype = None
    lib.oracle_silu_and_mul.argtypes = [u16p, i64, i64, ctypes.c_int, f64p, ctypes.c_int]
    lib.oracle_silu_and_mul.restype = None
    lib.oracle_merge_attn_states_lse.argtypes = [u16p, f32p, u16p, f32p, i64, i64, i64,
                                                 ctypes.c_int, f64p, f64p, ctypes.c_int]
    lib.oracle_merge_attn_states_lse.restype = None
    return lib


def _load():
    global _lib
    if _lib is None:
        _lib = declare(ctypes.CDLL(build()))
    return _lib


def _u16(a, shape, dtype=BF16):
    """Storage patterns of a value tensor: uint16 for the 16-bit types, uint32 for fp32."""
    a = np.ascontiguousarray(a)
    want = np.uint32 if dtype == FP32 else np.uint16
    if a.dtype != want:
        raise TypeError(f"expected {np.dtype(want).name} storage patterns, got {a.dtype}")
    if tuple(a.shape) != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {tuple(a.shape)}")
    return a


def _f32(a, shape):
    a = np.ascontiguousarray(a)
    if a.dtype != np.float32:
        raise TypeError(f"expected float32, got {a.dtype}")
    if tuple(a.shape) != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {tuple(a.shape)}")
    return a


def _ptr(a, ctype):
    if ctype is ctypes.c_uint16:  # value tensor: passed as void*
        return ctypes.c_void_p(a.ctypes.data)
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def widen(bits: int, dtype: int) -> float:
    """Exact value of one 16-bit storage pattern."""
    return float(_load().oracle_widen(int(bits), int(dtype)))


def round_to_storage(value: float, dtype: int) -> int:
    """Round one double to the storage format (nearest-even); returns the bit pattern."""
    return int(_load().oracle_round_to_storage(float(value), int(dtype)))


def fused_add_rmsnorm(x, residual, weight, eps: float, dtype: int, nthreads: int = 1):
    """Table 1, Kernel 2.  Returns (y float64 [T,H], residual_out storage patterns [T,H])."""
    x = np.ascontiguousarray(x)
    T, H = x.shape
    x = _u16(x, (T, H), dtype)
    residual = _u16(residual, (T, H), dtype)
    weight = _u16(weight, (H,), dtype)
    y = np.empty((T, H), dtype=np.float64)
    r_out = np.empty((T, H), dtype=x.dtype)
    _load().oracle_fused_add_rmsnorm(
        _ptr(x, ctypes.c_uint16), _ptr(residual, ctypes.c_uint16), _ptr(weight, ctypes.c_uint16),
        T, H, np.float32(eps).item(), int(dtype),
        _ptr(y, ctypes.c_double), _ptr(r_out, ctypes.c_uint16), int(nthreads))
    return y, r_out


def fused_allreduce_add_rmsnorm(parts, residual, weight, eps: float, dtype: int, nthreads: int = 1):
    """Kernel 2 of Table 1 on a hidden state given as N partial sums ``parts`` (a sequence of [T, H]
    pattern arrays in rank order): binary32 additions in rank order, the residual last.
    Returns (y float64 [T,H], residual_out storage patterns [T,H])."""
    if len(parts) < 1:
        raise ValueError("at least one partial is needed")
    first = np.ascontiguousarray(parts[0])
    T, H = first.shape
    parts = [_u16(p, (T, H), dtype) for p in parts]
    residual = _u16(residual, (T, H), dtype)
    weight = _u16(weight, (H,), dtype)
    table = (ctypes.c_void_p * len(parts))(*[p.ctypes.data for p in parts])
    y = np.empty((T, H), dtype=np.float64)
    r_out = np.empty((T, H), dtype=first.dtype)
    _load().oracle_fused_allreduce_add_rmsnorm(
        table, len(parts), _ptr(residual, ctypes.c_uint16), _ptr(weight, ctypes.c_uint16),
        T, H, np.float32(eps).item(), int(dtype),
        _ptr(y, ctypes.c_double), _ptr(r_out, ctypes.c_uint16), int(nthreads))
    return y, r_out


def silu_and_mul(inp, dtype: int, nthreads: int = 1):
    """Table 1, Kernel 3.  inp uint16 [T, 2D] = [gate | up]; returns float64 [T, D]."""
    inp = np.ascontiguousarray(inp)
    T, twoD = inp.shape
    if twoD % 2:
        raise ValueError("last dimension must be even")
    D = twoD // 2
    inp = _u16(inp, (T, twoD), dtype)
    out = np.empty((T, D), dtype=np.float64)
    _load().oracle_silu_and_mul(_ptr(inp, ctypes.c_uint16), T, D, int(dtype),
                                _ptr(out, ctypes.c_double), int(nthreads))
    return out


def merge_attn_states_lse(v_a, lse_a, v_b, lse_b, dtype: int, nthreads: int = 1):
    """Table 1, Kernel 1.  Returns (v_out float64 [T,Hh,D], lse_out float64 [T,Hh])."""
    v_a = np.ascontiguousarray(v_a)
    T, Hh, D = v_a.shape
    v_a = _u16(v_a, (T, Hh, D), dtype)
    v_b = _u16(v_b, (T, Hh, D), dtype)
    lse_a = _f32(lse_a, (T, Hh))
    lse_b = _f32(lse_b, (T, Hh))
    v_out = np.empty((T, Hh, D), dtype=np.float64)
    lse_out = np.empty((T, Hh), dtype=np.float64)
    _load().oracle_merge_attn_states_lse(
        _ptr(v_a, ctypes.c_uint16), _ptr(lse_a, ctypes.c_float),
        _ptr(v_b, ctypes.c_uint16), _ptr(lse_b, ctypes.c_float),
        T, Hh, D, int(dtype),
        _ptr(v_out, ctypes.c_double), _ptr(lse_out, ctypes.c_double), int(nthreads))
    return v_out, lse_out
