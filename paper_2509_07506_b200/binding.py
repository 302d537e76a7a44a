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
FASTCALL_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "_astra_fastcall.so")

ASTRA_BF16 = 0
ASTRA_FP16 = 1
ASTRA_FP32 = 2

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
    "astra_fused_add_rmsnorm_ex",
    "astra_silu_and_mul_ex",
    "astra_merge_attn_states_lse_ex",
    "astra_fused_allreduce_add_rmsnorm",
    "astra_fused_allreduce_add_rmsnorm_ex",
    "astra_status_string",
    "astra_build_id",
)

_DTYPE_CODE = {torch.bfloat16: ASTRA_BF16, torch.float16: ASTRA_FP16, torch.float32: ASTRA_FP32}


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
    lib.astra_fused_add_rmsnorm_ex.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, i64, i64, i64, f32, i32, vp]
    lib.astra_fused_add_rmsnorm_ex.restype = i32
    lib.astra_silu_and_mul_ex.argtypes = [vp, vp, vp, i64, i64, i64, i64, i64, i32, vp]
    lib.astra_silu_and_mul_ex.restype = i32
    lib.astra_merge_attn_states_lse_ex.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64,
                                                   ctypes.POINTER(ctypes.c_int64), i32, vp]
    lib.astra_merge_attn_states_lse_ex.restype = i32
    lib.astra_fused_allreduce_add_rmsnorm.argtypes = [vp, vp, ctypes.POINTER(vp), i32, vp, i64, i64, f32, i32, vp]
    lib.astra_fused_allreduce_add_rmsnorm.restype = i32
    lib.astra_fused_allreduce_add_rmsnorm_ex.argtypes = [ctypes.POINTER(vp), i32, ctypes.POINTER(vp), i32, vp,
                                                         ctypes.POINTER(vp), i32, vp, i64, i64, f32, i32, vp]
    lib.astra_fused_allreduce_add_rmsnorm_ex.restype = i32
    lib.astra_status_string.argtypes = [i32]
    lib.astra_status_string.restype = ctypes.c_char_p
    lib.astra_build_id.argtypes = []
    lib.astra_build_id.restype = ctypes.c_char_p
    _refuse_stale(lib)
    _load_fastcall(lib)
    _lib = lib
    return lib


_fast = None  # the _astra_fastcall extension module, once loaded


def _load_fastcall(lib) -> None:
    """Import the `_astra_fastcall` extension from the package directory and give it the addresses of
    the entry points resolved above.  It re-issues prepared calls without going through ctypes (about
    1 us less host time per launch) and, like the library, it is required: a missing or stale module
    is an error, not a reason to take another route."""
    global _fast
    try:
        from . import _astra_fastcall as fast
    except ImportError as exc:
        raise ImportError(
            f"{FASTCALL_PATH} is missing or cannot be loaded ({exc}): build it with "
            "`python -m paper_2509_07506_b200.build`") from exc
    from . import build as _build
    if os.path.isdir(_build.CSRC) and os.path.isdir(_build.INCLUDE) and fast.build_id() != _build.source_hash():
        raise ImportError(f"{FASTCALL_PATH} was built from other sources: rebuild it with "
                          "`python -m paper_2509_07506_b200.build`")
    for kind, fn in ((fast.KIND_RMSNORM, lib.astra_fused_add_rmsnorm), (fast.KIND_SILU, lib.astra_silu_and_mul),
                     (fast.KIND_MERGE, lib.astra_merge_attn_states_lse),
                     (fast.KIND_ALLREDUCE_RMSNORM, lib.astra_fused_allreduce_add_rmsnorm)):
        fast.bind(kind, ctypes.cast(fn, ctypes.c_void_p).value)
    _fast = fast


def _refuse_stale(lib) -> None:
    """Where the library sits beside its sources (a source checkout), it must have been built from
    exactly those sources: the hash compiled into it is compared with the hash of the files."""
    from . import build as _build
    if not (os.path.isdir(_build.CSRC) and os.path.isdir(_build.INCLUDE)):
        return
    built_from, on_disk = lib.astra_build_id().decode(), _build.source_hash()
    if built_from != on_disk:
        raise ImportError(
            f"{LIB_PATH} was built from other sources (library {built_from[:12]}, sources {on_disk[:12]}): "
            "rebuild it with `python -m paper_2509_07506_b200.build`")


def status_string(status: int) -> str:
    return load_library().astra_status_string(int(status)).decode()


def _same_device(t: torch.Tensor, name: str, device) -> None:
    """Every operand of a call must live on one GPU: the C side receives bare addresses and launches on
    that GPU, so a tensor from another one would be dereferenced as a foreign (or unmapped) address."""
    if device is not None and t.device != device:
        raise ValueError(f"{name} is on {t.device}, but the call's first tensor is on {device}")


def _check(t: torch.Tensor, name: str, dtype=None, shape=None, device=None) -> None:
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    _same_device(t, name, device)
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must have dtype {dtype}, got {t.dtype}")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} must have shape {tuple(shape)}, got {tuple(t.shape)}")


def _code(t: torch.Tensor, name: str) -> int:
    if t.dtype not in _DTYPE_CODE:
        raise TypeError(f"{name} must be bfloat16, float16 or float32, got {t.dtype}")
    return _DTYPE_CODE[t.dtype]


# torch's C accessor for the current stream handle; about 2 us cheaper per call than building a
# torch.cuda.Stream object just to read its handle.
_raw_current_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream(t: torch.Tensor, stream: Optional[torch.cuda.Stream]) -> int:
    if stream is not None:
        return stream.cuda_stream
    if _raw_current_stream is not None:
        return _raw_current_stream(t.device.index)
    return torch.cuda.current_stream(t.device).cuda_stream


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


class PreparedCall:
    """One validated call, kept ready to be issued again.

    The plain functions below check every tensor, read its address and convert the arguments on
    each call; for the small shapes of decode steps that host work takes longer than the kernel.
    A prepared call does all of it once: it keeps the converted arguments in a C struct of the
    ``_astra_fastcall`` extension (and references to the tensors, so their addresses stay valid) and
    ``__call__`` only looks up the current stream and hands the struct to the entry point, without
    ctypes in between.  The C entry point still checks every argument on every launch.  The tensors'
    contents may change between calls; their addresses, shapes and dtypes are fixed at preparation.
    Results are identical to the plain call's, which is itself ``prepare(...)()``.
    ``via_ctypes()`` issues the same call through ctypes (kept to compare the two routes).
    """

    __slots__ = ("name", "_fn", "_make_args", "_device", "_keep", "_ready", "_launch")

    def __init__(self, name: str, fn, make_args, device: torch.device, keep: tuple, ready):
        self.name = name
        self._fn = fn
        self._make_args = make_args  # builds the ctypes argument tuple, only when via_ctypes() asks for it
        self._device = device.index if device.index is not None else torch.cuda.current_device()
        self._keep = keep
        self._ready = ready
        self._launch = _fast.launch

    def __call__(self, stream: Optional[torch.cuda.Stream] = None) -> None:
        dev = self._device
        if stream is not None:
            handle = stream.cuda_stream
        elif _raw_current_stream is not None:
            handle = _raw_current_stream(dev)
        else:
            handle = torch.cuda.current_stream(dev).cuda_stream
        if _raw_current_device() == dev:
            st = self._launch(self._ready, handle)
        else:  # the C side launches on the current device
            with torch.cuda.device(dev):
                st = self._launch(self._ready, handle)
        if st != ASTRA_OK:
            raise AstraError(st, self.name)

    def via_ctypes(self, stream: Optional[torch.cuda.Stream] = None) -> None:
        """The same launch issued through ctypes instead of the extension module."""
        handle = stream.cuda_stream if stream is not None else _stream_of(self._device)
        args = self._make_args()
        with torch.cuda.device(self._device):
            st = self._fn(*args, handle)
        if st != ASTRA_OK:
            raise AstraError(st, self.name)


def _stream_of(dev: int) -> int:
    if _raw_current_stream is not None:
        return _raw_current_stream(dev)
    return torch.cuda.current_stream(dev).cuda_stream


_raw_current_device = getattr(torch._C, "_cuda_getDevice", None) or torch.cuda.current_device


def _ptr(t: Optional[torch.Tensor]):
    return ctypes.c_void_p(t.data_ptr()) if t is not None else None


def prepare_fused_add_rmsnorm(x: torch.Tensor, residual: torch.Tensor, weight: torch.Tensor,
                              eps: float) -> PreparedCall:
    """Validated, re-issuable form of :func:`astra_fused_add_rmsnorm`."""
    _check(x, "x")
    code = _code(x, "x")
    if x.dim() != 2:
        raise ValueError("x must be [T, H]")
    T, H = x.shape
    _check(residual, "residual", x.dtype, (T, H), x.device)
    _check(weight, "weight", x.dtype, (H,), x.device)
    args = lambda: (_ptr(x), _ptr(residual), _ptr(weight), ctypes.c_int64(T), ctypes.c_int64(H),  # noqa: E731
                    ctypes.c_float(float(eps)), ctypes.c_int(code))
    lib = load_library()
    ready = _fast.prepare(_fast.KIND_RMSNORM, (x.data_ptr(), residual.data_ptr(), weight.data_ptr()), (T, H),
                          float(eps), code, ())
    return PreparedCall("astra_fused_add_rmsnorm", lib.astra_fused_add_rmsnorm, args, x.device,
                        (x, residual, weight), ready)


def astra_fused_add_rmsnorm(x: torch.Tensor, residual: torch.Tensor, weight: torch.Tensor,
                            eps: float, stream: Optional[torch.cuda.Stream] = None) -> None:
    """In place: residual <- x + residual, x <- RMSNorm(x + residual) * weight.  x, residual [T, H]."""
    prepare_fused_add_rmsnorm(x, residual, weight, eps)(stream)


def prepare_silu_and_mul(out: torch.Tensor, input: torch.Tensor) -> PreparedCall:
    """Validated, re-issuable form of :func:`astra_silu_and_mul`."""
    _check(input, "input")
    code = _code(input, "input")
    if input.dim() != 2 or input.shape[1] % 2:
        raise ValueError("input must be [T, 2*D]")
    T, D = input.shape[0], input.shape[1] // 2
    _check(out, "out", input.dtype, (T, D), input.device)
    args = lambda: (_ptr(out), _ptr(input), ctypes.c_int64(T), ctypes.c_int64(D), ctypes.c_int(code))  # noqa: E731
    lib = load_library()
    ready = _fast.prepare(_fast.KIND_SILU, (out.data_ptr(), input.data_ptr()), (T, D), 0.0, code, ())
    return PreparedCall("astra_silu_and_mul", lib.astra_silu_and_mul, args, input.device, (out, input), ready)


def astra_silu_and_mul(out: torch.Tensor, input: torch.Tensor,
                       stream: Optional[torch.cuda.Stream] = None) -> None:
    """out[T, D] <- SiLU(input[:, :D]) * input[:, D:]."""
    prepare_silu_and_mul(out, input)(stream)


def prepare_merge_attn_states_lse(v_out: torch.Tensor, lse_out: Optional[torch.Tensor],
                                  v_a: torch.Tensor, lse_a: torch.Tensor,
                                  v_b: torch.Tensor, lse_b: torch.Tensor) -> PreparedCall:
    """Validated, re-issuable form of :func:`astra_merge_attn_states_lse`."""
    _check(v_a, "v_a")
    code = _code(v_a, "v_a")
    if v_a.dim() != 3:
        raise ValueError("v_a must be [T, Hh, D]")
    T, Hh, D = v_a.shape
    _check(v_b, "v_b", v_a.dtype, (T, Hh, D), v_a.device)
    _check(v_out, "v_out", v_a.dtype, (T, Hh, D), v_a.device)
    _check(lse_a, "lse_a", torch.float32, (T, Hh), v_a.device)
    _check(lse_b, "lse_b", torch.float32, (T, Hh), v_a.device)
    if lse_out is not None:
        _check(lse_out, "lse_out", torch.float32, (T, Hh), v_a.device)
    args = lambda: (_ptr(v_out), _ptr(lse_out), _ptr(v_a), _ptr(lse_a), _ptr(v_b), _ptr(lse_b),  # noqa: E731
                    ctypes.c_int64(T), ctypes.c_int64(Hh), ctypes.c_int64(D), ctypes.c_int(code))
    lib = load_library()
    ready = _fast.prepare(_fast.KIND_MERGE,
                          (v_out.data_ptr(), lse_out.data_ptr() if lse_out is not None else None, v_a.data_ptr(),
                           lse_a.data_ptr(), v_b.data_ptr(), lse_b.data_ptr()), (T, Hh, D), 0.0, code, ())
    return PreparedCall("astra_merge_attn_states_lse", lib.astra_merge_attn_states_lse, args,
                        v_a.device, (v_out, lse_out, v_a, lse_a, v_b, lse_b), ready)


def astra_merge_attn_states_lse(v_out: torch.Tensor, lse_out: Optional[torch.Tensor],
                                v_a: torch.Tensor, lse_a: torch.Tensor,
                                v_b: torch.Tensor, lse_b: torch.Tensor,
                                stream: Optional[torch.cuda.Stream] = None) -> None:
    """v_out, lse_out <- merge of (v_a, lse_a) and (v_b, lse_b).  v_* [T, Hh, D]; lse_* [T, Hh] fp32."""
    prepare_merge_attn_states_lse(v_out, lse_out, v_a, lse_a, v_b, lse_b)(stream)


def prepare_fused_allreduce_add_rmsnorm(y: torch.Tensor, residual: torch.Tensor, parts, weight: torch.Tensor,
                                        eps: float) -> PreparedCall:
    """Validated, re-issuable form of :func:`astra_fused_allreduce_add_rmsnorm`."""
    parts = list(parts)
    _check(y, "y")
    code = _code(y, "y")
    if y.dim() != 2:
        raise ValueError("y must be [T, H]")
    T, H = y.shape
    _check(residual, "residual", y.dtype, (T, H), y.device)
    _check(weight, "weight", y.dtype, (H,), y.device)
    if not 1 <= len(parts) <= 16:
        raise ValueError(f"between 1 and 16 partial hidden states are supported, got {len(parts)}")
    for i, p in enumerate(parts):
        # a partial may sit on another GPU (that is the point of the call): no device check here
        _check(p, f"parts[{i}]", y.dtype, (T, H))
    args = lambda: (_ptr(y), _ptr(residual), (ctypes.c_void_p * len(parts))(*[p.data_ptr() for p in parts]),  # noqa: E731
                    ctypes.c_int(len(parts)), _ptr(weight), ctypes.c_int64(T), ctypes.c_int64(H),
                    ctypes.c_float(float(eps)), ctypes.c_int(code))
    lib = load_library()
    ready = _fast.prepare(_fast.KIND_ALLREDUCE_RMSNORM, (y.data_ptr(), residual.data_ptr(), weight.data_ptr()),
                          (T, H), float(eps), code, tuple(p.data_ptr() for p in parts))
    return PreparedCall("astra_fused_allreduce_add_rmsnorm", lib.astra_fused_allreduce_add_rmsnorm,
                        args, y.device, (y, residual, weight, *parts), ready)


def astra_fused_allreduce_add_rmsnorm(y: torch.Tensor, residual: torch.Tensor, parts, weight: torch.Tensor,
                                      eps: float, stream: Optional[torch.cuda.Stream] = None) -> None:
    """y <- RMSNorm(sum(parts) + residual) * weight, residual <- sum(parts) + residual (in place).
    ``parts`` is the sequence of per-rank partial hidden states [T, H], in rank order; they are added
    in that order in binary32 and the residual last.  The partials may live on other GPUs whose
    memory this process can address; y, residual and weight live on the GPU that runs the kernel.
    The call waits for nothing: order it after the partials have been written."""
    prepare_fused_allreduce_add_rmsnorm(y, residual, parts, weight, eps)(stream)


def astra_fused_allreduce_add_rmsnorm_ex(y_outs, residual_outs, residual: torch.Tensor, parts, weight: torch.Tensor,
                                         eps: float, stream: Optional[torch.cuda.Stream] = None) -> None:
    """Two-shot form: this rank's block of rows [T, H] is reduced over ``parts`` (rank order, binary32,
    the residual last) and normalised once, and the results are stored to every tensor of ``y_outs``
    (the normalised rows) and of ``residual_outs`` (the new residual; one of them may be ``residual``
    itself).  All tensors are the [T, H] row block, i.e. slices ``buf[first:first + T]`` of the ranks'
    full buffers.  ``residual`` and ``weight`` live on the GPU that runs the kernel; partials and
    destinations may live on other GPUs whose memory this process can address.  The call waits for
    nothing and the destinations' owners must not read them before it has completed."""
    parts, y_outs, residual_outs = list(parts), list(y_outs), list(residual_outs)
    _check(residual, "residual")
    code = _code(residual, "residual")
    if residual.dim() != 2:
        raise ValueError("residual must be [T, H]")
    T, H = residual.shape
    _check(weight, "weight", residual.dtype, (H,), residual.device)
    for what, seq in (("parts", parts), ("y_outs", y_outs), ("residual_outs", residual_outs)):
        if not 1 <= len(seq) <= 16:
            raise ValueError(f"between 1 and 16 tensors are supported in {what}, got {len(seq)}")
        for i, t in enumerate(seq):
            # partials and destinations may sit on other GPUs (that is the point of the call): no device check
            _check(t, f"{what}[{i}]", residual.dtype, (T, H))
    table = lambda seq: (ctypes.c_void_p * len(seq))(*[t.data_ptr() for t in seq])  # noqa: E731
    with _on_device(residual):
        st = load_library().astra_fused_allreduce_add_rmsnorm_ex(
            table(y_outs), len(y_outs), table(residual_outs), len(residual_outs), residual.data_ptr(),
            table(parts), len(parts), weight.data_ptr(), T, H, float(eps), code, _stream(residual, stream))
    if st != ASTRA_OK:
        raise AstraError(st, "astra_fused_allreduce_add_rmsnorm_ex")


# ---- strided / out-of-place forms ---------------------------------------------------------------

def _check_rows(t: torch.Tensor, name: str, dtype, shape, device=None) -> None:
    """A tensor whose innermost dimension is contiguous; outer strides are free (non-negative)."""
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    _same_device(t, name, device)
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must have dtype {dtype}, got {t.dtype}")
    if tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} must have shape {tuple(shape)}, got {tuple(t.shape)}")
    if t.shape[-1] > 1 and t.stride(-1) != 1:
        raise ValueError(f"{name}: the innermost dimension must be contiguous")
    if any(st < 0 for st in t.stride()):
        raise ValueError(f"{name}: negative strides are not supported")


def _pitch(t: torch.Tensor) -> int:
    """Row pitch of a 2-D tensor (a single row may report any stride; use its width)."""
    return t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1])


def astra_fused_add_rmsnorm_ex(y: torch.Tensor, residual_out: torch.Tensor, x: torch.Tensor,
                               residual: torch.Tensor, weight: torch.Tensor, eps: float,
                               stream: Optional[torch.cuda.Stream] = None) -> None:
    """y <- RMSNorm(x + residual) * weight, residual_out <- x + residual; [T, H] tensors whose rows
    may be pitched (slices of wider buffers).  y may be x and residual_out may be residual."""
    if x.dim() != 2:
        raise ValueError("x must be [T, H]")
    code = _code(x, "x")
    T, H = x.shape
    for t, n in ((x, "x"), (residual, "residual"), (y, "y"), (residual_out, "residual_out")):
        _check_rows(t, n, x.dtype, (T, H), x.device)
    _check(weight, "weight", x.dtype, (H,), x.device)
    with _on_device(x):
        st = load_library().astra_fused_add_rmsnorm_ex(
            y.data_ptr(), residual_out.data_ptr(), x.data_ptr(), residual.data_ptr(), weight.data_ptr(),
            T, H, _pitch(y), _pitch(residual_out), _pitch(x), _pitch(residual), float(eps), code,
            _stream(x, stream))
    if st != ASTRA_OK:
        raise AstraError(st, "astra_fused_add_rmsnorm_ex")


def astra_silu_and_mul_ex(out: torch.Tensor, gate: torch.Tensor, up: torch.Tensor,
                          stream: Optional[torch.cuda.Stream] = None) -> None:
    """out[T, D] <- SiLU(gate) * up with separately addressed (possibly pitched) operands."""
    if gate.dim() != 2:
        raise ValueError("gate must be [T, D]")
    code = _code(gate, "gate")
    T, D = gate.shape
    for t, n in ((gate, "gate"), (up, "up"), (out, "out")):
        _check_rows(t, n, gate.dtype, (T, D), gate.device)
    with _on_device(gate):
        st = load_library().astra_silu_and_mul_ex(out.data_ptr(), gate.data_ptr(), up.data_ptr(), T, D,
                                                  _pitch(out), _pitch(gate), _pitch(up), code,
                                                  _stream(gate, stream))
    if st != ASTRA_OK:
        raise AstraError(st, "astra_silu_and_mul_ex")


def astra_merge_attn_states_lse_ex(v_out: torch.Tensor, lse_out: Optional[torch.Tensor],
                                   v_a: torch.Tensor, lse_a: torch.Tensor,
                                   v_b: torch.Tensor, lse_b: torch.Tensor,
                                   stream: Optional[torch.cuda.Stream] = None) -> None:
    """Merge for strided tensors: values [T, Hh, D] with D contiguous, scores [T, Hh] with any
    non-negative strides (e.g. the transposed view of a head-major [Hh, T] tensor)."""
    if v_a.dim() != 3:
        raise ValueError("v_a must be [T, Hh, D]")
    code = _code(v_a, "v_a")
    T, Hh, D = v_a.shape
    for t, n in ((v_a, "v_a"), (v_b, "v_b"), (v_out, "v_out")):
        _check_rows(t, n, v_a.dtype, (T, Hh, D), v_a.device)
    scores = [(lse_a, "lse_a"), (lse_b, "lse_b")] + ([(lse_out, "lse_out")] if lse_out is not None else [])
    for t, n in scores:
        if not isinstance(t, torch.Tensor) or not t.is_cuda or t.dtype != torch.float32:
            raise TypeError(f"{n} must be a float32 CUDA tensor")
        _same_device(t, n, v_a.device)
        if tuple(t.shape) != (T, Hh) or any(s < 0 for s in t.stride()):
            raise ValueError(f"{n} must have shape {(T, Hh)} and non-negative strides")
    so = (lse_out.stride(0), lse_out.stride(1)) if lse_out is not None else (0, 0)
    strides = (ctypes.c_int64 * 12)(v_a.stride(0), v_a.stride(1), v_b.stride(0), v_b.stride(1),
                                    v_out.stride(0), v_out.stride(1), lse_a.stride(0), lse_a.stride(1),
                                    lse_b.stride(0), lse_b.stride(1), so[0], so[1])
    with _on_device(v_a):
        st = load_library().astra_merge_attn_states_lse_ex(
            v_out.data_ptr(), lse_out.data_ptr() if lse_out is not None else None,
            v_a.data_ptr(), lse_a.data_ptr(), v_b.data_ptr(), lse_b.data_ptr(), T, Hh, D, strides, code,
            _stream(v_a, stream))
    if st != ASTRA_OK:
        raise AstraError(st, "astra_merge_attn_states_lse_ex")
