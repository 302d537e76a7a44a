"""CPU-only checks of the C ABI: the shared library builds and loads, exports every function that
include/astra.h declares, and rejects bad arguments with the documented status before anything
could be launched (none of these calls reaches a kernel launch)."""
import ctypes
import os
import re

import pytest

from paper_2509_07506_b200 import binding
from paper_2509_07506_b200 import build as astra_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    astra_build.build()
    return binding.load_library()


def declared_functions(header):
    text = open(os.path.join(ROOT, "include", header)).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return set(re.findall(r"\b(astra_[a-z0-9_]+)\s*\(", text))


def test_every_declared_function_is_exported(lib):
    assert sorted(f for f in os.listdir(os.path.join(ROOT, "include")) if f.endswith(".h")) == \
        ["astra.h", "astra_ablation.h"]
    names = declared_functions("astra.h")
    assert {"astra_fused_add_rmsnorm", "astra_silu_and_mul", "astra_merge_attn_states_lse",
            "astra_status_string"} <= names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in astra.h but not exported by libastra.so"
    assert set(binding.EXPORTED_SYMBOLS) == names


def test_ablation_library_exports_and_argument_errors():
    from paper_2509_07506_b200 import ablation
    astra_build.build_ablation()
    alib = ablation.load_library()
    names = declared_functions("astra_ablation.h")
    assert set(ablation.EXPORTED_SYMBOLS) == names
    for n in names:
        assert hasattr(alib, n), f"{n} is declared in astra_ablation.h but not exported"
    f = alib.astra_ablation_fused_add_rmsnorm
    assert f(0, None, A, A, 1, 8, 1e-6, 0, None) == binding.ASTRA_ERR_NULL_POINTER
    assert f(2, A, 2 * A, 3 * A, 1, 8, 1e-6, 0, None) == binding.ASTRA_ERR_BAD_SHAPE      # unknown design
    assert f(1, A, 2 * A, 3 * A, 1, 7, 1e-6, 0, None) == binding.ASTRA_ERR_BAD_SHAPE      # odd width, 32-bit design
    assert f(1, A + 2, 2 * A, 3 * A, 1, 8, 1e-6, 0, None) == binding.ASTRA_ERR_MISALIGNED
    assert f(0, A, 2 * A, 3 * A, 0, 8, 1e-6, 0, None) == binding.ASTRA_OK
    g = alib.astra_ablation_silu_and_mul
    assert g(0, A, None, 1, 8, 0, None) == binding.ASTRA_ERR_NULL_POINTER
    assert g(1, A, 2 * A, 1, 9, 0, None) == binding.ASTRA_ERR_BAD_SHAPE
    assert g(0, A, 2 * A, 1, 8, 4, None) == binding.ASTRA_ERR_BAD_DTYPE
    assert g(1, A, 2 * A, 0, 8, 0, None) == binding.ASTRA_OK
    h = alib.astra_ablation_merge_attn_states_lse
    assert h(0, A, None, A, A, A, A, 1, 1, 8, 0, None) == binding.ASTRA_ERR_NULL_POINTER
    assert h(1, A, A, A, A, A, A, 1, 1, 9, 0, None) == binding.ASTRA_ERR_BAD_SHAPE
    assert h(0, A, A, A, A, A, A, 0, 1, 8, 0, None) == binding.ASTRA_OK


def test_status_strings(lib):
    seen = set()
    for code in range(0, 7):
        s = lib.astra_status_string(code).decode()
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 7
    assert lib.astra_status_string(99).decode() == "unknown status"


A = 0x10000  # fake, 64 KiB-aligned "device" addresses: never dereferenced on these paths


def test_rmsnorm_argument_errors(lib):
    f = lib.astra_fused_add_rmsnorm
    assert f(None, A, A, 1, 8, 1e-6, 0, None) == binding.ASTRA_ERR_NULL_POINTER
    assert f(A, None, A, 1, 8, 1e-6, 0, None) == binding.ASTRA_ERR_NULL_POINTER
    assert f(A, A, None, 1, 8, 1e-6, 0, None) == binding.ASTRA_ERR_NULL_POINTER
    assert f(A, 2 * A, 3 * A, 1, 8, 1e-6, 7, None) == binding.ASTRA_ERR_BAD_DTYPE
    assert f(A, 2 * A, 3 * A, -1, 8, 1e-6, 0, None) == binding.ASTRA_ERR_BAD_SHAPE
    assert f(A, 2 * A, 3 * A, 1, 0, 1e-6, 0, None) == binding.ASTRA_ERR_BAD_SHAPE
    assert f(A, 2 * A, 3 * A, 1, 2 ** 31, 1e-6, 0, None) == binding.ASTRA_ERR_BAD_SHAPE
    assert f(A, 2 * A, 3 * A, 2 ** 40, 2 ** 30, 1e-6, 0, None) == binding.ASTRA_ERR_BAD_SHAPE
    assert f(A + 1, 2 * A, 3 * A, 1, 8, 1e-6, 0, None) == binding.ASTRA_ERR_MISALIGNED
    assert f(A, 2 * A, 3 * A + 1, 1, 8, 1e-6, 0, None) == binding.ASTRA_ERR_MISALIGNED
    assert f(A, A + 8, 3 * A, 1, 8, 1e-6, 0, None) == binding.ASTRA_ERR_OVERLAP
    assert f(A, 2 * A, A + 4, 1, 8, 1e-6, 0, None) == binding.ASTRA_ERR_OVERLAP
    assert f(A, 2 * A, 3 * A, 0, 8, 1e-6, 0, None) == binding.ASTRA_OK
    # a row is indexed in 16-bit units with 32-bit integers: at most 2^30 units per row
    assert f(A, 2 * A, 3 * A, 1, 2 ** 30 + 1, 1e-6, 0, None) == binding.ASTRA_ERR_BAD_SHAPE
    assert f(A, 2 * A, 3 * A, 1, 2 ** 29 + 1, 1e-6, binding.ASTRA_FP32, None) == binding.ASTRA_ERR_BAD_SHAPE
    assert f(A, 2 * A, 3 * A, 0, 2 ** 30, 1e-6, 0, None) == binding.ASTRA_OK
    assert f(A, 2 * A, 3 * A, 0, 2 ** 29, 1e-6, binding.ASTRA_FP32, None) == binding.ASTRA_OK


def test_empty_batches_do_not_examine_their_pointers(lib):
    """T == 0: an empty tensor may have a NULL address (torch reports 0 for it), the call is ASTRA_OK;
    shape and dtype errors are still reported."""
    assert lib.astra_fused_add_rmsnorm(None, None, None, 0, 8, 1e-6, 0, None) == binding.ASTRA_OK
    assert lib.astra_fused_add_rmsnorm_ex(None, None, None, None, None, 0, 8, 8, 8, 8, 8, 1e-6, 1, None) == binding.ASTRA_OK
    assert lib.astra_silu_and_mul(None, None, 0, 8, 0, None) == binding.ASTRA_OK
    assert lib.astra_silu_and_mul_ex(None, None, None, 0, 8, 8, 8, 8, 2, None) == binding.ASTRA_OK
    assert lib.astra_merge_attn_states_lse(None, None, None, None, None, None, 0, 2, 8, 0, None) == binding.ASTRA_OK
    assert lib.astra_merge_attn_states_lse_ex(None, None, None, None, None, None, 0, 2, 8, None, 0, None) == binding.ASTRA_OK
    assert lib.astra_fused_add_rmsnorm(None, None, None, 0, 0, 1e-6, 0, None) == binding.ASTRA_ERR_BAD_SHAPE
    assert lib.astra_silu_and_mul(None, None, 0, 8, 9, None) == binding.ASTRA_ERR_BAD_DTYPE
    assert lib.astra_merge_attn_states_lse(None, None, None, None, None, None, 0, 0, 8, 0, None) == binding.ASTRA_ERR_BAD_SHAPE


def test_refused_launch_is_reported_and_stops_the_call(lib):
    """Where no CUDA device exists the runtime refuses every launch on the host: a well-formed call
    must come back as ASTRA_ERR_CUDA (the launch's own status), again on the next call (nothing is
    left pending in between), and argument errors keep their own codes.  Skipped where a device
    exists: the fake addresses below must never reach a GPU."""
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present; the fake addresses of this test must not be launched on")
    for _ in range(2):
        assert lib.astra_fused_add_rmsnorm(A, 2 * A, 3 * A, 4, 4096, 1e-6, 0, None) == binding.ASTRA_ERR_CUDA
        assert lib.astra_fused_add_rmsnorm(A, 16 * A, 32 * A, 2, 40000, 1e-6, 0, None) == binding.ASTRA_ERR_CUDA  # cluster launch
        assert lib.astra_silu_and_mul(A, 16 * A, 4, 1024, 1, None) == binding.ASTRA_ERR_CUDA
        assert lib.astra_merge_attn_states_lse(A, 2 * A, 3 * A, 4 * A, 5 * A, 6 * A, 4, 2, 128, 0, None) == binding.ASTRA_ERR_CUDA
        assert lib.astra_silu_and_mul(A, None, 4, 1024, 1, None) == binding.ASTRA_ERR_NULL_POINTER
    assert "launch" in lib.astra_status_string(binding.ASTRA_ERR_CUDA).decode()


def test_allreduce_rmsnorm_argument_errors(lib):
    import ctypes as C
    f = lib.astra_fused_allreduce_add_rmsnorm
    Y, R, W = A, 2 * A, 3 * A

    def call(parts=(4 * A, 5 * A), n=None, y=Y, r=R, w=W, T=1, H=8, dtype=0):
        table = (C.c_void_p * max(1, len(parts)))(*parts) if parts is not None else None
        return f(y, r, table, len(parts) if n is None else n, w, T, H, 1e-6, dtype, None)

    assert call(y=None) == binding.ASTRA_ERR_NULL_POINTER
    assert call(r=None) == binding.ASTRA_ERR_NULL_POINTER
    assert call(w=None) == binding.ASTRA_ERR_NULL_POINTER
    assert call(parts=None, n=2) == binding.ASTRA_ERR_NULL_POINTER
    assert call(parts=(4 * A, None)) == binding.ASTRA_ERR_NULL_POINTER
    assert call(dtype=4) == binding.ASTRA_ERR_BAD_DTYPE
    assert call(n=0) == binding.ASTRA_ERR_BAD_SHAPE
    assert call(parts=tuple((4 + i) * A for i in range(17))) == binding.ASTRA_ERR_BAD_SHAPE
    assert call(T=-1) == binding.ASTRA_ERR_BAD_SHAPE
    assert call(H=0) == binding.ASTRA_ERR_BAD_SHAPE
    assert call(H=2 ** 30 + 1) == binding.ASTRA_ERR_BAD_SHAPE
    assert call(H=2 ** 29 + 1, dtype=binding.ASTRA_FP32) == binding.ASTRA_ERR_BAD_SHAPE
    assert call(T=2 ** 40, H=2 ** 30) == binding.ASTRA_ERR_BAD_SHAPE
    assert call(y=Y + 1) == binding.ASTRA_ERR_MISALIGNED
    assert call(parts=(4 * A, 5 * A + 1)) == binding.ASTRA_ERR_MISALIGNED
    assert call(parts=(4 * A + 2, 5 * A), dtype=binding.ASTRA_FP32) == binding.ASTRA_ERR_MISALIGNED
    assert call(y=R) == binding.ASTRA_ERR_OVERLAP                 # y over the residual
    assert call(parts=(4 * A, Y + 8)) == binding.ASTRA_ERR_OVERLAP    # y over a partial
    assert call(parts=(R, 5 * A)) == binding.ASTRA_ERR_OVERLAP        # the residual is also a partial
    assert call(w=Y + 4) == binding.ASTRA_ERR_OVERLAP
    assert call(T=0) == binding.ASTRA_OK
    assert call(T=0, parts=None, n=3, y=None, r=None, w=None) == binding.ASTRA_OK
    import torch
    if not torch.cuda.is_available():   # well-formed calls reach the launch, which a machine without a GPU refuses
        assert call(parts=(4 * A, 4 * A)) == binding.ASTRA_ERR_CUDA       # partials may overlap one another
        assert call(parts=tuple((4 + i) * A for i in range(16)), T=2, H=4100) == binding.ASTRA_ERR_CUDA
        assert call(parts=(16 * A,), T=1, H=40000, y=32 * A, r=48 * A, w=64 * A) == binding.ASTRA_ERR_CUDA


def test_allreduce_rmsnorm_ex_argument_errors(lib):
    """The two-shot form: several destinations per result.  Every destination is checked for NULL,
    alignment and overlap with every other operand; one residual destination may be the residual."""
    import ctypes as C
    f = lib.astra_fused_allreduce_add_rmsnorm_ex
    R, W = 2 * A, 3 * A

    def tab(ptrs):
        return (C.c_void_p * max(1, len(ptrs)))(*ptrs) if ptrs is not None else None

    def call(ys=(8 * A, 9 * A), rs=(R, 10 * A), r=R, parts=(4 * A, 5 * A), w=W, T=1, H=8, dtype=0, n_y=None, n_r=None):
        return f(tab(ys), len(ys) if n_y is None else n_y, tab(rs), len(rs) if n_r is None else n_r, r,
                 tab(parts), len(parts), w, T, H, 1e-6, dtype, None)

    assert call(ys=None, n_y=1) == binding.ASTRA_ERR_NULL_POINTER
    assert call(rs=None, n_r=1) == binding.ASTRA_ERR_NULL_POINTER
    assert call(r=None) == binding.ASTRA_ERR_NULL_POINTER
    assert call(ys=(8 * A, None)) == binding.ASTRA_ERR_NULL_POINTER
    assert call(rs=(R, None)) == binding.ASTRA_ERR_NULL_POINTER
    assert call(n_y=0) == binding.ASTRA_ERR_BAD_SHAPE
    assert call(n_r=0) == binding.ASTRA_ERR_BAD_SHAPE
    assert call(ys=tuple((20 + i) * A for i in range(17))) == binding.ASTRA_ERR_BAD_SHAPE
    assert call(rs=tuple((20 + i) * A for i in range(17))) == binding.ASTRA_ERR_BAD_SHAPE
    assert call(dtype=5) == binding.ASTRA_ERR_BAD_DTYPE
    assert call(ys=(8 * A, 9 * A + 1)) == binding.ASTRA_ERR_MISALIGNED
    assert call(rs=(R, 10 * A + 2), dtype=binding.ASTRA_FP32) == binding.ASTRA_ERR_MISALIGNED
    assert call(ys=(8 * A, 8 * A)) == binding.ASTRA_ERR_OVERLAP          # two destinations, one address
    assert call(ys=(8 * A, 10 * A)) == binding.ASTRA_ERR_OVERLAP         # a y destination over a residual destination
    assert call(ys=(8 * A, R)) == binding.ASTRA_ERR_OVERLAP              # y over the residual input
    assert call(rs=(R + 8, 10 * A)) == binding.ASTRA_ERR_OVERLAP         # a residual destination shifted into the residual
    assert call(rs=(R, 5 * A)) == binding.ASTRA_ERR_OVERLAP              # a residual destination over a partial
    assert call(ys=(8 * A, W + 4)) == binding.ASTRA_ERR_OVERLAP          # over the weight
    assert call(T=0) == binding.ASTRA_OK
    assert call(T=0, ys=None, rs=None, r=None, n_y=2, n_r=2) == binding.ASTRA_OK
    import torch
    if not torch.cuda.is_available():
        assert call() == binding.ASTRA_ERR_CUDA                          # in place plus one more destination
        assert call(rs=(10 * A, 11 * A)) == binding.ASTRA_ERR_CUDA        # no destination is the residual itself
        assert call(ys=tuple((20 + i) * A for i in range(16)), rs=tuple((40 + i) * A for i in range(16)), T=3, H=4100) \
            == binding.ASTRA_ERR_CUDA


def test_silu_argument_errors(lib):
    f = lib.astra_silu_and_mul
    assert f(None, A, 1, 8, 0, None) == binding.ASTRA_ERR_NULL_POINTER
    assert f(A, None, 1, 8, 0, None) == binding.ASTRA_ERR_NULL_POINTER
    assert f(A, 2 * A, 1, 8, 9, None) == binding.ASTRA_ERR_BAD_DTYPE
    assert f(A, 2 * A, -5, 8, 0, None) == binding.ASTRA_ERR_BAD_SHAPE
    assert f(A, 2 * A, 1, 0, 0, None) == binding.ASTRA_ERR_BAD_SHAPE
    assert f(A, 2 * A, 1, 2 ** 30, 0, None) == binding.ASTRA_ERR_BAD_SHAPE
    assert f(A + 1, 2 * A, 1, 8, 0, None) == binding.ASTRA_ERR_MISALIGNED
    assert f(A + 16, A, 1, 8, 0, None) == binding.ASTRA_ERR_OVERLAP   # out inside the up half
    assert f(A, A, 1, 8, 0, None) == binding.ASTRA_ERR_OVERLAP
    assert f(A, 2 * A, 0, 8, 0, None) == binding.ASTRA_OK


def test_merge_argument_errors(lib):
    f = lib.astra_merge_attn_states_lse
    ok = dict(v_out=A, lse_out=2 * A, v_a=3 * A, lse_a=4 * A, v_b=5 * A, lse_b=6 * A)

    def call(T=1, Hh=2, D=8, dtype=0, **kw):
        a = dict(ok); a.update(kw)
        return f(a["v_out"], a["lse_out"], a["v_a"], a["lse_a"], a["v_b"], a["lse_b"], T, Hh, D, dtype, None)

    for name in ("v_out", "v_a", "lse_a", "v_b", "lse_b"):
        assert call(**{name: None}) == binding.ASTRA_ERR_NULL_POINTER
    assert call(dtype=5) == binding.ASTRA_ERR_BAD_DTYPE
    assert call(T=-1) == binding.ASTRA_ERR_BAD_SHAPE
    assert call(Hh=0) == binding.ASTRA_ERR_BAD_SHAPE
    assert call(D=0) == binding.ASTRA_ERR_BAD_SHAPE
    assert call(T=2 ** 40, Hh=2 ** 20, D=2 ** 10) == binding.ASTRA_ERR_BAD_SHAPE
    assert call(v_a=3 * A + 1) == binding.ASTRA_ERR_MISALIGNED
    assert call(lse_a=4 * A + 2) == binding.ASTRA_ERR_MISALIGNED
    assert call(lse_out=2 * A + 2) == binding.ASTRA_ERR_MISALIGNED
    assert call(v_out=3 * A + 16) == binding.ASTRA_ERR_OVERLAP      # partial overlap with v_a
    assert call(lse_out=4 * A) == binding.ASTRA_ERR_OVERLAP         # score output over a score input
    assert call(lse_out=6 * A + 4) == binding.ASTRA_ERR_OVERLAP
    assert call(T=0) == binding.ASTRA_OK
    assert call(T=0, lse_out=None) == binding.ASTRA_OK


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "libastra.so"))
    with pytest.raises(ImportError):
        binding.load_library()


def test_rmsnorm_ex_argument_errors(lib):
    f = lib.astra_fused_add_rmsnorm_ex
    ok = dict(y=A, ro=2 * A, x=3 * A, r=4 * A, w=5 * A)

    def call(T=2, H=8, py=8, pro=8, px=8, pr=8, dtype=0, **kw):
        a = dict(ok); a.update(kw)
        return f(a["y"], a["ro"], a["x"], a["r"], a["w"], T, H, py, pro, px, pr, 1e-6, dtype, None)

    for name in ok:
        assert call(**{name: None}) == binding.ASTRA_ERR_NULL_POINTER
    assert call(dtype=9) == binding.ASTRA_ERR_BAD_DTYPE
    assert call(px=7) == binding.ASTRA_ERR_BAD_SHAPE          # rows would overlap
    assert call(py=4) == binding.ASTRA_ERR_BAD_SHAPE
    assert call(T=-1) == binding.ASTRA_ERR_BAD_SHAPE
    assert call(x=3 * A + 1) == binding.ASTRA_ERR_MISALIGNED
    assert call(y=3 * A + 8) == binding.ASTRA_ERR_OVERLAP      # y partially over x
    assert call(y=3 * A, py=16) == binding.ASTRA_ERR_OVERLAP   # same address, different pitch
    assert call(ro=3 * A) == binding.ASTRA_ERR_OVERLAP         # residual_out over x
    assert call(y=4 * A) == binding.ASTRA_ERR_OVERLAP          # y over residual
    assert call(T=0) == binding.ASTRA_OK
    assert call(T=0, y=3 * A, ro=4 * A) == binding.ASTRA_OK


def test_silu_ex_argument_errors(lib):
    f = lib.astra_silu_and_mul_ex
    assert f(None, A, 2 * A, 1, 8, 8, 8, 8, 0, None) == binding.ASTRA_ERR_NULL_POINTER
    assert f(A, None, 2 * A, 1, 8, 8, 8, 8, 0, None) == binding.ASTRA_ERR_NULL_POINTER
    assert f(A, 2 * A, None, 1, 8, 8, 8, 8, 0, None) == binding.ASTRA_ERR_NULL_POINTER
    assert f(A, 2 * A, 3 * A, 2, 8, 7, 8, 8, 0, None) == binding.ASTRA_ERR_BAD_SHAPE
    assert f(A, 2 * A, 3 * A, 2, 8, 8, 8, 4, 0, None) == binding.ASTRA_ERR_BAD_SHAPE
    assert f(A, 2 * A, 3 * A + 1, 2, 8, 8, 8, 8, 0, None) == binding.ASTRA_ERR_MISALIGNED
    assert f(A, 2 * A, A + 8, 2, 8, 8, 8, 8, 0, None) == binding.ASTRA_ERR_OVERLAP
    assert f(A, 2 * A, 3 * A, 0, 8, 8, 8, 8, 0, None) == binding.ASTRA_OK


def test_merge_ex_argument_errors(lib):
    import ctypes as C
    f = lib.astra_merge_attn_states_lse_ex
    T, Hh, D = 4, 2, 8
    dense = [Hh * D, D] * 3 + [Hh, 1] * 3

    def call(strides=dense, v_out=A, lse_out=2 * A, v_a=3 * A, lse_a=4 * A, v_b=5 * A, lse_b=6 * A, T=T, Hh=Hh,
             D=D, dtype=0):
        arr = (C.c_int64 * 12)(*strides) if strides is not None else None
        return f(v_out, lse_out, v_a, lse_a, v_b, lse_b, T, Hh, D, arr, dtype, None)

    assert call(strides=None) == binding.ASTRA_ERR_NULL_POINTER
    assert call(v_b=None) == binding.ASTRA_ERR_NULL_POINTER
    assert call(dtype=3) == binding.ASTRA_ERR_BAD_DTYPE
    assert call(T=2 ** 31, Hh=2) == binding.ASTRA_ERR_BAD_SHAPE
    assert call(T=2 ** 62, Hh=4) == binding.ASTRA_ERR_BAD_SHAPE   # T * Hh would wrap a 64-bit product
    assert call(T=2 ** 33, Hh=2 ** 31 - 1) == binding.ASTRA_ERR_BAD_SHAPE
    neg = list(dense); neg[0] = -16
    assert call(strides=neg) == binding.ASTRA_ERR_BAD_SHAPE
    squeezed = list(dense); squeezed[5] = 4           # v_out head stride < D: rows overlap
    assert call(strides=squeezed) == binding.ASTRA_ERR_BAD_SHAPE
    bcast = list(dense); bcast[10] = 0                 # lse_out token stride 0: rows overlap
    assert call(strides=bcast) == binding.ASTRA_ERR_BAD_SHAPE
    assert call(lse_a=4 * A + 2) == binding.ASTRA_ERR_MISALIGNED
    assert call(v_out=3 * A + 16) == binding.ASTRA_ERR_OVERLAP
    other = list(dense); other[4] = 2 * Hh * D          # same address as v_a but other strides
    assert call(v_out=3 * A, strides=other) == binding.ASTRA_ERR_OVERLAP
    assert call(lse_out=4 * A) == binding.ASTRA_ERR_OVERLAP
    assert call(T=0) == binding.ASTRA_OK
    head_major = list(dense); head_major[6:12] = [1, T] * 3
    assert call(T=0, strides=head_major) == binding.ASTRA_OK


def test_interleaved_slices_of_one_buffer_are_not_overlap(lib):
    """x and residual as column slices of one wide buffer: their address spans interleave, but no
    element is shared; T = 0 cannot show it, so the check is exercised through its error codes."""
    f = lib.astra_fused_add_rmsnorm_ex
    H, pitch = 8, 32
    x, r, w = A, A + 2 * 16, 5 * A               # columns [0, 8) and [16, 24) of a 32-wide buffer
    # a non-overlapping call would go on to launch, so only the rejecting direction is tested here:
    # shifting r so that it shares columns 4..11 with x must be refused, in place or not
    assert f(x, A + 2 * 4, x, A + 2 * 4, w, 4, H, pitch, pitch, pitch, pitch, 1e-6, 0, None) == binding.ASTRA_ERR_OVERLAP
    # r one row down and 4 columns left of x's end: row j of r overlaps row j+1 of x
    assert f(x, A + 2 * (pitch - 4), x, A + 2 * (pitch - 4), w, 4, H, pitch, pitch, pitch, pitch, 1e-6, 0, None) \
        == binding.ASTRA_ERR_OVERLAP
    assert r  # the accepting direction is covered by the GPU tests (slices of one buffer)


def test_overlap_check_against_brute_force(lib):
    """The pitched overlap test that guards the out-of-place / sliced calls, against element sets
    enumerated by brute force: with equal pitches it must be exact (slices of one buffer interleave
    without sharing an element), with different pitches it may only err towards reporting overlap.
    Runs where no GPU exists: a call that passes the check goes on to the launch, which such a
    machine refuses (ASTRA_ERR_CUDA), so nothing is ever launched on these fake addresses."""
    import random
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present; the fake addresses of this test must not be launched on")
    f = lib.astra_fused_add_rmsnorm_ex
    rng = random.Random(7)
    base, far = 64 * A, 4096 * A
    checked = {"overlap": 0, "clear": 0}
    for _ in range(4000):
        T, H = rng.randint(1, 5), rng.randint(1, 6)
        px, py = rng.randint(H, 12), rng.randint(H, 12)
        if rng.random() < 0.6:
            py = px
        dy = rng.randint(-40, 40)                      # y starts dy elements after x
        x, y = base, base + 2 * dy
        ex = {2 * (t * px + j) for t in range(T) for j in range(H)}
        ey = {2 * (dy + t * py + j) for t in range(T) for j in range(H)}
        same = (dy == 0 and px == py)
        truly = bool(ex & ey) and not same
        st = f(y, far, x, 2 * far, 3 * far, T, H, py, H, px, H, 1e-6, 0, None)
        assert st in (binding.ASTRA_ERR_OVERLAP, binding.ASTRA_ERR_CUDA)
        reported = st == binding.ASTRA_ERR_OVERLAP
        if px == py or T == 1:
            assert reported == truly, (T, H, px, py, dy)
        else:
            assert reported or not truly, (T, H, px, py, dy)   # never a missed overlap
        checked["overlap" if truly else "clear"] += 1
    assert checked["overlap"] > 300 and checked["clear"] > 300


def test_strided_output_rows_never_share_elements(lib):
    """The strided merge writes one row of D elements per (token, head); a stride pair under which
    two of those rows share an element must be refused (ASTRA_ERR_BAD_SHAPE), checked against brute
    force.  The test may refuse some exotic disjoint layouts, never accept an overlapping one.
    Runs only where no GPU exists (accepted calls end at the refused launch)."""
    import ctypes as C
    import random
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present; the fake addresses of this test must not be launched on")
    f = lib.astra_merge_attn_states_lse_ex
    rng = random.Random(11)
    far = 4096 * A
    accepted = refused_disjoint = refused_overlapping = 0
    for _ in range(4000):
        T, Hh, D = rng.randint(1, 4), rng.randint(1, 4), rng.randint(1, 5)
        st, sh = rng.randint(0, 24), rng.randint(0, 24)
        rows = [set(range(t * st + h * sh, t * st + h * sh + D)) for t in range(T) for h in range(Hh)]
        overlapping = any(rows[i] & rows[j] for i in range(len(rows)) for j in range(i))
        big = 64    # input and score strides: dense in a space of their own
        strides = (C.c_int64 * 12)(big * 4, big, big * 4, big, st, sh, Hh, 1, Hh, 1, Hh, 1)
        code = f(far, 2 * far, 3 * far, 4 * far, 5 * far, 6 * far, T, Hh, D, strides, 0, None)
        assert code in (binding.ASTRA_ERR_BAD_SHAPE, binding.ASTRA_ERR_CUDA), code
        if code == binding.ASTRA_ERR_CUDA:
            assert not overlapping, (T, Hh, D, st, sh)   # an accepted layout is always disjoint
            accepted += 1
        elif overlapping:
            refused_overlapping += 1
        else:
            refused_disjoint += 1
    assert accepted > 300 and refused_overlapping > 300
    assert refused_disjoint < accepted   # the check is conservative only for unusual interleavings


def test_fp32_storage_needs_four_byte_alignment(lib):
    FP32 = binding.ASTRA_FP32
    assert FP32 == 2
    # 2-byte-aligned pointers are fine for the 16-bit types and misaligned for fp32
    assert lib.astra_silu_and_mul(A + 2, 2 * A, 0, 8, 0, None) == binding.ASTRA_OK
    assert lib.astra_silu_and_mul(A + 2, 2 * A, 1, 8, FP32, None) == binding.ASTRA_ERR_MISALIGNED
    assert lib.astra_fused_add_rmsnorm(A, 2 * A + 2, 3 * A, 1, 8, 1e-6, FP32, None) == binding.ASTRA_ERR_MISALIGNED
    assert lib.astra_merge_attn_states_lse(A, 2 * A, 3 * A + 2, 4 * A, 5 * A, 6 * A, 1, 2, 8, FP32, None) \
        == binding.ASTRA_ERR_MISALIGNED
    # overlap is judged in bytes of the storage type: [A, A+32) and [A+16, ...) overlap for fp32 rows of 8
    assert lib.astra_fused_add_rmsnorm(A, A + 16, 3 * A, 1, 8, 1e-6, FP32, None) == binding.ASTRA_ERR_OVERLAP
    assert lib.astra_silu_and_mul(A + 40, A, 1, 8, FP32, None) == binding.ASTRA_ERR_OVERLAP   # inside the up half
    assert lib.astra_silu_and_mul(A, 2 * A, 0, 8, FP32, None) == binding.ASTRA_OK


def test_headers_are_plain_c_and_link_from_c(tmp_path):
    """The public headers compile as strict C99, and a C program linked against libastra.so can call
    the error paths (nothing is launched)."""
    import subprocess
    astra_build.build()
    src = tmp_path / "use_from_c.c"
    src.write_text(r'''
#include <stdio.h>
#include "astra.h"
#include "astra_ablation.h"
int main(void) {
    float store[16] = {0};
    char *buf = (char *)store;  /* 4-byte aligned, as fp32 operands must be */
    astra_status_t s = astra_silu_and_mul(NULL, buf, 1, 8, ASTRA_BF16, NULL);
    if (s != ASTRA_ERR_NULL_POINTER) return 1;
    s = astra_fused_add_rmsnorm(buf, buf + 32, buf + 48, 0, 8, 1e-6f, ASTRA_FP32, NULL);
    if (s != ASTRA_OK) return 2;
    if (astra_status_string(ASTRA_ERR_OVERLAP)[0] == 0) return 3;
    printf("%s\n", astra_status_string(s));
    return 0;
}
''')
    exe = tmp_path / "use_from_c"
    libdir = os.path.dirname(astra_build.LIB_PATH)
    subprocess.check_call(["gcc", "-std=c99", "-pedantic", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"),
                           str(src), "-o", str(exe), "-L", libdir, "-lastra", f"-Wl,-rpath,{libdir}"])
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0 and out.stdout.strip() == "ok"


# ---- the _astra_fastcall extension (prepared calls re-issued without ctypes) --------------------

def test_fastcall_module_launches_what_ctypes_launches(lib):
    """The extension hands a prepared struct to the same entry points: for fake addresses (nothing
    can be launched on a machine without a GPU, and every argument error is reported first) each
    status equals the one the ctypes call returns for the same arguments."""
    fast = binding._fast
    assert fast is not None and fast.build_id() == astra_build.source_hash()
    cases = [
        (fast.KIND_RMSNORM, lib.astra_fused_add_rmsnorm, (A, 2 * A, 3 * A), (4, 64), 1e-6, 0, ()),
        (fast.KIND_RMSNORM, lib.astra_fused_add_rmsnorm, (A, A, 3 * A), (4, 64), 1e-6, 0, ()),          # overlap
        (fast.KIND_RMSNORM, lib.astra_fused_add_rmsnorm, (A + 1, 2 * A, 3 * A), (4, 64), 1e-6, 1, ()),  # misaligned
        (fast.KIND_RMSNORM, lib.astra_fused_add_rmsnorm, (A, 2 * A, 3 * A), (4, 0), 1e-6, 0, ()),       # bad shape
        (fast.KIND_RMSNORM, lib.astra_fused_add_rmsnorm, (None, None, None), (0, 64), 1e-6, 2, ()),     # empty batch
        (fast.KIND_SILU, lib.astra_silu_and_mul, (A, 2 * A), (4, 64), 0.0, 0, ()),
        (fast.KIND_SILU, lib.astra_silu_and_mul, (A, 2 * A), (4, 64), 0.0, 7, ()),                      # bad dtype
        (fast.KIND_SILU, lib.astra_silu_and_mul, (A, None), (4, 64), 0.0, 0, ()),                       # NULL
        (fast.KIND_MERGE, lib.astra_merge_attn_states_lse, (A, 2 * A, 3 * A, 4 * A, 5 * A, 6 * A), (4, 8, 64), 0.0, 0, ()),
        (fast.KIND_MERGE, lib.astra_merge_attn_states_lse, (A, None, 3 * A, 4 * A, 5 * A, 6 * A), (4, 8, 64), 0.0, 1, ()),
        (fast.KIND_MERGE, lib.astra_merge_attn_states_lse, (A, 4 * A, 3 * A, 4 * A, 5 * A, 6 * A), (4, 8, 64), 0.0, 0, ()),
    ]
    seen = set()
    for kind, fn, ptrs, ext, eps, dtype, parts in cases:
        ready = fast.prepare(kind, ptrs, ext, eps, dtype, parts)
        if kind == fast.KIND_RMSNORM:
            want = fn(*ptrs, *ext, eps, dtype, None)
        else:
            want = fn(*ptrs, *ext, dtype, None)
        got = fast.launch(ready, 0)
        assert got == want, (kind, ptrs, ext, dtype, got, want)
        seen.add(got)
    assert {binding.ASTRA_OK, binding.ASTRA_ERR_NULL_POINTER, binding.ASTRA_ERR_BAD_SHAPE, binding.ASTRA_ERR_BAD_DTYPE,
            binding.ASTRA_ERR_MISALIGNED, binding.ASTRA_ERR_OVERLAP} <= seen
    # the all-reduce form: the table of partials lives in the prepared struct
    table = (ctypes.c_void_p * 3)(4 * A, 5 * A, 6 * A)
    want = lib.astra_fused_allreduce_add_rmsnorm(A, 2 * A, table, 3, 3 * A, 4, 64, 1e-6, 0, None)
    got = fast.launch(fast.prepare(fast.KIND_ALLREDUCE_RMSNORM, (A, 2 * A, 3 * A), (4, 64), 1e-6, 0, (4 * A, 5 * A, 6 * A)), 0)
    assert got == want
    table = (ctypes.c_void_p * 2)(4 * A, A)   # a partial that is the output
    want = lib.astra_fused_allreduce_add_rmsnorm(A, 2 * A, table, 2, 3 * A, 4, 64, 1e-6, 0, None)
    got = fast.launch(fast.prepare(fast.KIND_ALLREDUCE_RMSNORM, (A, 2 * A, 3 * A), (4, 64), 1e-6, 0, (4 * A, A)), 0)
    assert got == want == binding.ASTRA_ERR_OVERLAP


def test_fastcall_module_refuses_malformed_preparations(lib):
    fast = binding._fast
    with pytest.raises(ValueError):
        fast.prepare(9, (A,), (1,), 0.0, 0, ())
    with pytest.raises(ValueError):
        fast.prepare(fast.KIND_SILU, (A, 2 * A, 3 * A), (4, 64), 0.0, 0, ())       # three pointers for a two-pointer call
    with pytest.raises(ValueError):
        fast.prepare(fast.KIND_MERGE, (A,) * 6, (4, 64), 0.0, 0, ())              # two extents for a three-extent call
    with pytest.raises(ValueError):
        fast.prepare(fast.KIND_RMSNORM, (A, 2 * A, 3 * A), (4, 64), 0.0, 0, (A,))  # partials on a call without any
    with pytest.raises(ValueError):
        fast.prepare(fast.KIND_ALLREDUCE_RMSNORM, (A, 2 * A, 3 * A), (4, 64), 0.0, 0, ())
    with pytest.raises(ValueError):
        fast.prepare(fast.KIND_ALLREDUCE_RMSNORM, (A, 2 * A, 3 * A), (4, 64), 0.0, 0, (A,) * 17)
    with pytest.raises(TypeError):
        fast.prepare(fast.KIND_SILU, (A, "x"), (4, 64), 0.0, 0, ())
    with pytest.raises(TypeError):
        fast.launch(object(), 0)
    with pytest.raises(TypeError):
        fast.Prepared()
