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


def declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(astra_[a-z0-9_]+)\s*\(", text))
    return names


def test_every_declared_function_is_exported(lib):
    names = declared_functions()
    assert {"astra_fused_add_rmsnorm", "astra_silu_and_mul", "astra_merge_attn_states_lse",
            "astra_status_string"} <= names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/ but not exported"
    assert set(binding.EXPORTED_SYMBOLS) <= names


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


def test_silu_argument_errors(lib):
    f = lib.astra_silu_and_mul
    assert f(None, A, 1, 8, 0, None) == binding.ASTRA_ERR_NULL_POINTER
    assert f(A, None, 1, 8, 0, None) == binding.ASTRA_ERR_NULL_POINTER
    assert f(A, 2 * A, 1, 8, 2, None) == binding.ASTRA_ERR_BAD_DTYPE
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
