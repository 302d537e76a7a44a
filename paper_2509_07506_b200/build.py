"""Build ``libastra.so`` (the CUDA kernels and their C ABI) for sm_100a with nvcc, the ablation
library beside it, and ``_astra_fastcall`` (a small CPython extension that re-issues prepared calls
without ctypes) with the host C compiler.

Usage: ``python -m paper_2509_07506_b200.build [--force]``.  The shared objects are written next
to this file; nothing is installed outside the source tree.
"""
from __future__ import annotations

import hashlib
import os
import re
import shutil
import subprocess
import sys
import sysconfig

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG_DIR)
CSRC = os.path.join(PKG_DIR, "csrc")
INCLUDE = os.path.join(ROOT, "include")
LIB_PATH = os.path.join(PKG_DIR, "libastra.so")
ABLATION_LIB_PATH = os.path.join(PKG_DIR, "libastra_ablation.so")
FASTCALL_PATH = os.path.join(PKG_DIR, "_astra_fastcall.so")

SOURCES = ["astra.cu", "astra_allreduce.cu"]
ABLATION_SOURCES = ["ablation.cu"]
FASTCALL_SOURCES = ["fastcall.c"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-std=c++17", "-lineinfo",
    "-Xcompiler", "-fPIC", "-shared",
    "-cudart", "static",
    "--threads", "0",
]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found: libastra.so cannot be built")
    return exe


def _inputs():
    files = [os.path.join(INCLUDE, f) for f in os.listdir(INCLUDE) if f.endswith(".h")]
    files += [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cu", ".cuh", ".h", ".c"))]
    return files


_ID_MARKER = b"astra-build-id:"


def source_hash(extra_flags=()) -> str:
    """SHA-256 over the names and contents of every header and CUDA source (and the extra compiler
    flags of a variant build).  It is compiled into each library, so a library can be matched to the
    sources beside it by content; file times, which a copy or a checkout rewrites, play no part."""
    h = hashlib.sha256()
    for path in sorted(_inputs()):
        h.update(os.path.basename(path).encode() + b"\0")
        with open(path, "rb") as fh:
            h.update(fh.read())
        h.update(b"\0")
    for flag in extra_flags:
        h.update(flag.encode() + b"\0")
    return h.hexdigest()


def embedded_hash(lib_path: str):
    """The source hash compiled into a built library (read from the file, without loading it), or None."""
    try:
        with open(lib_path, "rb") as fh:
            blob = fh.read()
    except OSError:
        return None
    m = re.search(re.escape(_ID_MARKER) + rb"([0-9a-f]{64})", blob)
    return m.group(1).decode() if m else None


def is_stale(lib_path: str = LIB_PATH, extra_flags=()) -> bool:
    """True when the library is missing or was not built from the sources now on disk."""
    return embedded_hash(lib_path) != source_hash(extra_flags)


def _compile(lib_path: str, sources, force: bool, verbose: bool, extra_flags=()) -> str:
    if not force and not is_stale(lib_path, extra_flags):
        return lib_path
    tmp = lib_path + f".tmp{os.getpid()}"
    cmd = [_nvcc(), *NVCC_FLAGS, *extra_flags, f'-DASTRA_BUILD_ID="{source_hash(extra_flags)}"',
           "-I", INCLUDE, "-I", CSRC, "-o", tmp]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in sources]
    subprocess.check_call(cmd)
    os.replace(tmp, lib_path)
    return lib_path


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile libastra.so (and the _astra_fastcall extension the binding loads with it) if missing or
    built from other sources; returns the library's path."""
    build_fastcall(force)
    return _compile(LIB_PATH, SOURCES, force, verbose)


def build_fastcall(force: bool = False) -> str:
    """Compile the _astra_fastcall extension (plain C against the CPython headers) if it is missing
    or was built from other sources; returns its path."""
    if not force and not is_stale(FASTCALL_PATH):
        return FASTCALL_PATH
    cc = shutil.which("gcc") or shutil.which("cc")
    if cc is None:
        raise RuntimeError("no C compiler found: _astra_fastcall cannot be built")
    tmp = FASTCALL_PATH + f".tmp{os.getpid()}"
    cmd = [cc, "-O2", "-std=c11", "-fPIC", "-shared", "-fvisibility=hidden", f'-DASTRA_BUILD_ID="{source_hash()}"',
           "-I", sysconfig.get_paths()["include"], "-I", INCLUDE, "-o", tmp]
    cmd += [os.path.join(CSRC, s) for s in FASTCALL_SOURCES]
    subprocess.check_call(cmd)
    os.replace(tmp, FASTCALL_PATH)
    return FASTCALL_PATH


def ensure_built(ablation: bool = False) -> str:
    """Build if the library is missing or does not match the sources on disk.  A library that cannot
    be rebuilt (no compiler on this machine) and does not match is an error: results must never come
    from a library other than the one the sources describe."""
    return build_ablation() if ablation else build()


def build_variant(lib_path: str, defines: dict) -> str:
    """Compile libastra's sources to `lib_path` with extra preprocessor definitions (used by the
    tests to lower the per-launch limits so that the multi-launch splitting runs on small inputs)."""
    flags = [f"-D{k}={v}" for k, v in sorted(defines.items())]
    return _compile(lib_path, SOURCES, False, False, flags)


def build_ablation(force: bool = False, verbose: bool = False) -> str:
    """Compile libastra_ablation.so (the paper's design pairs, for the ablation measurements)."""
    return _compile(ABLATION_LIB_PATH, ABLATION_SOURCES, force, verbose)


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
    print(FASTCALL_PATH)
    print(build_ablation(force="--force" in sys.argv, verbose="-v" in sys.argv))
