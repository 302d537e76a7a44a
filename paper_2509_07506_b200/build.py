"""Build ``libastra.so`` (the CUDA kernels and their C ABI) for sm_100a with nvcc.

Usage: ``python -m paper_2509_07506_b200.build [--force]``.  The shared object is written next
to this file; nothing is installed outside the source tree.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG_DIR)
CSRC = os.path.join(PKG_DIR, "csrc")
INCLUDE = os.path.join(ROOT, "include")
LIB_PATH = os.path.join(PKG_DIR, "libastra.so")
ABLATION_LIB_PATH = os.path.join(PKG_DIR, "libastra_ablation.so")

SOURCES = ["astra.cu"]
ABLATION_SOURCES = ["ablation.cu"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-std=c++17", "-lineinfo",
    "-Xcompiler", "-fPIC", "-shared",
    "-cudart", "static",
]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found: libastra.so cannot be built")
    return exe


def _inputs():
    files = [os.path.join(INCLUDE, f) for f in os.listdir(INCLUDE) if f.endswith(".h")]
    files += [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cu", ".cuh", ".h"))]
    return files


def is_stale(lib_path: str = LIB_PATH) -> bool:
    if not os.path.exists(lib_path):
        return True
    built = os.path.getmtime(lib_path)
    return any(os.path.getmtime(f) > built for f in _inputs())


def _compile(lib_path: str, sources, force: bool, verbose: bool, extra_flags=()) -> str:
    if not force and not is_stale(lib_path):
        return lib_path
    tmp = lib_path + f".tmp{os.getpid()}"
    cmd = [_nvcc(), *NVCC_FLAGS, *extra_flags, "-I", INCLUDE, "-I", CSRC, "-o", tmp]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in sources]
    subprocess.check_call(cmd)
    os.replace(tmp, lib_path)
    return lib_path


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile libastra.so if it is missing or older than any source; returns its path."""
    return _compile(LIB_PATH, SOURCES, force, verbose)


def ensure_built(ablation: bool = False) -> str:
    """Build if missing or stale; if the rebuild is impossible (no compiler on this machine) but a
    built library is present, keep using it and say so.  A missing library is always an error."""
    path = ABLATION_LIB_PATH if ablation else LIB_PATH
    try:
        return build_ablation() if ablation else build()
    except Exception as exc:  # noqa: BLE001
        if os.path.exists(path):
            print(f"[astra build] could not rebuild {os.path.basename(path)} ({exc}); using the existing one",
                  file=sys.stderr)
            return path
        raise


def build_variant(lib_path: str, defines: dict) -> str:
    """Compile libastra's sources to `lib_path` with extra preprocessor definitions (used by the
    tests to lower the per-launch limits so that the multi-launch splitting runs on small inputs)."""
    flags = [f"-D{k}={v}" for k, v in defines.items()]
    return _compile(lib_path, SOURCES, True, False, flags)


def build_ablation(force: bool = False, verbose: bool = False) -> str:
    """Compile libastra_ablation.so (the paper's design pairs, for the ablation measurements)."""
    return _compile(ABLATION_LIB_PATH, ABLATION_SOURCES, force, verbose)


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
    print(build_ablation(force="--force" in sys.argv, verbose="-v" in sys.argv))
