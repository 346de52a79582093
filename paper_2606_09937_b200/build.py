"""Builds librksc.so (sm_100a) in-tree with nvcc.  `python -m paper_2606_09937_b200.build`."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
REPO_DIR = os.path.dirname(PKG_DIR)
CSRC = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.path.join(PKG_DIR, "librksc.so")
SOURCES = ["api.cu", "plan.cpp", "gate.cu", "attn_warp.cu", "attn_tc.cu", "merge.cu", "rsbcm.cu", "cgee.cu", "pipeline.cpp"]
HEADERS = ["rksc_internal.h", "kernels.h"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the CUDA library cannot be built")


def _stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS]
    deps.append(os.path.join(REPO_DIR, "include", "rksc.h"))
    deps.append(os.path.abspath(__file__))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, extra_flags=(), out_path: str = LIB_PATH) -> str:
    """Compile every CUDA source for sm_100a and link the shared library; returns its path.

    ``extra_flags`` / ``out_path`` build a variant (e.g. ``-DRKSC_WAIT_PROFILE``) beside the product library."""
    if out_path == LIB_PATH and not force and not _stale():
        return LIB_PATH
    cmd = [
        _nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
        "-shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
        "-I", os.path.join(REPO_DIR, "include"), "-I", CSRC,
        "-DRKSC_BUILD",
    ]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += list(extra_flags)
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    cmd += ["-o", out_path + ".tmp"]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    os.replace(out_path + ".tmp", out_path)
    if verbose:
        print(res.stderr)
    return out_path


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
