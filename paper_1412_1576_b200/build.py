"""Builds the CUDA library in-tree with nvcc for sm_100a.

``python -m paper_1412_1576_b200.build`` (or ``build_library()``) compiles
``csrc/*.cu`` into ``paper_1412_1576_b200/_lib/liblda_b200.so``.  nvcc
cross-compiles without a GPU.  FMA contraction is off (``-fmad=false``) so the
acceptance test of the sampler rounds exactly like plain IEEE double arithmetic.
"""

from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB_DIR = os.path.join(HERE, "_lib")
LIB_PATH = os.path.join(LIB_DIR, "liblda_b200.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-fmad=false", "-Xcompiler", "-fPIC", "-shared", "-Xptxas", "-v",
]


def _nvcc() -> str:
    cand = os.environ.get("NVCC") or "/usr/local/cuda/bin/nvcc"
    return cand if os.path.exists(cand) else "nvcc"


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + \
        glob.glob(os.path.join(HERE, "..", "include", "*.h"))
    return any(os.path.getmtime(p) > t for p in deps)


def build_library(force: bool = False, verbose: bool = False, extra_flags=(), out: str | None = None) -> str:
    """Compiles every source to an object file (in parallel) and links them.  ``extra_flags`` and
    ``out`` build a variant of the library somewhere else (objects then go to a folder of their own)."""
    out = out or LIB_PATH
    if not force and not extra_flags and out == LIB_PATH and not _stale():
        return LIB_PATH
    os.makedirs(os.path.dirname(out), exist_ok=True)
    obj_dir = os.path.join(os.path.dirname(out), "_build" if out == LIB_PATH and not extra_flags
                           else "_build_" + os.path.basename(out))
    os.makedirs(obj_dir, exist_ok=True)
    compile_flags = [f for f in NVCC_FLAGS if f != "-shared"] + list(extra_flags)
    procs = []
    for src in sources():
        obj = os.path.join(obj_dir, os.path.basename(src)[:-3] + ".o")
        cmd = [_nvcc()] + compile_flags + ["-c", src, "-o", obj]
        procs.append((cmd, obj, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    log, failed, objs = "", False, []
    for cmd, obj, pr in procs:
        text = pr.communicate()[0]
        log += " ".join(cmd) + "\n" + text
        failed = failed or pr.returncode != 0
        objs.append(obj)
    if not failed:
        tmp = out + f".{os.getpid()}.tmp"
        cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-shared"] + objs + ["-o", tmp]
        res = subprocess.run(cmd, capture_output=True, text=True)
        log += " ".join(cmd) + "\n" + res.stdout + res.stderr
        failed = res.returncode != 0
        if not failed:
            os.replace(tmp, out)
    with open(os.path.join(os.path.dirname(out), "build.log" if out == LIB_PATH else os.path.basename(out) + ".log"),
              "w") as f:
        f.write(log)
    if failed:
        raise RuntimeError("nvcc failed:\n" + log[-8000:])
    if verbose:
        print(log)
    return out


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv))
