"""Builds the CUDA library (sm_100a only) in-tree with nvcc.

    python -m paper_2609_09821_b200.build [--force] [--verbose] [--debug]

The shared object lands in paper_2609_09821_b200/_build/libim_b200.so; it is a
plain C-ABI library (see include/im.h) with no Python or torch dependency.
--debug also builds libim_b200_debug.so: the same objects with the env kernel compiled
-DIM_DEBUG (every index it forms is bounds-checked and reported in the status word), the
stand-in for a memory checker on machines where none can be run.
"""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
OUT_DIR = os.path.join(_HERE, "_build")
LIB_PATH = os.path.join(OUT_DIR, "libim_b200.so")
DEBUG_LIB_PATH = os.path.join(OUT_DIR, "libim_b200_debug.so")
DEBUG_SOURCES = ["env_kernel.cu"]          # translation units that have IM_DEBUG checks
SOURCES = ["im_api.cu", "env_kernel.cu", "mlp_simt.cu", "mlp_tc.cu", "policy_noalloc.cu", "rollout.cu", "aos_adapter.cu", "ppo.cu", "optim.cu", "train.cu", "trainer.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    raise RuntimeError("nvcc not found")


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    path = _build(force, verbose, False)
    if debug:
        _build(force, verbose, True)
    return path


def _build(force: bool, verbose: bool, debug: bool) -> str:
    os.makedirs(OUT_DIR, exist_ok=True)
    lib_path = DEBUG_LIB_PATH if debug else LIB_PATH
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    headers.append(os.path.join(os.path.dirname(_HERE), "include", "im.h"))
    objs = []
    procs = []
    for src in SOURCES:
        s = os.path.join(CSRC, src)
        dbg = debug and src in DEBUG_SOURCES
        o = os.path.join(OUT_DIR, src.replace(".cu", "_debug.o" if dbg else ".o"))
        objs.append(o)
        if force or _stale(o, [s] + headers):
            cmd = [_nvcc()] + NVCC_FLAGS + (["-DIM_DEBUG"] if dbg else []) + (["-Xptxas", "-v"] if verbose else []) + ["-c", s, "-o", o]
            procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    failed = False
    for src, p in procs:
        out, _ = p.communicate()
        if p.returncode != 0 or verbose:
            sys.stderr.write("---- %s\n%s\n" % (src, out))
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    if force or procs or _stale(lib_path, objs):
        cmd = [_nvcc(), "-shared", "-Wno-deprecated-gpu-targets", "-o", lib_path + ".tmp"] + objs + \
              ["-Xlinker", "--exclude-libs,ALL"]
        subprocess.check_call(cmd)
        os.replace(lib_path + ".tmp", lib_path)
    return lib_path


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug="--debug" in sys.argv))
