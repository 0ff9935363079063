"""Build the CUDA library in-tree: nvcc, sm_100a only, one shared object next to this file."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
LIB = os.path.join(HERE, "libasd_b200.so")
SOURCES = ["asd_api.cu", "asd_kernels.cu", "asd_resident.cu", "asd_gemm.cu", "asd_mlp_fused.cu", "asd_static.cu", "asd_schedule.cu"]


def _newest(paths):
    return max(os.path.getmtime(p) for p in paths)


def build(force: bool = False, verbose: bool = False) -> str:
    srcs = [os.path.join(HERE, "csrc", s) for s in SOURCES]
    deps = srcs + [os.path.join(HERE, "csrc", "asd_internal.h"), os.path.join(HERE, "csrc", "asd_device.cuh"),
                   os.path.join(HERE, "csrc", "asd_tc.cuh"),
                   os.path.join(ROOT, "include", "asd.h")]
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= _newest(deps):
        return LIB
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC",
             "-I" + os.path.join(ROOT, "include")]
    if verbose:
        flags.append("-Xptxas=-v")
    # one object per translation unit, compiled side by side (no device code is linked across them)
    obj_dir = os.path.join(HERE, "_build")
    os.makedirs(obj_dir, exist_ok=True)
    hdr_time = _newest(deps[len(srcs):])
    jobs = []
    for src in srcs:
        obj = os.path.join(obj_dir, os.path.basename(src)[:-3] + ".o")
        if force or verbose or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(src), hdr_time):
            jobs.append((src, subprocess.Popen([nvcc] + flags + ["-c", src, "-o", obj], stdout=subprocess.PIPE,
                                               stderr=subprocess.STDOUT, text=True)))
    log = []
    for src, proc in jobs:
        out, _ = proc.communicate()
        log.append(out)
        if proc.returncode != 0:
            raise RuntimeError("nvcc failed on " + src + ":\n" + out)
    objs = [os.path.join(obj_dir, os.path.basename(src)[:-3] + ".o") for src in srcs]
    res = subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-cudart", "static", "-o", LIB] + objs,
                         capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("link failed:\n" + res.stdout + res.stderr)
    if verbose:
        print("".join(log))
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
