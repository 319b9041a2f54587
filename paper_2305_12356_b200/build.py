"""Compile the CUDA sources in csrc/ for sm_100a into in-tree shared libraries.

  libmofq.so        the C-ABI library declared in include/mofq.h
  libmofq_synth.so  the synthetic-input generator (inputs only; no quantisation arithmetic)
"""
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(_HERE)
CSRC = os.path.join(_HERE, "csrc")
INCLUDE = os.path.join(ROOT, "include")
BUILD_DIR = os.path.join(_HERE, "_build")

LIB = os.path.join(_HERE, "libmofq.so")
SYNTH_LIB = os.path.join(_HERE, "libmofq_synth.so")

LIB_SOURCES = ["mofq_kq.cu", "mofq_kq_mt.cu", "mofq_kq_rows.cu", "mofq_layer.cu", "mofq_api.cu", "mofq_noalloc.cu", "mofq_diag.cu"]
SYNTH_SOURCES = ["mofq_synth.cu"]

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-I", INCLUDE, "-I", CSRC]


def _nvcc():
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _newer(target, deps):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def _headers():
    hs = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    hs += [os.path.join(INCLUDE, f) for f in os.listdir(INCLUDE)]
    return hs


def _build_lib(target, sources, force, verbose):
    os.makedirs(BUILD_DIR, exist_ok=True)
    objs, procs = [], []
    for src in sources:
        sp = os.path.join(CSRC, src)
        obj = os.path.join(BUILD_DIR, src + ".o")
        objs.append(obj)
        if force or _newer(obj, [sp] + _headers()):
            cmd = [_nvcc(), *NVCC_FLAGS, "-c", sp, "-o", obj]
            if verbose:
                cmd.insert(1, "-Xptxas=-v")
            procs.append((cmd, subprocess.Popen(cmd)))
    for cmd, p in procs:
        if p.wait() != 0:
            raise RuntimeError("nvcc failed: " + " ".join(cmd))
    if procs or not os.path.exists(target):
        tmp = target + ".tmp.%d" % os.getpid()
        subprocess.run([_nvcc(), "-Wno-deprecated-gpu-targets", "-shared", "-o", tmp, *objs, "-lcudart"], check=True)
        os.replace(tmp, target)
    return target


def build(force=False, verbose=False):
    _build_lib(LIB, LIB_SOURCES, force, verbose)
    _build_lib(SYNTH_LIB, SYNTH_SOURCES, force, verbose)
    return LIB, SYNTH_LIB


if __name__ == "__main__":
    import sys
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
