"""Builds libslide_attn.so (sm_100a) from csrc/ with nvcc, in-tree.

    python -m paper_2304_04237_b200.build [--force] [--verbose] [--probes] [--timeline]

Objects go to paper_2304_04237_b200/_build/, the library next to this file.  nvcc
cross-compiles, so no GPU is needed to build.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libslide_attn.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    return "nvcc"


def _newest_header() -> float:
    hs = glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(CSRC, "*.h")) + \
        glob.glob(os.path.join(ROOT, "include", "*.h"))
    return max(os.path.getmtime(h) for h in hs)


def build(force: bool = False, verbose: bool = False) -> str:
    os.makedirs(OBJ, exist_ok=True)
    srcs = sorted(glob.glob(os.path.join(CSRC, "*.cu")))
    hdr_t = _newest_header()
    extra = ["-Xptxas", "-v"] if verbose else []
    jobs = []
    for s in srcs:
        o = os.path.join(OBJ, os.path.basename(s)[:-3] + ".o")
        if force or not os.path.exists(o) or os.path.getmtime(o) < max(os.path.getmtime(s), hdr_t):
            jobs.append([_nvcc(), *NVCC_FLAGS, *extra, "-c", s, "-o", o])

    def run(cmd):
        return cmd, subprocess.run(cmd, capture_output=True, text=True)

    with ThreadPoolExecutor(max_workers=min(8, max(1, len(jobs)))) as ex:
        for cmd, r in ex.map(run, jobs):
            if verbose or r.returncode != 0:
                sys.stderr.write(" ".join(cmd) + "\n" + r.stdout + r.stderr)
            if r.returncode != 0:
                raise RuntimeError("nvcc failed for " + cmd[-3])
    objs = [os.path.join(OBJ, os.path.basename(s)[:-3] + ".o") for s in srcs]
    if jobs or force or not os.path.exists(LIB):
        tmp = LIB + f".tmp{os.getpid()}"
        cmd = [_nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a", *objs, "-o", tmp]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
            raise RuntimeError("link failed")
        os.replace(tmp, LIB)
    return LIB


def build_probes() -> list:
    """Compiles the stand-alone measurement programs of probes/ (not part of the library)."""
    src_dir = os.path.join(HERE, "probes")
    out_dir = os.path.join(src_dir, "_build")
    os.makedirs(out_dir, exist_ok=True)
    outs = []
    for s in sorted(glob.glob(os.path.join(src_dir, "*.cu"))):
        exe = os.path.join(out_dir, os.path.basename(s)[:-3])
        r = subprocess.run([_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
                            "-I", CSRC, "-I", os.path.join(ROOT, "include"), s, "-o", exe], capture_output=True, text=True)
        if r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
            raise RuntimeError("nvcc failed for " + s)
        outs.append(exe)
    return outs


def build_timeline() -> str:
    """A second copy of the library with -DSLIDE_ATTN_TIMELINE (clock stamps in the projection kernel's role loops),
    as probes/_build/libslide_attn_timeline.so; read by probes/proj_timeline.py."""
    out_dir = os.path.join(HERE, "probes", "_build", "timeline")
    os.makedirs(out_dir, exist_ok=True)
    objs = []
    for s in sorted(glob.glob(os.path.join(CSRC, "*.cu"))):
        o = os.path.join(out_dir, os.path.basename(s)[:-3] + ".o")
        r = subprocess.run([_nvcc(), *NVCC_FLAGS, "-DSLIDE_ATTN_TIMELINE", "-c", s, "-o", o], capture_output=True, text=True)
        if r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
            raise RuntimeError("nvcc failed for " + s)
        objs.append(o)
    lib = os.path.join(HERE, "probes", "_build", "libslide_attn_timeline.so")
    r = subprocess.run([_nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a", *objs, "-o", lib],
                       capture_output=True, text=True)
    if r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
        raise RuntimeError("link failed")
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
    if "--probes" in sys.argv:
        print("\n".join(build_probes()))
    if "--timeline" in sys.argv:
        print(build_timeline())
