"""Build ``libdeer.so`` (the C-ABI library) in-tree with nvcc for sm_100a.

``python -m paper_2512_15176_b200.build`` or :func:`build`.  Objects go to
``_build/`` next to this file; a source is recompiled only when it, or a header,
is newer than its object.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(ROOT, "include")
BUILD = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libdeer.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-I", INCLUDE, "-I", CSRC,
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found; cannot build libdeer.so")


def sources():
    return sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cu"))


def _headers_mtime() -> float:
    hs = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    hs += [os.path.join(INCLUDE, f) for f in os.listdir(INCLUDE)]
    return max(os.path.getmtime(h) for h in hs)


PROBES_LIB = os.path.join(HERE, "libdeer_probes.so")


def build(force: bool = False, verbose: bool = False, ptxas_info: bool = False, probes: bool = False) -> str:
    """Build the library; with ``probes`` a second one, ``libdeer_probes.so``, compiled with DEER_TIMING_PROBES (the
    kernels then record clock values at the hand-overs of their pipelines; see ``profile_case.py --probes``)."""
    build_dir = BUILD + ("_probes" if probes else "")
    lib = PROBES_LIB if probes else LIB
    os.makedirs(build_dir, exist_ok=True)
    nvcc = _nvcc()
    hm = _headers_mtime()
    flags = list(NVCC_FLAGS)
    if probes:
        flags += ["-DDEER_TIMING_PROBES"]
    if ptxas_info:
        flags += ["-Xptxas", "-v"]
    jobs = []
    objs = []
    for src in sources():
        obj = os.path.join(build_dir, os.path.basename(src)[:-3] + ".o")
        objs.append(obj)
        if force or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(src), hm):
            jobs.append([nvcc, *flags, "-c", src, "-o", obj])

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or ptxas_info or r.returncode != 0:
            sys.stderr.write(" ".join(cmd) + "\n" + r.stdout + r.stderr)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed for " + cmd[-3])

    with ThreadPoolExecutor(max_workers=min(8, max(1, len(jobs)))) as ex:
        list(ex.map(run, jobs))
    if jobs or not os.path.exists(lib):
        run([nvcc, "-shared", "-o", lib, *objs])
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, ptxas_info="--ptxas" in sys.argv, probes="--probes" in sys.argv))
