"""Build the CUDA library in-tree for sm_100a (nvcc cross-compiles without a GPU).

    python -m paper_1911_09030_b200.build [--force] [--debug]

Produces `paper_1911_09030_b200/liblocal_adaalter.so`; with --debug the checked build
`liblocal_adaalter_debug.so` (the same sources with -DLA_DEBUG: kernels range-check their
addresses).  Object files go to `paper_1911_09030_b200/_build/` (`_build/debug/`).  Device code is compiled with `-fmad=false`: every
fused multiply-add in the kernels is written explicitly, none may be introduced.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "liblocal_adaalter.so")
NVCC = os.environ.get("NVCC", "nvcc")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
         "-fmad=false", "-Xcompiler", "-fPIC", "-Xcompiler", "-O2",
         "-Xfatbin=-compress-all"]   # every worker count up to 16 has its own kernels: keep the image small


def _sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps():
    return (glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(CSRC, "*.inc"))
            + glob.glob(os.path.join(HERE, "..", "include", "*.h")))


def _stale(target, inputs):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(p) > t for p in inputs)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    OBJ = os.path.join(HERE, "_build", "debug") if debug else globals()["OBJ"]
    LIB = os.path.join(HERE, "liblocal_adaalter_debug.so") if debug else globals()["LIB"]
    FLAGS = globals()["FLAGS"] + (["-DLA_DEBUG"] if debug else [])
    os.makedirs(OBJ, exist_ok=True)
    srcs, deps = _sources(), _deps()
    if debug:  # the checked build instantiates the first set of worker counts only (compile time)
        keep = {"la_sweep_w%d.cu" % w for w in (0, 1, 2, 3, 4, 6, 8, 12, 16)}
        srcs = [s for s in srcs if not os.path.basename(s).startswith("la_sweep_w") or os.path.basename(s) in keep]
    jobs = []
    for s in srcs:
        o = os.path.join(OBJ, os.path.basename(s)[:-3] + ".o")
        if force or _stale(o, [s] + deps):
            jobs.append((s, o))

    def cc(job):
        s, o = job
        cmd = [NVCC] + FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-c", s, "-o", o]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed for %s:\n%s" % (s, r.stderr))
        return r.stderr

    with ThreadPoolExecutor(max_workers=max(1, min(8, len(jobs) or 1))) as ex:
        logs = list(ex.map(cc, jobs))
    if verbose:
        sys.stderr.write("".join(logs))
    objs = [os.path.join(OBJ, os.path.basename(s)[:-3] + ".o") for s in srcs]
    if force or jobs or _stale(LIB, objs):
        cmd = [NVCC, "-shared", "-o", LIB + ".tmp"] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError("link failed:\n" + r.stderr)
        os.replace(LIB + ".tmp", LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
