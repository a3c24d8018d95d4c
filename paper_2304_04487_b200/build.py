"""Build ``libllma_b200.so`` in-tree with nvcc for sm_100a."""
from __future__ import annotations

import glob
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
# LLMA_BUILD_STAMPS=1 builds the measurement variant (in-kernel timestamps, see LLMA_STAMPS in csrc/common.cuh)
# into the same library name but a build folder of its own; switch back by rebuilding without the variable.
STAMPS = os.environ.get("LLMA_BUILD_STAMPS") == "1"
OBJ = os.path.join(HERE, "_build_stamps" if STAMPS else "_build")
LIB = os.path.join(HERE, "libllma_b200.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
         "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr"] + (["-DLLMA_STAMPS"] if STAMPS else [])


def _sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale(target, deps):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    os.makedirs(OBJ, exist_ok=True)
    headers = glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh")) + \
        glob.glob(os.path.join(HERE, "..", "include", "*.h"))
    jobs = []
    objs = []
    for src in _sources():
        obj = os.path.join(OBJ, os.path.basename(src)[:-3] + ".o")
        objs.append(obj)
        if force or _stale(obj, [src] + headers):
            cmd = [NVCC] + FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-c", src, "-o", obj]
            jobs.append(cmd)

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0 or verbose:
            print(" ".join(cmd)); print(r.stdout); print(r.stderr)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed: " + " ".join(cmd))

    with ThreadPoolExecutor(max_workers=8) as ex:
        list(ex.map(run, jobs))
    marker = os.path.join(OBJ, ".linked")
    if force or jobs or _stale(LIB, objs) or not os.path.exists(marker):
        run([NVCC, "-shared", "-o", LIB] + objs + ["-cudart", "static"])
        for d in (os.path.join(HERE, "_build"), os.path.join(HERE, "_build_stamps")):   # the library now holds THIS variant
            if os.path.exists(os.path.join(d, ".linked")):
                os.remove(os.path.join(d, ".linked"))
        open(marker, "w").close()
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
