"""Build the CUDA library in-tree: csrc/*.cu -> libpvq_b200.so next to this file.

`python -m paper_2410_16926_b200.build [--force] [--verbose] [--debug]`.  sm_100a only.
Objects go to _build/ (not committed); translation units compile in parallel.

--debug builds libpvq_b200_debug.so instead: the bounds-checked variant (-DPVQ_DEBUG, see
pvq_debug_status in include/pvq.h) of the kernels that keep their tables in shared memory;
the global-table kernels are left out of it (calls that need them return "unsupported").
"""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
OBJDIR = os.path.join(ROOT, "_build")
LIB = os.path.join(HERE, "libpvq_b200.so")
DEBUG_LIB = os.path.join(HERE, "libpvq_b200_debug.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def _sources():
    return sorted(f for f in os.listdir(CSRC) if f.endswith(".cu"))


def _headers_mtime():
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    paths.append(os.path.join(ROOT, "include", "pvq.h"))
    return max(os.path.getmtime(p) for p in paths)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    objdir = os.path.join(OBJDIR, "debug") if debug else OBJDIR
    lib = DEBUG_LIB if debug else LIB
    os.makedirs(objdir, exist_ok=True)
    hdr = _headers_mtime()
    jobs, objs = [], []
    sources = _sources()
    extra = []
    if debug:  # the shared-memory kernels only; the rest of the launchers answer "unsupported"
        sources = [f for f in sources if not f.startswith(("pvq_big", "pvq_wide"))]
        extra = ["-DPVQ_DEBUG"]
    for src in sources:
        s = os.path.join(CSRC, src)
        o = os.path.join(objdir, src[:-3] + ".o")
        objs.append(o)
        if force or not os.path.exists(o) or os.path.getmtime(o) < max(os.path.getmtime(s), hdr):
            cmd = ["nvcc"] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-c", s, "-o", o]
            jobs.append(cmd)

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        return cmd, r

    if jobs:
        with ThreadPoolExecutor(max_workers=min(os.cpu_count() or 8, len(jobs))) as ex:
            for cmd, r in ex.map(run, jobs):
                if verbose or r.returncode != 0:
                    sys.stderr.write(" ".join(cmd) + "\n" + r.stdout + r.stderr)
                if r.returncode != 0:
                    raise RuntimeError("nvcc failed for " + cmd[-3])
    if jobs or not os.path.exists(lib):
        link = ["nvcc", "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", lib] + objs
        r = subprocess.run(link, capture_output=True, text=True)
        if r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
            raise RuntimeError("link failed")
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug="--debug" in sys.argv))
