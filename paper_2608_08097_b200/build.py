"""Builds the CUDA library (csrc/*.cu -> liboasis.so, in-tree) for sm_100a.

nvcc cross-compiles without a GPU.  Objects are rebuilt only when their source (or a
header) is newer; `python -m paper_2608_08097_b200.build --force` rebuilds everything,
`--verbose` adds -Xptxas -v (registers, spills, shared memory per kernel), `--checked` builds
the bounds-check variant (liboasis_checked.so, -DOASIS_BOUNDS_CHECK: every index read from a
device array is range-checked on the device; see include/oasis.h).
"""
import concurrent.futures
import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "liboasis.so")
OBJ_CHECKED = os.path.join(HERE, "build_checked")
LIB_CHECKED = os.path.join(HERE, "liboasis_checked.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]
FLAGS = ["-O3", "-std=c++17", "-lineinfo", "-Xcompiler", "-fPIC"]


def _newest_header():
    hdrs = glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(HERE, "..", "include", "*.h"))
    return max(os.path.getmtime(h) for h in hdrs)


def _compile(src, verbose, obj_dir=OBJ, defines=()):
    obj = os.path.join(obj_dir, os.path.basename(src)[:-3] + ".o")
    cmd = [NVCC, *ARCH, *FLAGS, *defines, "-c", src, "-o", obj]
    if verbose:
        cmd[1:1] = ["-Xptxas", "-v"]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed for %s:\n%s\n%s" % (src, r.stdout, r.stderr))
    return obj, r.stderr


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    obj_dir, lib = (OBJ_CHECKED, LIB_CHECKED) if checked else (OBJ, LIB)
    defines = ("-DOASIS_BOUNDS_CHECK",) if checked else ()
    os.makedirs(obj_dir, exist_ok=True)
    srcs = sorted(glob.glob(os.path.join(CSRC, "*.cu")))
    hdr_time = _newest_header()
    todo, objs = [], []
    for s in srcs:
        obj = os.path.join(obj_dir, os.path.basename(s)[:-3] + ".o")
        objs.append(obj)
        if (force or verbose or not os.path.exists(obj)
                or os.path.getmtime(obj) < max(os.path.getmtime(s), hdr_time)):
            todo.append(s)
    if todo:
        with concurrent.futures.ThreadPoolExecutor(max_workers=8) as ex:
            for obj, log in ex.map(lambda s: _compile(s, verbose, obj_dir, defines), todo):
                if verbose and log:
                    sys.stderr.write(log)
    if todo or not os.path.exists(lib) or any(os.path.getmtime(o) > os.path.getmtime(lib) for o in objs):
        cmd = [NVCC, *ARCH, "-shared", "-cudart", "static", "-o", lib, *objs]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError("link failed:\n%s\n%s" % (r.stdout, r.stderr))
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, checked="--checked" in sys.argv))
