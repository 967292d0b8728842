"""Compile libufp4.so (the C-ABI CUDA library) in-tree for sm_100a with nvcc.  Cross-compiles without a GPU.

Each .cu file becomes an object under build/ (git-ignored), compiled in parallel and only when it, a header or the flags
changed; the objects are then linked into libufp4.so.
"""
import concurrent.futures
import glob
import hashlib
import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
OBJ_DIR = os.path.join(_HERE, "build")
LIB = os.path.join(_HERE, "libufp4.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=default",
    # bit-exact quantizer arithmetic: IEEE division/sqrt, no flush-to-zero, no implicit FMA contraction
    "-prec-div=true", "-prec-sqrt=true", "-ftz=false", "-fmad=false",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _headers():
    return sorted(glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(_HERE, "..", "include", "*.h")))


def _stamp(extra):
    """Hash of everything besides the source file itself that an object depends on."""
    h = hashlib.sha256(" ".join(NVCC_FLAGS + list(extra)).encode())
    for p in _headers():
        with open(p, "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def _compile_one(nvcc, src, obj, extra, verbose):
    cmd = [nvcc, *NVCC_FLAGS, *extra, *(["-Xptxas", "-v"] if verbose else []), "-c", "-o", obj, src]
    out = subprocess.run(cmd, capture_output=True, text=True)
    if out.returncode != 0:
        raise RuntimeError("nvcc failed on %s:\n%s" % (src, out.stderr))
    return out.stderr


def build(force: bool = False, verbose: bool = False, extra_flags=(), lib_path: str = LIB) -> str:
    nvcc = os.environ.get("NVCC", "nvcc")
    extra = list(extra_flags)
    stamp = _stamp(extra)
    tag = os.path.splitext(os.path.basename(lib_path))[0]
    os.makedirs(OBJ_DIR, exist_ok=True)
    jobs, objs = [], []
    for src in sources():
        obj = os.path.join(OBJ_DIR, "%s.%s.%s.o" % (tag, os.path.splitext(os.path.basename(src))[0], stamp))
        objs.append(obj)
        if force or not os.path.exists(obj) or os.path.getmtime(obj) < os.path.getmtime(src):
            jobs.append((src, obj))
    if not jobs and os.path.exists(lib_path) and all(os.path.getmtime(lib_path) >= os.path.getmtime(o) for o in objs):
        return lib_path
    with concurrent.futures.ThreadPoolExecutor(max_workers=min(8, max(1, len(jobs)))) as pool:
        logs = list(pool.map(lambda j: _compile_one(nvcc, j[0], j[1], extra, verbose), jobs))
    if verbose:
        sys.stderr.write("".join(logs))
    # objects of earlier header / flag states are no longer reachable: drop them
    for old in glob.glob(os.path.join(OBJ_DIR, tag + ".*.o")):
        if old not in objs:
            os.remove(old)
    tmp = lib_path + ".tmp.%d" % os.getpid()
    subprocess.check_call([nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp, *objs])
    os.replace(tmp, lib_path)
    return lib_path


if __name__ == "__main__":
    print(build(force="-f" in sys.argv or "-v" in sys.argv, verbose="-v" in sys.argv))
