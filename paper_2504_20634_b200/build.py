"""Build libfbsr.so in-tree with nvcc for sm_100a.

    python -m paper_2504_20634_b200.build [--force] [--verbose]

The kernel templates are instantiated once per (target format, operation group),
one translation unit per format and group compiled in parallel, then linked with the entry points
into ``paper_2504_20634_b200/libfbsr.so``.  Works without a GPU (cross-compile).
"""
import concurrent.futures
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libfbsr.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
         "-Xcompiler", "-fPIC", "-Xcompiler", "-O2", "--fmad=false"]
HEADERS = ["fbsr_device.cuh", "fbsr_kernels.cuh", "fbsr_internal.h", os.path.join("..", "..", "include", "fbsr.h")]


def _units():
    units = [("fbsr_api.o", "fbsr_api.cu", []), ("fbsr_descriptor.o", "fbsr_descriptor.cu", [])]
    for group in (2, 6, 5, 3, 1, 0, 4):       # the longest compilations first
        for fmt in range(5):
            if group in (2, 3, 6) and fmt < 2:
                continue                      # 16-bit sources and the Algorithm-1 steps go to the 8-bit targets only
            units.append(("fbsr_dispatch_f%d_g%d.o" % (fmt, group), "fbsr_dispatch.cu",
                          ["-DFBSR_FMT=%d" % fmt, "-DFBSR_GROUP=%d" % group]))
    return units


def _newest_source():
    paths = [os.path.join(CSRC, h) for h in HEADERS] + [os.path.join(CSRC, "fbsr_api.cu"),
                                                        os.path.join(CSRC, "fbsr_dispatch.cu"),
                                                        os.path.join(CSRC, "fbsr_descriptor.cu"), __file__]
    return max(os.path.getmtime(p) for p in paths)


def _compile(unit, verbose, force=False):
    obj, src, defs = unit
    # an object newer than the headers, its own source and this file is kept
    deps = [os.path.join(CSRC, h) for h in HEADERS] + [os.path.join(CSRC, src), __file__]
    out = os.path.join(OBJ, obj)
    if not force and not verbose and os.path.exists(out) and os.path.getmtime(out) >= max(os.path.getmtime(d) for d in deps):
        return obj, ""
    cmd = [NVCC, *FLAGS, *(["-Xptxas", "-v"] if verbose else []), *defs, "-c", os.path.join(CSRC, src),
           "-o", os.path.join(OBJ, obj)]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed for %s:\n%s\n%s" % (obj, res.stdout, res.stderr))
    return obj, res.stderr


def build(force=False, verbose=False):
    """Compile (if stale) and return the path of libfbsr.so."""
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= _newest_source():
        return LIB
    os.makedirs(OBJ, exist_ok=True)
    units = _units()
    with concurrent.futures.ThreadPoolExecutor(max_workers=min(len(units), os.cpu_count() or 4)) as pool:
        for obj, log in pool.map(lambda u: _compile(u, verbose, force), units):
            if verbose:
                with open(os.path.join(OBJ, obj + ".ptxas.txt"), "w") as fh:
                    fh.write(log)
    tmp = LIB + ".tmp.%d" % os.getpid()
    cmd = [NVCC, "-shared", "-o", tmp, *[os.path.join(OBJ, u[0]) for u in units], "-lcudart"]
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
