"""Builds liboq.so (C-ABI library, sm_100a only) in-tree with nvcc.

    python -m paper_2607_02461_b200.build [--verbose]

Every source is compiled to an object file of its own (in parallel, only when it or a header is newer), then linked.
OQ_NVCC_FLAGS in the environment adds compiler flags (e.g. -DOQ_RQMM_TIMING for the instrumented kernel).
"""
import os
import shlex
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "liboq.so")
SOURCES = ["oq_host.cu", "oq_rotate_quantize.cu", "oq_rq_mm.cu", "oq_qlinear.cu", "oq_forward_host.cu", "oq_noalloc.cu",
           "oq_adaln.cu", "oq_block.cu"]
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC"]


def _extra():
    return shlex.split(os.environ.get("OQ_NVCC_FLAGS", ""))


def _headers():
    return [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))] + \
           [os.path.join(HERE, "..", "include", "oq.h"), __file__]


def _stamp():
    return LIB + ".flags"          # the flags liboq.so was built with (travels with it)


def _stale(target, deps):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(p) > t for p in deps)


def build(force=False, verbose=False):
    """Compile every CUDA source into paper_2607_02461_b200/liboq.so; returns the path."""
    flags = " ".join(FLAGS + _extra())
    if not os.path.exists(_stamp()) or open(_stamp()).read() != flags:
        force = True
    srcs = [s for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]
    hdrs = _headers()
    if not force and not _stale(LIB, [os.path.join(CSRC, s) for s in srcs] + hdrs):
        return LIB                 # up to date (the object files need not exist: they do not travel with the library)
    os.makedirs(OBJ, exist_ok=True)
    if not os.path.exists(os.path.join(OBJ, "flags.txt")) or open(os.path.join(OBJ, "flags.txt")).read() != flags:
        force = True               # objects built with other flags
    jobs = []
    for s in srcs:
        src, obj = os.path.join(CSRC, s), os.path.join(OBJ, s[:-3] + ".o")
        if force or _stale(obj, [src] + hdrs):
            jobs.append((src, obj))

    def compile_one(job):
        src, obj = job
        cmd = ["nvcc"] + FLAGS + _extra() + (["-Xptxas", "-v"] if verbose else []) + ["-c", src, "-o", obj]
        return subprocess.run(cmd, capture_output=True, text=True)

    with ThreadPoolExecutor(max_workers=max(1, min(len(jobs), os.cpu_count() or 1))) as pool:
        results = list(pool.map(compile_one, jobs))
    failed = False
    for res in results:
        if verbose or res.returncode:
            sys.stderr.write(res.stdout + res.stderr)
        failed = failed or res.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed building liboq.so")
    objs = [os.path.join(OBJ, s[:-3] + ".o") for s in srcs]
    res = subprocess.run(["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-cudart", "static", "-o", LIB] + objs,
                         capture_output=True, text=True)
    if verbose or res.returncode:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode:
        raise RuntimeError("nvcc failed linking liboq.so")
    open(_stamp(), "w").write(flags)
    open(os.path.join(OBJ, "flags.txt"), "w").write(flags)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
