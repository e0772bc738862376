"""Build step: compiles the CUDA sources in ``csrc/`` into ``libsa.so`` next to this file.

nvcc cross-compiles for sm_100a without a GPU.  Every ``.cu`` file is compiled to an object of its
own (in parallel, under ``build/``) and re-compiled only when it, a header or the flags changed;
the objects are then linked into the shared object.
``python -m paper_2609_09208_b200.build [--force] [--verbose] [-DNAME[=VALUE] ...]``.
"""
from __future__ import annotations

import glob
import hashlib
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libsa.so")
OBJ_DIR = os.path.join(_HERE, "build")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--fmad=true",            # contraction is harmless where it is allowed; exact steps use __f*_rn intrinsics
    "-Xcompiler", "-fPIC",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _headers():
    return sorted(glob.glob(os.path.join(CSRC, "*.cuh"))) + [os.path.join(_HERE, "..", "include", "sa.h")]


def _nvcc() -> str:
    return os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")


def _tag(defines) -> str:
    return hashlib.sha1(" ".join(NVCC_FLAGS + list(defines)).encode()).hexdigest()[:10]


def _compile_one(src, obj, defines, verbose):
    tmp = obj + ".%d.tmp" % os.getpid()
    cmd = [_nvcc()] + NVCC_FLAGS + list(defines) + (["-Xptxas", "-v"] if verbose else []) + ["-c", "-o", tmp, src]
    subprocess.check_call(cmd)
    os.replace(tmp, obj)


def build(force: bool = False, verbose: bool = False, defines=(), out: str = LIB) -> str:
    """Compile what is stale and link ``out``.  ``defines``: extra ``-D...`` flags (a distinct object cache per set)."""
    tag = _tag(defines)
    stamp = os.path.join(OBJ_DIR, os.path.basename(out) + ".tag")      # which object set the library was linked from
    linked = open(stamp).read() if os.path.exists(stamp) else None
    hdr_time = max(os.path.getmtime(h) for h in _headers())
    src_time = max(hdr_time, max(os.path.getmtime(s) for s in sources()))
    if not force and os.path.exists(out) and os.path.getmtime(out) >= src_time and linked in (tag, None if not defines else tag):
        return out                                  # up to date (a library shipped without its objects is trusted by its date)
    os.makedirs(OBJ_DIR, exist_ok=True)
    jobs, objs = [], []
    for src in sources():
        obj = os.path.join(OBJ_DIR, "%s.%s.o" % (os.path.splitext(os.path.basename(src))[0], tag))
        objs.append(obj)
        if force or not os.path.exists(obj) or os.path.getmtime(obj) < max(hdr_time, os.path.getmtime(src)):
            jobs.append((src, obj))
    if jobs:
        with ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 1)) as ex:
            for f in [ex.submit(_compile_one, s, o, defines, verbose) for s, o in jobs]:
                f.result()
    if jobs or linked != tag or not os.path.exists(out) or any(os.path.getmtime(o) > os.path.getmtime(out) for o in objs):
        tmp = out + ".%d.tmp" % os.getpid()
        subprocess.check_call([_nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp] + objs)
        os.replace(tmp, out)
        with open(stamp, "w") as f:
            f.write(tag)
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv,
                defines=[a for a in sys.argv[1:] if a.startswith("-D")]))
