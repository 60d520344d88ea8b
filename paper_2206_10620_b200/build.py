"""Build libpatconv.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_HERE, "csrc")
_INC = os.path.join(os.path.dirname(_HERE), "include")
LIB_PATH = os.path.join(_HERE, "libpatconv.so")
_SOURCES = ["patconv.cu", "blockgemm.cu", "dwconv.cu", "probe.cu", "pack.cpp"]
_DEPS = _SOURCES + ["patconv_internal.h", "gen_core.py", "gen_blockgemm.py", os.path.join(_INC, "patconv.h"),
                    os.path.join(_INC, "blockgemm.h"), os.path.join(_INC, "dwconv.h")]


_OBJ_DIR = os.path.join(_HERE, "_build")
# what each source includes besides itself
_INCLUDES = {
    "patconv.cu": ["patconv_internal.h", "gen_core.py", os.path.join(_INC, "patconv.h")],
    "blockgemm.cu": ["patconv_internal.h", "gen_blockgemm.py", os.path.join(_INC, "patconv.h"),
                     os.path.join(_INC, "blockgemm.h")],
    "dwconv.cu": ["patconv_internal.h", os.path.join(_INC, "patconv.h"), os.path.join(_INC, "dwconv.h")],
    "probe.cu": [os.path.join(_INC, "patconv.h")],
    "pack.cpp": ["patconv_internal.h", os.path.join(_INC, "patconv.h")],
}


def _mtime(name: str) -> float:
    return os.path.getmtime(os.path.join(_CSRC, name))


def _stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    return any(_mtime(d) > t for d in _DEPS)


def build(force: bool = False, verbose: bool = False) -> str:
    """Generate the per-pattern code, compile every source that changed to an object of its
    own, and link the shared library."""
    if not force and not _stale():
        return LIB_PATH
    gen = os.path.join(_CSRC, "core_gen.inc")
    subprocess.check_call([sys.executable, os.path.join(_CSRC, "gen_core.py"), gen])
    subprocess.check_call([sys.executable, os.path.join(_CSRC, "gen_blockgemm.py"),
                           os.path.join(_CSRC, "blockgemm_core.inc")])
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(_OBJ_DIR, exist_ok=True)
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
             "-Xcompiler", "-fPIC", "-I", _INC, "-I", _CSRC]
    if verbose:
        flags += ["-Xptxas", "-v"]
    objs, jobs = [], []
    for src in _SOURCES:
        obj = os.path.join(_OBJ_DIR, os.path.splitext(src)[0] + ".o")
        objs.append(obj)
        newest = max([_mtime(src)] + [_mtime(d) for d in _INCLUDES[src]])
        if force or verbose or not os.path.exists(obj) or os.path.getmtime(obj) < newest:
            jobs.append((obj, subprocess.Popen([nvcc] + flags + ["-c", os.path.join(_CSRC, src), "-o", obj + ".tmp"])))
    for obj, job in jobs:                       # the compilations run side by side
        if job.wait() != 0:
            raise subprocess.CalledProcessError(job.returncode, "nvcc -c (%s)" % obj)
        os.replace(obj + ".tmp", obj)
    tmp = LIB_PATH + ".tmp%d" % os.getpid()
    subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", tmp] + objs)
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
