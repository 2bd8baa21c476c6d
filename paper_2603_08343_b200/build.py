"""Builds csrc/ into libwht_affine.so (sm_100a) next to this file, with nvcc.

One object per translation unit (the C ABI and one file per kernel family), compiled in parallel
into `_build/`, then linked; an object is rebuilt only when its source or a header it includes is newer than it.
"""
from __future__ import annotations

import os
import re
import shutil
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ_DIR = os.path.join(HERE, "_build")
LIB_PATH = os.path.join(HERE, "libwht_affine.so")
SOURCES = ["wht_affine.cu", "family_misc.cu", "family_bfly_fwd.cu", "family_bfly_bwd.cu", "family_tp.cu",
           "family_mma.cu", "family_umma_fwd.cu", "family_umma_bwd.cu", "family_umma_tp.cu"]
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found; set NVCC or install the CUDA toolkit")


_INCLUDE = re.compile(r'^\s*#include\s+"([^"]+)"', re.M)


def _newest_dependency_mtime(path: str, seen=None) -> float:
    """mtime of the newest file among `path` and the files it includes with quotes, recursively."""
    seen = set() if seen is None else seen
    path = os.path.normpath(path)
    if path in seen or not os.path.exists(path):
        return 0.0
    seen.add(path)
    newest = os.path.getmtime(path)
    with open(path) as f:
        for inc in _INCLUDE.findall(f.read()):
            newest = max(newest, _newest_dependency_mtime(os.path.join(os.path.dirname(path), inc), seen))
    return newest


def source_digest(names) -> str:
    """sha256 over the named files of csrc/ (in the order given): ties a recorded measurement to the
    sources of the kernel it was taken on."""
    import hashlib
    h = hashlib.sha256()
    for name in names:
        with open(os.path.join(CSRC, name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def _run(cmd):
    proc = subprocess.run(cmd, capture_output=True, text=True)
    if proc.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + " ".join(cmd) + "\n" + proc.stdout + proc.stderr)
    return proc.stderr


def build(force: bool = False, verbose: bool = False, defines: tuple = ()) -> str:
    """Compile what is missing or older than its sources; return the library's path.

    `verbose` adds -Xptxas -v (registers, spills and shared memory of every kernel, on stderr);
    `defines` are extra -D flags (a debug build); both rebuild everything.
    """
    force = force or verbose or bool(defines)
    sources = [os.path.join(CSRC, s) for s in SOURCES]
    if not force and os.path.exists(LIB_PATH) and \
            os.path.getmtime(LIB_PATH) >= max(_newest_dependency_mtime(p) for p in sources):
        return LIB_PATH  # up to date, whether or not the objects are still around
    os.makedirs(OBJ_DIR, exist_ok=True)
    nvcc = _nvcc()
    jobs = []
    for src in SOURCES:
        path = os.path.join(CSRC, src)
        obj = os.path.join(OBJ_DIR, src[:-3] + ".o")
        stale = force or not os.path.exists(obj) or os.path.getmtime(obj) < _newest_dependency_mtime(path)
        if stale:
            cmd = [nvcc, "-std=c++17", "-O3", "-lineinfo", *ARCH, "-Xcompiler", "-fPIC", "-c", path, "-o", obj]
            cmd += [f"-D{d}" for d in defines]
            if verbose:
                cmd.insert(1, "-Xptxas=-v")
            jobs.append(cmd)
    objs = [os.path.join(OBJ_DIR, s[:-3] + ".o") for s in SOURCES]
    if not jobs and os.path.exists(LIB_PATH) and os.path.getmtime(LIB_PATH) >= max(os.path.getmtime(o) for o in objs):
        return LIB_PATH
    with ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 4) or 1) as pool:
        logs = list(pool.map(_run, jobs))
    if verbose:
        sys.stderr.write("".join(logs))
    _run([nvcc, *ARCH, "-Xcompiler", "-fPIC", "-shared", "-o", LIB_PATH, *objs])
    if defines:  # a special build must not pass for the regular one on the next call
        for o in objs:
            os.utime(o, (0, 0))
    return LIB_PATH


if __name__ == "__main__":
    if "--digest" in sys.argv:  # python -m paper_2603_08343_b200.build --digest a.cuh,b.cu
        print(source_digest(sys.argv[sys.argv.index("--digest") + 1].split(",")))
    else:
        print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
