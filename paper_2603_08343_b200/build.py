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


# only the C ABI file looks at WHT_DEBUG: the debug library links the regular family objects
DEBUG_SOURCES = ("wht_affine.cu",)
LIB_DEBUG_PATH = os.path.join(HERE, "libwht_affine_debug.so")


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compile what is missing or older than its sources; return the library's path.

    `verbose` adds -Xptxas -v (registers, spills and shared memory of every kernel, on stderr) and
    rebuilds everything.  `debug` builds libwht_affine_debug.so instead: the same kernels with the C ABI
    compiled with -DWHT_DEBUG (guard regions around every output and scratch buffer, see the header).
    """
    force = force or verbose
    lib = LIB_DEBUG_PATH if debug else LIB_PATH
    sources = [os.path.join(CSRC, s) for s in SOURCES]
    if not force and os.path.exists(lib) and \
            os.path.getmtime(lib) >= max(_newest_dependency_mtime(p) for p in sources):
        return lib  # up to date, whether or not the objects are still around
    os.makedirs(OBJ_DIR, exist_ok=True)
    nvcc = _nvcc()
    jobs, objs = [], []
    for src in SOURCES:
        path = os.path.join(CSRC, src)
        special = debug and src in DEBUG_SOURCES
        obj = os.path.join(OBJ_DIR, src[:-3] + ("_debug.o" if special else ".o"))
        objs.append(obj)
        stale = force or not os.path.exists(obj) or os.path.getmtime(obj) < _newest_dependency_mtime(path)
        if stale:
            cmd = [nvcc, "-std=c++17", "-O3", "-lineinfo", *ARCH, "-Xcompiler", "-fPIC", "-c", path, "-o", obj]
            if special:
                cmd.append("-DWHT_DEBUG")
            if verbose:
                cmd.insert(1, "-Xptxas=-v")
            jobs.append(cmd)
    if not jobs and os.path.exists(lib) and os.path.getmtime(lib) >= max(os.path.getmtime(o) for o in objs):
        return lib
    with ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 4) or 1) as pool:
        logs = list(pool.map(_run, jobs))
    if verbose:
        sys.stderr.write("".join(logs))
    _run([nvcc, *ARCH, "-Xcompiler", "-fPIC", "-shared", "-o", lib, *objs])
    return lib


def ptxas_summary() -> str:
    """Rebuilds everything with -Xptxas -v and returns one line per kernel: registers per thread, spill
    bytes, static shared memory (what the compiler reports; nothing is disassembled)."""
    import io
    from contextlib import redirect_stderr
    buf = io.StringIO()
    with redirect_stderr(buf):
        build(verbose=True)
    text = buf.getvalue()
    try:
        demangled = subprocess.run(["c++filt"], input=text, capture_output=True, text=True).stdout or text
    except OSError:
        demangled = text
    rows, name, spill = [], None, (0, 0)
    for line in demangled.splitlines():
        m = re.search(r"Compiling entry function '(.+)' for", line)
        if m:
            name = m.group(1)
            continue
        m = re.search(r"(\d+) bytes stack frame, (\d+) bytes spill stores, (\d+) bytes spill loads", line)
        if m:
            spill = (int(m.group(2)), int(m.group(3)))
            continue
        m = re.search(r"Used (\d+) registers", line)
        if m and name:
            smem = re.search(r"(\d+) bytes smem", line)
            short = re.sub(r"\(.*$", "", name).replace("void ", "").replace("wht::", "")
            rows.append((short, int(m.group(1)), spill[0], spill[1], int(smem.group(1)) if smem else 0))
            name, spill = None, (0, 0)
    rows.sort()
    out = ["kernel | registers/thread | spill stores B | spill loads B | static smem B",
           "---|---|---|---|---"]
    out += [f"{n} | {r} | {ss} | {sl} | {sm}" for n, r, ss, sl, sm in rows]
    worst = [r for r in rows if r[2] or r[3]]
    out.append("")
    out.append(f"{len(rows)} kernels; with spills: " + (", ".join(f"{n} ({ss}/{sl} B)" for n, _, ss, sl, _ in worst) or "none"))
    return "\n".join(out)


if __name__ == "__main__":
    if "--ptxas-summary" in sys.argv:
        print(ptxas_summary())
    elif "--digest" in sys.argv:  # python -m paper_2603_08343_b200.build --digest a.cuh,b.cu
        print(source_digest(sys.argv[sys.argv.index("--digest") + 1].split(",")))
    else:
        print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
