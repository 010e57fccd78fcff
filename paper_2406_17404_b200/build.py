"""Builds libtrj.so (sm_100a only) next to this file with plain nvcc; no torch headers involved."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libtrj.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: libtrj cannot be built")


def sources():
    return sorted(f for f in os.listdir(CSRC) if f.endswith((".cu", ".cpp")))


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(verbose: bool = False, force: bool = False, timeline: bool = False, debug: bool = False) -> str:
    """Compile every source under csrc/ and link libtrj.so; returns its path.  ``timeline=True`` builds a second
    library, libtrj_timeline.so, with -DTRJ_TIMELINE (clock stamps in the per-layer kernels; measurement only);
    ``debug=True`` builds libtrj_debug.so with -DTRJ_DEBUG (index checks in the kernels that address the cache)."""
    global OBJ, LIB
    if timeline or debug:
        tag = "timeline" if timeline else "debug"
        saved = OBJ, LIB, list(NVCC_FLAGS)
        OBJ, LIB = os.path.join(HERE, "_build_" + tag), os.path.join(HERE, "libtrj_%s.so" % tag)
        NVCC_FLAGS.append("-DTRJ_TIMELINE" if timeline else "-DTRJ_DEBUG")
        try:
            return build(verbose, force)
        finally:
            OBJ, LIB = saved[0], saved[1]
            NVCC_FLAGS[:] = saved[2]
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    headers.append(os.path.join(ROOT, "include", "trj.h"))
    if not force and not verbose and not _stale(LIB, [os.path.join(CSRC, s) for s in sources()] + headers):
        return LIB                      # the library is newer than every source: nothing to do
    nvcc = _nvcc()
    os.makedirs(OBJ, exist_ok=True)
    objs, procs = [], []
    for src in sources():
        path = os.path.join(CSRC, src)
        obj = os.path.join(OBJ, os.path.splitext(src)[0] + ".o")
        objs.append(obj)
        if force or _stale(obj, [path] + headers):
            cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-x", "cu", "-c", path, "-o", obj]
            procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    failed = []
    for src, p in procs:
        out, _ = p.communicate()
        if verbose or p.returncode != 0:
            sys.stderr.write(f"--- {src}\n{out}\n")
        if p.returncode != 0:
            failed.append(src)
    if failed:
        raise RuntimeError("nvcc failed for: " + ", ".join(failed))
    if force or procs or _stale(LIB, objs):
        cmd = [nvcc, "-shared", "-o", LIB] + objs + ["-gencode", "arch=compute_100a,code=sm_100a", "-lcudart"]
        r = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
        if r.returncode != 0:
            raise RuntimeError("link failed:\n" + r.stdout)
    return LIB


if __name__ == "__main__":
    print(build(verbose="-v" in sys.argv, force="-f" in sys.argv, timeline="--timeline" in sys.argv,
                debug="--debug" in sys.argv))
