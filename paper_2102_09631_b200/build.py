"""Build libdad.so (the CUDA library behind the C ABI of include/dad.h) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libdad.so")

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "-Xcompiler", "-fPIC", "-Xptxas", "-v", "--expt-relaxed-constexpr",
]
OBJ_DIR = os.path.join(HERE, "_build")


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _headers():
    return glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(p) > t for p in sources() + _headers())


CHECK_LIB = os.path.join(HERE, "libdad_check.so")
CHECK_FLAGS = ["-DDAD_BOUNDS_CHECK", "-rdc=true"]


def build_check(force: bool = False, verbose: bool = False) -> str:
    """The bounds-check build of the same sources (libdad_check.so, see csrc/bounds.cuh): load it with DAD_LIB."""
    return build(force=force, verbose=verbose, lib=CHECK_LIB, extra=CHECK_FLAGS)


def build(force: bool = False, verbose: bool = False, lib: str = LIB, extra=None) -> str:
    """Compile every .cu under csrc/ (one object each, in parallel; an object is reused while it is newer than
    its source and every header) and link them into libdad.so; returns its path.  Raises if nvcc fails."""
    LIB = lib
    if not force and not _stale(LIB):
        return LIB
    from concurrent.futures import ThreadPoolExecutor
    nvcc = os.environ.get("NVCC", "nvcc")
    os.makedirs(OBJ_DIR, exist_ok=True)
    extra = list(extra or []) + os.environ.get("DAD_NVCC_EXTRA", "").split()
    tag = ("-" + "".join(c if c.isalnum() else "_" for c in " ".join(extra))) if extra else ""
    hdr_t = max(os.path.getmtime(p) for p in _headers())
    log_lines, failed = [], []

    def compile_one(src):
        obj = os.path.join(OBJ_DIR, os.path.basename(src)[:-3] + tag + ".o")
        if not force and os.path.exists(obj) and os.path.getmtime(obj) > max(os.path.getmtime(src), hdr_t):
            return obj, "", 0
        cmd = [nvcc] + NVCC_FLAGS + extra + ["-I", os.path.join(ROOT, "include"), "-I", CSRC, "-c", "-o", obj, src]
        res = subprocess.run(cmd, capture_output=True, text=True)
        return obj, " ".join(cmd) + "\n" + res.stdout + res.stderr, res.returncode

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        results = list(pool.map(compile_one, sources()))
    objs = []
    for obj, text, rc in results:
        objs.append(obj)
        log_lines.append(text)
        if rc != 0:
            failed.append(obj)
    tmp = LIB + f".tmp{os.getpid()}"
    if not failed:
        cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a"] + [x for x in extra if x.startswith("-rdc")] + ["-shared", "-o", tmp] + objs
        res = subprocess.run(cmd, capture_output=True, text=True)
        log_lines.append(" ".join(cmd) + "\n" + res.stdout + res.stderr)
        if res.returncode != 0:
            failed.append(tmp)
    log = os.path.join(HERE, "build.log")
    with open(log, "w") as f:
        f.write("\n".join(log_lines))
    if verbose or failed:
        sys.stderr.write("\n".join(log_lines))
    if failed:
        raise RuntimeError(f"nvcc failed (see {log})")
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    if "--check" in sys.argv:
        print(build_check(force="--force" in sys.argv, verbose="-v" in sys.argv))
    else:
        print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
