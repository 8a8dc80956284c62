"""Builds librouterelay.so (sm_100a only) next to this file with nvcc.

    python -m paper_2609_07306_b200.build [-v]
"""
from __future__ import annotations

import glob
import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "librouterelay.so")


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + \
        glob.glob(os.path.join(HERE, "..", "include", "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(verbose: bool = False, force: bool = False) -> str:
    """One nvcc process per source file (in parallel) into a scratch folder, then one link."""
    if not force and not is_stale():
        return LIB
    import tempfile
    from concurrent.futures import ThreadPoolExecutor
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
             "-Xcompiler", "-fPIC"] + os.environ.get("RR_EXTRA_NVCC_FLAGS", "").split()
    if verbose:
        flags += ["-Xptxas", "-v"]
    nvcc = _nvcc()
    with tempfile.TemporaryDirectory(prefix="rr_build_") as tmp:
        def compile_one(src):
            obj = os.path.join(tmp, os.path.basename(src)[:-3] + ".o")
            res = subprocess.run([nvcc] + flags + ["-c", src, "-o", obj], capture_output=True,
                                 text=True)
            return src, obj, res
        with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
            done = list(ex.map(compile_one, sources()))
        log = "".join(f"== {os.path.basename(s)}\n{r.stdout}{r.stderr}" for s, _, r in done)
        if any(r.returncode != 0 for _, _, r in done):
            raise RuntimeError("nvcc failed:\n" + log)
        res = subprocess.run([nvcc, "-shared", "-cudart", "static", "-gencode",
                              "arch=compute_100a,code=sm_100a", "-o", LIB] + [o for _, o, _ in done],
                             capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError("link failed:\n" + res.stdout + res.stderr)
    if verbose:
        print(log)
    return LIB


if __name__ == "__main__":
    build(verbose="-v" in sys.argv, force=True)
    print(LIB)
