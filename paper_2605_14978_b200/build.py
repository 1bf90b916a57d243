"""Build ``libppow.so`` (sm_100a only) in-tree with nvcc.  ``python -m paper_2605_14978_b200.build``."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libppow.so")
LIB_CHECKED = os.path.join(HERE, "libppow_checked.so")   # the same sources with -DPPOW_CHECKED (bounds-checked build)
LIB_TIMELINE = os.path.join(HERE, "libppow_timeline.so")  # ... with -DPPOW_TIMELINE (per-warp timeline of the row kernel)
ROOT = os.path.dirname(HERE)


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps():
    return sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))


def is_stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(f) > t for f in _deps())


def build(force: bool = False, verbose: bool = False, checked: bool = False, timeline: bool = False) -> str:
    """Compile every .cu under csrc/ into one shared library for sm_100a.  ``checked``: the bounds-checked
    build (every kernel-computed index tested before use, failures counted and skipped, never trapped)."""
    lib = LIB_CHECKED if checked else LIB_TIMELINE if timeline else LIB
    if not force and not is_stale(lib):
        return lib
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = lib + ".tmp.%d" % os.getpid()
    cmd = [nvcc, "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "-Xcompiler", "-fPIC", "-shared", "-o", tmp] + (["-DPPOW_CHECKED"] if checked else ["-DPPOW_TIMELINE"] if timeline else []) + sources()
    if verbose:
        cmd[1:1] = ["-Xptxas", "-v"]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose:
        sys.stderr.write(res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stderr)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose=True))
    print(build(force=True, checked=True))
    print(build(force=True, timeline=True))
