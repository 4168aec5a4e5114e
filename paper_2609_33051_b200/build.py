"""Build libsketchssm.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG_DIR)
CSRC = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.path.join(PKG_DIR, "libsketchssm.so")
# (source, object suffix, extra defines); the two-kernel decode is compiled once per (recurrence kind, I/O type)
UNITS = [("api.cu", "", []), ("decode.cu", "", []), ("update.cu", "", []), ("update_tc.cu", "", []),
         ("update_tc_ws.cu", "", []), ("update_tc_ws_gdn.cu", "", []), ("update_tc_ws_kda.cu", "", []), ("decode_static.cu", "", []), ("selftest.cu", "", []), ("coef_map.cu", "", []),
         *[("decode_split.cu", f"_k{k}_io{io}", [f"-DSKETCHSSM_GROUP_KIND={k}", f"-DSKETCHSSM_GROUP_IO={io}"])
           for k in range(3) for io in range(2)]]
HEADERS = [os.path.join(CSRC, "internal.cuh"), os.path.join(CSRC, "lanegroup.cuh"), os.path.join(CSRC, "tc_common.cuh"),
           os.path.join(ROOT, "include", "sketchssm.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found; cannot build libsketchssm.so")


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every .cu to an object (parallel-friendly, incremental) and link the shared library."""
    nvcc = _nvcc()
    objdir = os.path.join(PKG_DIR, "build")
    os.makedirs(objdir, exist_ok=True)
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
             "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if verbose:
        flags += ["-Xptxas", "-v"]
    procs, objs = [], []
    for src, suffix, defs in UNITS:
        sp = os.path.join(CSRC, src)
        obj = os.path.join(objdir, src.replace(".cu", suffix + ".o"))
        objs.append(obj)
        if force or _stale(obj, [sp] + HEADERS):
            procs.append((src + suffix, subprocess.Popen([nvcc, *flags, *defs, "-c", sp, "-o", obj],
                                                stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    for src, pr in procs:
        out, _ = pr.communicate()
        if verbose or pr.returncode != 0:
            sys.stderr.write(out)
        if pr.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}")
    if force or procs or _stale(LIB_PATH, objs):
        subprocess.check_call([nvcc, "-shared", "-o", LIB_PATH, *objs, "-gencode", "arch=compute_100a,code=sm_100a"])
    return LIB_PATH


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
