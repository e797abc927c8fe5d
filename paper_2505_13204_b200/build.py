"""Builds ``libaasd.so`` (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

The streaming kernels are compiled once per logits dtype in translation units of their own
(``-DAASD_DT=0`` fp32, ``-DAASD_DT=1`` bf16), in parallel, then linked with the host side.
``build(check=True)`` builds ``libaasd_check.so`` instead: the same sources with
``-DAASD_BOUNDS_CHECK``, in which the kernels range-check the indices they compute and
report a violation in the status word (a debugging build; the tests run it on small cases).
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libaasd.so")
LIB_CHECK = os.path.join(HERE, "libaasd_check.so")
OBJ_DIR = os.path.join(HERE, "_build")
# (source, object tag, extra defines)
UNITS = [("aasd.cu", "host", [])] + [
    (src, "%s_dt%d" % (src[:-3], dt), ["-DAASD_DT=%d" % dt])
    for src in ("aasd_verify.cu", "aasd_align.cu", "aasd_align_gumbel.cu", "aasd_tree.cu") for dt in (1, 0)]
DEPENDS = ["aasd.cu", "aasd_verify.cu", "aasd_align.cu", "aasd_align_gumbel.cu", "aasd_tree.cu", "aasd_host.h",
           "aasd_device.cuh", "aasd_rows.cuh", "aasd_sampler.cuh", "aasd_stream.cuh", "aasd_tokens.cuh",
           "aasd_tree.cuh", os.path.join("..", "..", "include", "aasd.h")]
# -fno-gnu-unique / -Bsymbolic: two builds of the library (the normal and the checked one) can
# live in one process without sharing function-local statics or binding to each other's symbols
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-fno-gnu-unique"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def up_to_date(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return False
    t = os.path.getmtime(lib)
    return all(os.path.getmtime(os.path.join(CSRC, d)) <= t for d in DEPENDS)


def build(force: bool = False, verbose: bool = False, check: bool = False) -> str:
    lib = LIB_CHECK if check else LIB
    if not force and up_to_date(lib):
        return lib
    tag = "check" if check else "rel"
    os.makedirs(OBJ_DIR, exist_ok=True)
    extra = (["-DAASD_BOUNDS_CHECK"] if check else []) + (["-Xptxas", "-v"] if verbose else [])

    def compile_unit(unit):
        src, name, defs = unit
        obj = os.path.join(OBJ_DIR, "%s_%s_%d.o" % (name, tag, os.getpid()))
        cmd = [_nvcc()] + NVCC_FLAGS + extra + defs + ["-c", os.path.join(CSRC, src), "-o", obj]
        r = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
        return obj, r.returncode, r.stdout, " ".join(cmd)

    with ThreadPoolExecutor(max_workers=min(len(UNITS), os.cpu_count() or 1)) as ex:
        results = list(ex.map(compile_unit, UNITS))
    objs = []
    for obj, rc, out, cmd in results:
        if verbose or rc != 0:
            sys.stderr.write(out)
        if rc != 0:
            raise subprocess.CalledProcessError(rc, cmd)
        objs.append(obj)
    tmp = lib + ".tmp.%d" % os.getpid()
    subprocess.check_call([_nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-Xlinker", "-Bsymbolic"]
                          + objs + ["-o", tmp])
    os.replace(tmp, lib)
    for obj in objs:
        os.unlink(obj)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, check="--check" in sys.argv))
