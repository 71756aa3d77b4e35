"""Builds the CUDA library in-tree with nvcc for sm_100a (cross-compiles without a GPU).

    python -m paper_2401_10774_b200.build [--force] [--verbose] [--timing-aids] [--debug-checks]

--timing-aids compiles with -DMEDUSA_TIMING_AIDS: only such a build reads the MEDUSA_* environment switches used
for comparison runs (ring depth, serialised launches, dropped kernel classes); the default build reads none.
--debug-checks builds a second library, libmedusa_b200_checked.so (-DMEDUSA_DEBUG_CHECKS): after the stages of a step it
launches small kernels that test what the stage produced (finite logits, token / node / row indices in range, the cache
length inside the cache) and record MEDUSA_ERR_NONFINITE or MEDUSA_ERR_BOUNDS in the device status word.  Nothing
traps and nothing is skipped; the default library contains none of these launches.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG, "csrc")
OBJ = os.path.join(PKG, "build")
LIB = os.path.join(PKG, "libmedusa_b200.so")
LIB_CHECKED = os.path.join(PKG, "libmedusa_b200_checked.so")
SOURCES = ["api.cu", "gemm_tc.cu", "simt_kernels.cu", "attention.cu", "attention_flash.cu", "attention_tc.cu", "heads.cu", "posterior.cu", "train_heads.cu", "tree_host.cpp"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr"]


def _nvcc() -> str:
    for p in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if p and (os.path.sep not in p or os.path.exists(p)):
            return p
    raise RuntimeError("nvcc not found")


def _newest_header() -> float:
    t = 0.0
    for d in (CSRC, os.path.join(os.path.dirname(PKG), "include")):
        for f in os.listdir(d):
            if f.endswith((".h", ".cuh")):
                t = max(t, os.path.getmtime(os.path.join(d, f)))
    return t


def build_library(force: bool = False, verbose: bool = False, timing_aids: bool = False, debug_checks: bool = False) -> str:
    obj_dir = OBJ + ("_checked" if debug_checks else "")
    lib_path = LIB_CHECKED if debug_checks else LIB
    os.makedirs(obj_dir, exist_ok=True)
    nvcc = _nvcc()
    # a change of flavour rebuilds everything
    stamp = os.path.join(obj_dir, "flavour")
    flavour = ("timing-aids" if timing_aids else "default") + ("+checks" if debug_checks else "")
    if not os.path.exists(stamp) or open(stamp).read() != flavour:
        force = True
    extra = (["-DMEDUSA_TIMING_AIDS"] if timing_aids else []) + (["-DMEDUSA_DEBUG_CHECKS"] if debug_checks else [])
    hdr = _newest_header()
    jobs = []
    objs = []
    for src in SOURCES:
        s = os.path.join(CSRC, src)
        o = os.path.join(obj_dir, os.path.splitext(src)[0] + ".o")
        objs.append(o)
        if force or not os.path.exists(o) or os.path.getmtime(o) < max(os.path.getmtime(s), hdr):
            cmd = [nvcc] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-x", "cu", "-c", s, "-o", o]
            jobs.append(cmd)

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or r.returncode:
            sys.stderr.write(" ".join(cmd) + "\n" + r.stdout + r.stderr)
        if r.returncode:
            raise RuntimeError("nvcc failed: " + " ".join(cmd))

    with ThreadPoolExecutor(max_workers=4) as ex:
        list(ex.map(run, jobs))
    if jobs or not os.path.exists(lib_path):
        tmp = lib_path + ".%d.tmp" % os.getpid()
        run([nvcc, "-shared", "-o", tmp] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"])
        os.replace(tmp, lib_path)
    with open(stamp, "w") as f:
        f.write(flavour)
    return lib_path


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="--verbose" in sys.argv, timing_aids="--timing-aids" in sys.argv,
                        debug_checks="--debug-checks" in sys.argv))
