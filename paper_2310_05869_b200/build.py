"""Builds the C-ABI library (libhyperattn.so) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.path.join(PKG_DIR, "libhyperattn.so")
SOURCES = ["api.cu", "hash.cu", "sort.cu", "attn_mma.cu", "attn_tc.cu", "merge.cu", "noalloc.cu", "backward.cu", "caps.cu", "alpha.cu", "vnorm.cu"]
NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    raise RuntimeError("nvcc not found")


def needs_build() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(PKG_DIR, "..", "include", "hyperattn.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB_PATH
    objs = []
    procs = []
    for src in SOURCES:
        obj = os.path.join(CSRC, src.replace(".cu", ".o"))
        cmd = [_nvcc(), *NVCC_FLAGS, "-c", os.path.join(CSRC, src), "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    failed = False
    for src, pr in procs:
        out, _ = pr.communicate()
        if verbose or pr.returncode:
            sys.stderr.write(f"--- {src}\n{out}\n")
        failed |= pr.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    subprocess.check_call([_nvcc(), "-shared", "-o", LIB_PATH, *objs, "-lcudart"])
    return LIB_PATH


WAIT_TEST_LIB = os.path.join(PKG_DIR, "libhyperattn_waittest.so")


def build_wait_test_library(force: bool = False) -> str:
    """A second copy of the library for ONE test (tests/test_gpu_wait_limit.py): the attention kernel compiled with
    a 20 ms limit on its waits and a switch that makes one K / V tile never arrive, once, so that the path on which
    a wait gives up (status word, draining, TMEM release) can be run.  Never loaded by the package itself."""
    if not force and os.path.exists(WAIT_TEST_LIB) and os.path.getmtime(WAIT_TEST_LIB) >= os.path.getmtime(build_library()):
        return WAIT_TEST_LIB
    build_library()
    obj = os.path.join(CSRC, "attn_tc_waittest.o")
    subprocess.check_call([_nvcc(), *NVCC_FLAGS, "-DHA_WAIT_LIMIT_NS=20000000ull", "-DHA_TEST_DROP_ARRIVAL", "-c",
                           os.path.join(CSRC, "attn_tc.cu"), "-o", obj])
    objs = [os.path.join(CSRC, src.replace(".cu", ".o")) for src in SOURCES if src != "attn_tc.cu"] + [obj]
    subprocess.check_call([_nvcc(), "-shared", "-o", WAIT_TEST_LIB, *objs, "-lcudart"])
    return WAIT_TEST_LIB


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv))
    print(build_wait_test_library(force="--force" in sys.argv))
