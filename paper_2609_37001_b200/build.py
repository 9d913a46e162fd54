"""Builds libpsa.so (the C-ABI library) in-tree with nvcc for sm_100a.

    python -m paper_2609_37001_b200.build [--force] [--verbose] [--checked]

--checked builds libpsa_checked.so instead: the same library with -DPSA_DEBUG_CHECKS, in which the
attention kernel verifies every index, coordinate and slot it computes before using it and reports a
violation through the status word (PSA_ERR_INTERNAL) instead of touching memory.
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libpsa.so")
LIB_CHECKED = os.path.join(HERE, "libpsa_checked.so")
SOURCES = ["psa_host.cu", "psa_mask_build.cu", "psa_attn_sm100.cu", "psa_search.cu"]
HEADERS = [os.path.join(CSRC, "psa_common.cuh"), os.path.join(ROOT, "include", "psa.h")]


def _nvcc():
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def needs_build(lib=LIB):
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + HEADERS
    return any(os.path.getmtime(d) > t for d in deps)


def build(force=False, verbose=False, checked=False):
    lib = LIB_CHECKED if checked else LIB
    if not force and not needs_build(lib):
        return lib
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
           "-o", lib] + (["-DPSA_DEBUG_CHECKS"] if checked else []) + [os.path.join(CSRC, s) for s in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    r = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed building " + os.path.basename(lib))
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, checked="--checked" in sys.argv))
