"""Builds the CUDA library in-tree: csrc/*.cu -> libexcp.so (sm_100a only)."""
from __future__ import annotations

import hashlib
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libexcp.so")
SOURCES = ["stats.cu", "mask_compact.cu", "kmeans.cu", "pack.cu", "decode.cu", "excp_api.cu", "excp_noalloc.cu", "selftest.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-fmad=false", "-Xcompiler", "-fPIC", "-cudart", "static"]


def extra_flags() -> list[str]:
    """Extra nvcc flags from the environment (EXCP_NVCC_FLAGS), e.g. -DEXCP_DEBUG_BOUNDS for the build whose
    kernels check every index they form and report through the call's status instead of faulting."""
    return os.environ.get("EXCP_NVCC_FLAGS", "").split()


def lib_path() -> str:
    """libexcp.so for the plain build; a build with extra flags gets a name of its own (and its own objects), so
    that it never replaces the plain library."""
    flags = extra_flags()
    if not flags:
        return LIB
    return os.path.join(HERE, "libexcp-" + hashlib.sha1(" ".join(flags).encode()).hexdigest()[:8] + ".so")


def _stale(lib: str) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cu", ".cuh"))]
    deps.append(os.path.join(os.path.dirname(HERE), "include", "excp.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compiles the library if it is missing or older than its sources; returns its path."""
    lib = lib_path()
    if not force and not _stale(lib):
        return lib
    tag = os.path.basename(lib)[len("libexcp"):-len(".so")]        # "" or "-<hash>"
    nvcc = os.environ.get("NVCC", "nvcc")
    objs = []
    procs = []
    for src in SOURCES:
        obj = os.path.join(CSRC, src[:-3] + tag + ".o")
        cmd = [nvcc, *NVCC_FLAGS, *extra_flags(), "-c", os.path.join(CSRC, src), "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    failed = False
    for src, p in procs:
        out, _ = p.communicate()
        if p.returncode != 0 or verbose:
            sys.stderr.write(f"--- {src}\n{out}\n")
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    subprocess.check_call([nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-cudart", "static", "-o", lib, *objs, "-lrt", "-ldl", "-lpthread"])
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
