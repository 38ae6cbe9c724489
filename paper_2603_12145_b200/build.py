"""Compile the CUDA libraries in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(HERE, "..", "include")
NVCC_FLAGS = ["-std=c++17", "-O3", "-lineinfo",
              "-gencode", "arch=compute_100a,code=sm_100a",
              "-Xcompiler", "-fPIC", "-shared", "--cudart=shared"]

# library -> (sources, other files it depends on)
TARGETS = {
    "libpong_b200.so": (["pong_api.cu", "pong_kernels.cu", "pong_noalloc.cu"],
                        ["pong_rules.cuh", "pong_kernels.cuh", os.path.join(INCLUDE, "pong.h")]),
    "libcartpole_b200.so": (["cartpole.cu"], [os.path.join(INCLUDE, "cartpole.h")]),
    "libgru_policy_b200.so": (["gru_policy.cu"], [os.path.join(INCLUDE, "gru_policy.h")]),
}
LIB = os.path.join(HERE, "libpong_b200.so")
CARTPOLE_LIB = os.path.join(HERE, "libcartpole_b200.so")
GRU_POLICY_LIB = os.path.join(HERE, "libgru_policy_b200.so")


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def _paths(name):
    sources, deps = TARGETS[name]
    src = [os.path.join(CSRC, s) for s in sources]
    dep = [d if os.path.isabs(d) else os.path.join(CSRC, d) for d in deps]
    return os.path.join(HERE, name), src, dep


def is_stale(name: str = "libpong_b200.so") -> bool:
    lib, src, dep = _paths(name)
    if not os.path.exists(lib):
        return True
    built = os.path.getmtime(lib)
    return any(os.path.getmtime(d) > built for d in src + dep)


def build_one(name: str, force: bool = False, verbose: bool = False) -> str:
    lib, src, _ = _paths(name)
    if not force and not is_stale(name):
        return lib
    tmp = lib + ".tmp.%d" % os.getpid()
    cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + src
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose:
        sys.stderr.write(res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    os.replace(tmp, lib)
    return lib


def build(force: bool = False, verbose: bool = False) -> str:
    """Build every library that is missing or older than its sources; returns
    the path of the Pong library."""
    for name in TARGETS:
        build_one(name, force, verbose)
    return LIB


if __name__ == "__main__":
    build(force=True, verbose="-v" in sys.argv)
    print(LIB)
    print(CARTPOLE_LIB)
    print(GRU_POLICY_LIB)
