"""Build the CUDA shared library in-tree with nvcc (sm_100a only).

    python -m paper_2607_24027_b200.build [--force] [--verbose]

Produces ``paper_2607_24027_b200/libsol_attn.so``.  nvcc cross-compiles without a GPU.
"""
from __future__ import annotations

import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libsol_attn.so")
SOURCES = ["api.cu", "pool.cu", "fwd_mma_sync.cu", "fwd_sm100.cu", "thresholds_static.cu", "route_materialized.cu",
           "route_prepass.cu"]
HEADERS = [os.path.join(CSRC, "common.cuh"), os.path.join(CSRC, "ptx_sm100.cuh"), os.path.join(CSRC, "tmap.cuh"),
           os.path.join(CSRC, "fwd_sm100_prof.cuh"),
           os.path.join(ROOT, "include", "sol_attn.h")]


def _nvcc() -> str:
    cand = os.environ.get("NVCC") or "/usr/local/cuda/bin/nvcc"
    return cand if os.path.exists(cand) else "nvcc"


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + [h for h in HEADERS if os.path.exists(h)]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, profile: bool = False) -> str:
    """Compile every kernel for sm_100a and link the C-ABI library; returns its path.

    ``profile=True`` builds ``libsol_attn_prof.so`` instead, whose fused kernel records how many
    cycles each warp role spends in each kind of wait (a development aid, never the default).
    """
    if profile:
        return _build_variant(os.path.join(PKG, "libsol_attn_prof.so"), ["-DSOL_PROFILE"], "_prof", verbose)
    if not force and not _stale():
        return LIB
    return _build_variant(LIB, [], "", verbose)


def _build_variant(lib: str, defines, suffix: str, verbose: bool) -> str:
    objs = []
    common = [_nvcc(), "-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
              "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    common += defines
    if verbose:
        common += ["-Xptxas", "-v"]
    procs = []
    for s in SOURCES:
        obj = os.path.join(CSRC, s.replace(".cu", suffix + ".o"))
        objs.append(obj)
        procs.append((s, subprocess.Popen(common + ["-c", os.path.join(CSRC, s), "-o", obj],
                                          stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    failed = False
    for s, p in procs:
        out, _ = p.communicate()
        if verbose or p.returncode != 0:
            sys.stderr.write(f"--- {s}\n{out}\n")
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    link = [_nvcc(), "-shared", "-o", lib] + objs + ["-lcudart"]
    subprocess.run(link, check=True)
    return lib


if __name__ == "__main__":
    path = build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, profile="--profile" in sys.argv)
    print(path)
