"""Build libgraft.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

Every source becomes an object under _build/ (rebuilt when it or one of its headers is newer) and the objects are
linked into libgraft.so.  The table-precompute GEMM (csrc/tables_gemm.cu) is built from the CUTLASS / CuTe sm100
templates; their headers come from a CUTLASS tree vendored in the Python environment (GRAFT_CUTLASS_DIR overrides).
Without such a tree csrc/tables_gemm_stub.cu is linked instead: the library is complete, and the table precompute
runs its fp32 FMA kernel for every input.
"""
from __future__ import annotations

import importlib.util
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libgraft.so")
GRAFT_H = os.path.join("..", "..", "include", "graft.h")
ALL_HEADERS = ["common.cuh", "internal.h", "edge_score.cuh", "cosine.cuh", "saba.cuh", GRAFT_H]
# source -> headers it depends on
SOURCES = {
    "api.cu": ALL_HEADERS,
    "vocab_pass.cu": ALL_HEADERS,
    "tdes.cu": ALL_HEADERS,
    "tree.cu": ALL_HEADERS,
    "tdes_train.cu": ["common.cuh", "internal.h", GRAFT_H],
    "saba_fit.cu": ["common.cuh", "internal.h", GRAFT_H],
}
GEMM_SRC = {"tables_gemm.cu": ["internal.h", GRAFT_H]}       # with a CUTLASS tree
GEMM_STUB = {"tables_gemm_stub.cu": ["internal.h", GRAFT_H]}  # without one
# no --use_fast_math: the fp64 pieces (log-sum-exp fold, SABA) and the fp32 divisions must stay IEEE
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC"]


def cutlass_dir() -> str | None:
    """Root of a CUTLASS tree with include/ and tools/util/include/ (version 4.x: sm100 collective builders), or None."""
    cands = []
    if os.environ.get("GRAFT_CUTLASS_DIR"):
        cands.append(os.environ["GRAFT_CUTLASS_DIR"])
    for pkg, sub in (("flashinfer", os.path.join("data", "cutlass")), ("tilelang", os.path.join("3rdparty", "cutlass"))):
        spec = importlib.util.find_spec(pkg)
        if spec and spec.submodule_search_locations:
            cands.append(os.path.join(list(spec.submodule_search_locations)[0], sub))
    for c in cands:
        if os.path.exists(os.path.join(c, "include", "cutlass", "gemm", "collective", "builders", "sm100_umma_builder.inl")):
            return c
    return None


def sources() -> dict:
    """The sources of this build: the tensor-core GEMM when a CUTLASS tree is at hand, its stand-in otherwise."""
    if os.environ.get("GRAFT_NO_CUTLASS") or cutlass_dir() is None:
        return {**SOURCES, **GEMM_STUB}
    return {**SOURCES, **GEMM_SRC}


def _stale(target: str, deps: list[str]) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def _obj(src: str) -> str:
    return os.path.join(OBJ, src.replace(".cu", ".o"))


def needs_build() -> bool:
    srcs = sources()
    for src, hdrs in srcs.items():
        if _stale(_obj(src), [os.path.join(CSRC, src)] + [os.path.join(CSRC, h) for h in hdrs]):
            return True
    return _stale(LIB, [_obj(s) for s in srcs])


def build(force: bool = False, verbose: bool = False) -> str:
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(OBJ, exist_ok=True)
    inc = ["-I", os.path.join(HERE, "..", "include")]
    cmds = []
    srcs = sources()
    for src, hdrs in srcs.items():
        deps = [os.path.join(CSRC, src)] + [os.path.join(CSRC, h) for h in hdrs]
        if not (force or _stale(_obj(src), deps)):
            continue
        extra = []
        if src == "tables_gemm.cu":
            cut = cutlass_dir()
            extra = ["--expt-relaxed-constexpr", "-diag-suppress", "20012", "-I", os.path.join(cut, "include"),
                     "-I", os.path.join(cut, "tools", "util", "include")]
        cmds.append([nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + inc + extra +
                    ["-c", os.path.join(CSRC, src), "-o", _obj(src)])
    procs = [subprocess.Popen(c) for c in cmds]  # the sources compile side by side
    failed = [c for c, pr in zip(cmds, procs) if pr.wait() != 0]
    if failed:
        raise subprocess.CalledProcessError(1, failed[0])
    stamp = os.path.join(OBJ, "linked_sources.txt")  # relink when the set of sources changes (GEMM <-> stand-in)
    names = " ".join(sorted(srcs))
    if force or _stale(LIB, [_obj(s) for s in srcs]) or not os.path.exists(stamp) or open(stamp).read() != names:
        subprocess.check_call([nvcc, "-shared", "-o", LIB] + [_obj(s) for s in srcs] + ["-lcudart"])
        with open(stamp, "w") as f:
            f.write(names)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
