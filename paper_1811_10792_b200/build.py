"""Builds libsgp.so (sm_100a) in-tree with nvcc.  Usable as ``python -m paper_1811_10792_b200.build``."""
from __future__ import annotations

import os
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG_DIR)
CSRC = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.path.join(PKG_DIR, "libsgp.so")

SOURCES = ["regs_inst_v4.cu", "regs_inst_v4_diag.cu", "regs_inst_v1.cu", "regs_inst_v1_diag.cu", "tma_inst.cu",
           "tma_inst_diag.cu", "sgp_api.cu", "launch_regs.cu", "launch_tma.cu", "launch_cluster.cu", "launch_peel.cu", "sgp_static.cu", "sgp_rank.cu", "schedule.cpp"]
HEADERS = ["step_common.cuh", "step_regs_kernel.cuh", "step_tma_kernel.cuh", "step_cluster_kernel.cuh", "step_peel_kernel.cuh", "regs_instances.inc",
           "tma_instances.inc", "aux_kernels.cuh", "rank_kernels.cuh", "launch.h", "schedule.h"]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC,-Wall,-Wextra",
]
LINK_FLAGS = ["-shared", "-cudart", "static"]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def needs_build() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS] + [os.path.join(ROOT, "include", "sgp.h")]
    return any(os.path.getmtime(p) > t for p in deps)


def build(force: bool = False, verbose: bool = False, extra_flags=(), lib_path: str = LIB_PATH) -> str:
    """Compiles the library if it is missing or older than its sources; returns its path.

    Every source is compiled to an object of its own, in parallel, then linked.  `extra_flags` reach every
    compile (e.g. ("-DSGP_CHECKED",) with another `lib_path` for the bounds-checked build)."""
    if not force and lib_path == LIB_PATH and not needs_build():
        return lib_path
    from concurrent.futures import ThreadPoolExecutor
    tag = os.path.splitext(os.path.basename(lib_path))[0]
    import tempfile
    obj_dir = os.path.join(tempfile.gettempdir(), "sgp_build_%d" % os.getuid(), tag)      # objects stay out of the tree
    os.makedirs(obj_dir, exist_ok=True)
    inc = ["-I", os.path.join(ROOT, "include"), "-I", CSRC]

    def compile_one(src):
        obj = os.path.join(obj_dir, os.path.splitext(src)[0] + ".o")
        cmd = [_nvcc(), *NVCC_FLAGS, *extra_flags, *inc, "-c", os.path.join(CSRC, src), "-o", obj]
        if verbose:
            print(" ".join(cmd), file=sys.stderr)
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}:\n" + res.stdout + res.stderr)
        if verbose and (res.stdout or res.stderr):
            print(res.stdout + res.stderr, file=sys.stderr)
        return obj

    with ThreadPoolExecutor(max_workers=min(len(SOURCES), os.cpu_count() or 1)) as pool:
        objs = list(pool.map(compile_one, SOURCES))
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", *LINK_FLAGS, *objs, "-o", lib_path]
    if verbose:
        print(" ".join(cmd), file=sys.stderr)
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("link failed:\n" + res.stdout + res.stderr)
    return lib_path


CHECKED_LIB_PATH = os.path.join(PKG_DIR, "libsgp_checked.so")


def build_checked(force: bool = False, verbose: bool = False) -> str:
    """The bounds-checked build (-DSGP_CHECKED): every table index and global offset is tested before use."""
    if not force and os.path.exists(CHECKED_LIB_PATH):
        t = os.path.getmtime(CHECKED_LIB_PATH)
        deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS] + [os.path.join(ROOT, "include", "sgp.h")]
        if all(os.path.getmtime(p) <= t for p in deps):
            return CHECKED_LIB_PATH
    return build(force=True, verbose=verbose, extra_flags=("-DSGP_CHECKED",), lib_path=CHECKED_LIB_PATH)


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True,
                extra_flags=("-Xptxas", "-v") if "--ptxas" in sys.argv else ()))
