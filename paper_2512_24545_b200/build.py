"""Build libmdbf.so in-tree with nvcc for sm_100a (cross-compiles without a GPU).

    python -m paper_2512_24545_b200.build [--force] [--verbose] [--bounds-check]

--bounds-check (or MDBF_BOUNDS_CHECK=1 in the environment, which is how a test run selects it) compiles the
index checks of the forward kernels' stores in (-DMDBF_BOUNDS_CHECK): a store outside its buffer is skipped and
recorded as MDBF_ERR_BOUNDS in the handle's status word.  The library is rebuilt when the requested variant differs
from the one on disk.
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libmdbf.so")
SOURCES = ["mdbf_api.cu", "pack.cu", "reconstruct.cu", "forward_alu.cu", "forward_prefill.cu", "forward_tmem_t1.cu", "forward_t1.cu", "forward_static.cu", "forward_mat.cu", "msvid.cu", "gemm3x.cu", "admm.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr"]
STAMP = os.path.join(HERE, "libmdbf.variant")          # which variant libmdbf.so holds


def _bounds_check_requested(flag: bool | None) -> bool:
    if flag is not None:
        return flag
    return os.environ.get("MDBF_BOUNDS_CHECK", "0") not in ("", "0")


def _newest_source() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    paths.append(os.path.join(ROOT, "include", "mdbf.h"))
    return max(os.path.getmtime(p) for p in paths)


def build(force: bool = False, verbose: bool = False, bounds_check: bool | None = None) -> str:
    variant = "bounds-check" if _bounds_check_requested(bounds_check) else "default"
    on_disk = open(STAMP).read().strip() if os.path.exists(STAMP) else "default"
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= _newest_source() and on_disk == variant:
        return LIB
    flags = NVCC_FLAGS + (["-DMDBF_BOUNDS_CHECK"] if variant == "bounds-check" else [])
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objs = []
    procs = []
    for src in SOURCES:
        obj = os.path.join(CSRC, src.replace(".cu", ".o"))
        cmd = [nvcc, *flags, "-I", os.path.join(ROOT, "include"), "-I", CSRC, "-c",
               os.path.join(CSRC, src), "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas")
            cmd.insert(2, "-v")
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
    subprocess.check_call([nvcc, "-shared", "-o", LIB, *objs, "-lcudart", "-lcublas", "-lcusolver",
                           "-Xlinker", "-rpath=/usr/local/cuda/lib64"])
    with open(STAMP, "w") as f:
        f.write(variant + "\n")
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv,
                bounds_check=True if "--bounds-check" in sys.argv else None))
