"""Compile the CUDA sources in csrc/ into libgemm2m.so (sm_100a only), next to this file."""
from __future__ import annotations

import os
import shutil
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
SOURCES = ["api.cu", "tables.cu", "scan.cu", "residues.cu", "post.cu", "post_fp.cu", "post_herk.cu", "gemm_check.cu", "gemm_i8_2cta.cu", "static_scratch.cu"]
HEADERS = ["common.cuh", "gemm_ptx.cuh", "prepost_common.cuh", "residues_common.cuh", "post_common.cuh", "post_mma.cuh", os.path.join("..", "..", "include", "gemm2m.h")]
LIB = os.path.join(HERE, "libgemm2m.so")


def nvcc_path() -> str:
    cand = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(cand):
        raise RuntimeError("nvcc not found: the gemm2m CUDA library cannot be built")
    return cand


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not is_stale():
        return LIB
    cmd = [nvcc_path(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
           "-Xcompiler", "-fPIC", "-shared"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES] + ["-o", LIB + ".tmp"]
    subprocess.run(cmd, check=True)
    os.replace(LIB + ".tmp", LIB)
    return LIB


def build_issue_rates(out_dir: str | None = None) -> str:
    """Compiles csrc/issue_rates.cu (a stand-alone microbenchmark of instruction issue rates, not part of the library) into
    an executable under out_dir (default: next to this file, as issue_rates.bin) and returns its path."""
    exe = os.path.join(out_dir or HERE, "issue_rates.bin")
    cmd = [nvcc_path(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
           os.path.join(CSRC, "issue_rates.cu"), "-o", exe + ".tmp"]
    subprocess.run(cmd, check=True)
    os.replace(exe + ".tmp", exe)
    return exe


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
