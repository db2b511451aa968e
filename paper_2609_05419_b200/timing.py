"""Per-phase timing of any entry point on synthetic inputs (CUDA events recorded by the library on the call's stream).

  python -m paper_2609_05419_b200.timing --op zgemm --m 8192 --n 8192 --k 8192 --nmod 16
  python -m paper_2609_05419_b200.timing --op cgemm --m 16384 --n 16384 --k 4096 --nmod 7
  python -m paper_2609_05419_b200.timing --op zherk --n 8192 --k 8192 --nmod 16

Prints one JSON line: effective TFLOP/s (8mnk/t for GEMM, 4n^2k/t for HERK), milliseconds per call and per phase.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding as b
from . import inputs


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--op", default="zgemm", choices=["zgemm", "cgemm", "zherk"])
    ap.add_argument("--m", type=int, default=8192)
    ap.add_argument("--n", type=int, default=8192)
    ap.add_argument("--k", type=int, default=8192)
    ap.add_argument("--nmod", type=int, default=16)
    ap.add_argument("--dist", default="uniform", choices=["uniform", "phi"])
    ap.add_argument("--phi", type=float, default=0.5)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--seed", type=int, default=1)
    a = ap.parse_args()
    m, n, k, nmod = (a.n if a.op == "zherk" else a.m), a.n, a.k, a.nmod
    dtype = np.complex64 if a.op == "cgemm" else np.complex128
    tdtype = torch.complex64 if a.op == "cgemm" else torch.complex128
    dev = lambda x: torch.from_numpy(np.ascontiguousarray(x.T)).cuda().t()
    if a.op == "zherk":
        A = dev(inputs.herk_input(n, k, a.seed, a.dist, a.phi))
        B = None
        opcode, flops = b.OP_ZHERK, 4.0 * n * n * k
    else:
        Ah, Bh = inputs.complex_inputs(m, n, k, a.seed, a.dist, a.phi, dtype=dtype)
        A, B = dev(Ah), dev(Bh)
        opcode, flops = (b.OP_CGEMM if a.op == "cgemm" else b.OP_ZGEMM), 8.0 * m * n * k
    C = torch.empty((n, m), dtype=tdtype, device="cuda").t()
    ws = torch.zeros(b.workspace_bytes(opcode, m, n, k, nmod), dtype=torch.uint8, device="cuda")
    b.set_workspace(ws)
    stream = torch.cuda.current_stream()

    def call():
        if a.op == "zherk":
            b.zherk2m(A, C, nmod, stream)
        elif a.op == "cgemm":
            b.cgemm2m(A, B, C, nmod, stream)
        else:
            b.zgemm2m(A, B, C, nmod, stream)

    for _ in range(max(a.warmup, 1)):
        call()
    b.device_status()
    b.set_profiling(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(a.steps):
        call()
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / a.steps
    phase, calls = b.phase_ms()
    b.set_profiling(False)
    b.device_status()
    total, per = b.last_launch_count()
    gemms = nmod if a.op == "zherk" else 2 * nmod
    print(json.dumps({"op": a.op, "m": m, "n": n, "k": k, "nmod": nmod, "ms_per_call": ms, "effective_tflops": flops / ms / 1e9,
                      "scan_ms": phase[0], "residues_ms": phase[1], "gemm_ms": phase[2], "post_ms": phase[3],
                      "gemm_int8_tops": 2.0 * gemms * m * n * k / phase[2] / 1e9 if phase[2] > 0 else None,
                      "launches_per_call": per}))
    b.set_workspace(None)


if __name__ == "__main__":
    main()
