"""Per-phase timing of any entry point on synthetic inputs (CUDA events recorded by the library on the call's stream).

  python -m paper_2609_05419_b200.timing --op zgemm --m 8192 --n 8192 --k 8192 --nmod 16
  python -m paper_2609_05419_b200.timing --op cgemm --m 16384 --n 16384 --k 4096 --nmod 7
  python -m paper_2609_05419_b200.timing --op zherk --n 8192 --k 8192 --nmod 16

  python -m paper_2609_05419_b200.timing --op dsyrk --n 8192 --k 8192 --nmod 16      (also zher2k, dsyr2k)
  python -m paper_2609_05419_b200.timing --op dgemm --m 8192 --n 8192 --k 8192 --nmod 15     (real Ozaki-II scheme)
  python -m paper_2609_05419_b200.timing --op zgemm_eis --m 8192 --n 8192 --k 8192 --nmod 16 (Eisenstein-integer variant)

  python -m paper_2609_05419_b200.timing --op zgemm_host --m 8192 --n 8192 --k 8192 --nmod 16 (host operands, copies inside the call)
  python -m paper_2609_05419_b200.timing --op int8_yardstick --m 8192 --n 8192 --k 8192 --nmod 16
      (NOT this library: 2 x nmod int8 GEMMs with int32 output by the vendor library through torch._int_mm, back to back,
       as a yardstick for the tensor-core phase only)

Prints one JSON line: effective TFLOP/s (BLAS flop counts: 8mnk for GEMM, 4n^2k HERK, 8n^2k HER2K, n^2k SYRK, 2n^2k SYR2K,
divided by the time), milliseconds per call and per phase.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding as b
from . import inputs


def yardstick(a):
    """The vendor library's int8 GEMM (int32 output, no modular reduction) on operands of the residue planes' shape."""
    g = torch.Generator(device="cuda").manual_seed(a.seed)
    X = torch.randint(-120, 121, (a.m, a.k), dtype=torch.int8, device="cuda", generator=g)
    Y = torch.randint(-120, 121, (a.n, a.k), dtype=torch.int8, device="cuda", generator=g).t()     # K-major like the planes
    count = 2 * a.nmod
    run = lambda: [torch._int_mm(X, Y) for _ in range(count)]
    for _ in range(max(a.warmup, 1)):
        run()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(a.steps):
        run()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / a.steps
    print(json.dumps({"op": a.op, "m": a.m, "n": a.n, "k": a.k, "gemms_per_step": count, "ms_per_step": ms,
                      "int8_tops": 2.0 * count * a.m * a.n * a.k / ms / 1e9, "output": "int32, no reduction modulo m"}))


def host_call(a):
    """zgemm2m_host on pinned host operands: milliseconds per call with the transfers inside."""
    m, n, k, nmod = a.m, a.n, a.k, a.nmod
    Ah, Bh = inputs.complex_inputs(m, n, k, a.seed, a.dist, a.phi)
    pin = lambda x: torch.from_numpy(np.ascontiguousarray(x.T)).pin_memory().t()
    A, B = pin(Ah), pin(Bh)
    C = torch.empty((n, m), dtype=torch.complex128).pin_memory().t()
    ws = torch.zeros(b.workspace_bytes(b.OP_ZGEMM_HOST, m, n, k, nmod), dtype=torch.uint8, device="cuda")
    b.set_workspace(ws)
    stream = torch.cuda.current_stream()
    for _ in range(max(a.warmup, 1)):
        b.zgemm2m_host(A, B, C, nmod, stream)
    b.device_status()
    b.set_profiling(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(a.steps):
        b.zgemm2m_host(A, B, C, nmod, stream)
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / a.steps
    phase, _ = b.phase_ms()
    b.set_profiling(False)
    b.device_status()
    print(json.dumps({"op": a.op, "m": m, "n": n, "k": k, "nmod": nmod, "ms_per_call": ms, "effective_tflops": 8.0 * m * n * k / ms / 1e9,
                      "h2d_bytes": 16 * (m * k + k * n), "d2h_bytes": 16 * m * n,
                      "bus_gbs_h2d_if_alone": 16 * (m * k + k * n) / ms / 1e6,
                      "scan_ms": phase[0], "residues_ms": phase[1], "gemm_ms": phase[2], "post_ms": phase[3]}))
    b.set_workspace(None)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--op", default="zgemm", choices=["zgemm", "cgemm", "zherk", "zher2k", "dsyrk", "dsyr2k", "dgemm", "zgemm_eis", "zgemm_host", "int8_yardstick"])
    ap.add_argument("--m", type=int, default=8192)
    ap.add_argument("--n", type=int, default=8192)
    ap.add_argument("--k", type=int, default=8192)
    ap.add_argument("--nmod", type=int, default=16)
    ap.add_argument("--dist", default="uniform", choices=["uniform", "phi"])
    ap.add_argument("--phi", type=float, default=0.5)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--seed", type=int, default=1)
    ap.add_argument("--panels", type=int, default=0, help="most column panels per call (1 = every phase on the caller's stream, one after the other)")
    a = ap.parse_args()
    if a.panels:
        b.debug_set_panels(a.panels)
    if a.op == "int8_yardstick":
        return yardstick(a)
    if a.op == "zgemm_host":
        return host_call(a)
    rank = a.op in ("zherk", "zher2k", "dsyrk", "dsyr2k")
    m, n, k, nmod = (a.n if rank else a.m), a.n, a.k, a.nmod
    dtype = np.complex64 if a.op == "cgemm" else np.complex128
    tdtype = torch.complex64 if a.op == "cgemm" else torch.complex128
    dev = lambda x: torch.from_numpy(np.ascontiguousarray(x.T)).cuda().t()
    if rank:
        real = a.op in ("dsyrk", "dsyr2k")
        two = a.op in ("zher2k", "dsyr2k")
        gen = lambda seed: inputs.herk_input(n, k, seed, a.dist, a.phi)
        A = dev(np.asfortranarray(gen(a.seed).real.copy()) if real else gen(a.seed))
        B = (dev(np.asfortranarray(gen(a.seed + 1).real.copy()) if real else gen(a.seed + 1))) if two else None
        opcode = {"zherk": b.OP_ZHERK, "zher2k": b.OP_ZHER2K, "dsyrk": b.OP_DSYRK, "dsyr2k": b.OP_DSYR2K}[a.op]
        flops = {"zherk": 4.0, "zher2k": 8.0, "dsyrk": 1.0, "dsyr2k": 2.0}[a.op] * n * n * k     # BLAS flop counts
        tdtype = torch.float64 if real else torch.complex128
    elif a.op == "dgemm":              # real Ozaki-II scheme: the real parts of the same synthetic inputs
        Ah, Bh = inputs.complex_inputs(m, n, k, a.seed, a.dist, a.phi)
        A, B = dev(np.asfortranarray(Ah.real.copy())), dev(np.asfortranarray(Bh.real.copy()))
        opcode, flops, tdtype = b.OP_DGEMM_OZAKI2, 2.0 * m * n * k, torch.float64
    else:
        Ah, Bh = inputs.complex_inputs(m, n, k, a.seed, a.dist, a.phi, dtype=dtype)
        A, B = dev(Ah), dev(Bh)
        opcode = {"cgemm": b.OP_CGEMM, "zgemm_eis": b.OP_ZGEMM_EISENSTEIN}.get(a.op, b.OP_ZGEMM)
        flops = 8.0 * m * n * k
    C = torch.empty((n, m), dtype=tdtype, device="cuda").t()
    ws = torch.zeros(b.workspace_bytes(opcode, m, n, k, nmod), dtype=torch.uint8, device="cuda")
    b.set_workspace(ws)
    stream = torch.cuda.current_stream()

    def call():
        if a.op == "zherk":
            b.zherk2m(A, C, nmod, stream)
        elif a.op == "zher2k":
            b.zher2k2m(A, B, C, nmod, stream)
        elif a.op == "dsyrk":
            b.dsyrk2m(A, C, nmod, stream)
        elif a.op == "dsyr2k":
            b.dsyr2k2m(A, B, C, nmod, stream)
        elif a.op == "cgemm":
            b.cgemm2m(A, B, C, nmod, stream)
        elif a.op == "dgemm":
            b.dgemm_ozaki2(A, B, C, nmod, stream)
        elif a.op == "zgemm_eis":
            b.zgemm2m_eisenstein(A, B, C, nmod, stream)
        else:
            b.zgemm2m(A, B, C, nmod, stream)

    for _ in range(max(a.warmup, 1)):
        call()
    b.device_status()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(a.steps):
        call()
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / a.steps
    b.set_profiling(True)              # the phase times come from a second loop: the events around every phase cost time at small sizes
    for _ in range(a.steps):
        call()
    torch.cuda.synchronize()
    phase, calls = b.phase_ms()
    b.set_profiling(False)
    b.device_status()
    total, per = b.last_launch_count()
    planes = 2 * min(nmod, 22) + 3 * max(nmod - 22, 0)       # complex GEMM: 2 real GEMMs per 2M modulus, 3 per 3M modulus
    if a.op == "zgemm_eis":
        planes = 2 * nmod
    gemms = {"zherk": nmod, "zher2k": 2 * nmod, "dsyrk": nmod, "dsyr2k": 2 * nmod, "dgemm": nmod}.get(a.op, planes)
    kin = (k + 1) // 2 if a.op in ("dsyrk", "dsyr2k") else k
    print(json.dumps({"op": a.op, "m": m, "n": n, "k": k, "nmod": nmod, "ms_per_call": ms, "effective_tflops": flops / ms / 1e9,
                      "scan_ms": phase[0], "residues_ms": phase[1], "gemm_ms": phase[2], "post_ms": phase[3],
                      "gemm_int8_tops": 2.0 * gemms * m * n * kin / phase[2] / 1e9 if phase[2] > 0 else None,
                      "launches_per_call": per}))
    b.set_workspace(None)


if __name__ == "__main__":
    main()
