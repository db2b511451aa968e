"""Benchmark of the gemm2m hot path (2M multiplication + Ozaki-II) on B200.

One step = one call of the chosen entry point (exponent scan, quantise + residues, int8 GEMMs, post-processing) on a
synthetic problem.  Prints ONE JSON line (rank 0).  The default is the headline configuration: zgemm2m, m = n = k = 8192,
16 moduli, inputs (rand-0.5)*exp(0.5*randn).

  python bench.py                          # zgemm2m, 1 GPU
  python bench.py --op cgemm               # cgemm2m, complex64, m = n = 16384, k = 4096, 7 moduli, parts uniform(-1, 1)
  python bench.py --op zherk               # zherk2m, n = k = 8192, 16 moduli, parts uniform(-1, 1); flops counted as 4 n^2 k
  python bench.py --impl reference         # the CPU oracle timed on the host cores (a baseline, not a target)
  torchrun ... bench.py --gpus N           # N independent replicas (the path is single-GPU; no collective)
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

UNIT = "TFLOP/s"
INT8_NOMINAL_TOPS = 4500.0          # dense int8, nominal
INT8_OVER_BF16 = 2.0                # nominal ratio used to turn the measured bf16 peak into an int8 peak
# DRAM bytes (read + write) of a GEMM launch per byte of the int8 planes it touches, from the ncu capture of one panel launch
# of the 4096^3, 16-modulus case: (673.9 + 123.9) MB over 805.3 MB of planes.
GEMM_DRAM_BYTES_PER_PLANE_BYTE = (673.872384e6 + 123.916288e6) / (32 * 4096 * (4096 + 1024 + 1024))

# Per operation: metric name, default shape and modulus count, input distribution, flop count of the BLAS operation.
OPS = {
    "zgemm": dict(metric="zgemm2m_effective_tflops_8mnk_per_t", m=8192, n=8192, k=8192, nmod=16, dist="phi"),
    "cgemm": dict(metric="cgemm2m_effective_tflops_8mnk_per_t", m=16384, n=16384, k=4096, nmod=7, dist="uniform"),
    "zherk": dict(metric="zherk2m_effective_tflops_4n2k_per_t", m=8192, n=8192, k=8192, nmod=16, dist="uniform"),
}


def flops_of(a):
    return 4.0 * a.n * a.n * a.k if a.op == "zherk" else 8.0 * a.m * a.n * a.k


def job_value(flops_per_rank_step, world, ms_per_step):
    """Whole-job throughput in TFLOP/s: every rank processed its own problem in the (max over ranks) step time."""
    return flops_per_rank_step * world / (ms_per_step * 1e-3) / 1e12


def max_over_ranks(x, world, device):
    """Max of a per-rank scalar over all ranks (any torch.distributed backend); identity for one rank."""
    if world == 1:
        return float(x)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--op", default="zgemm", choices=sorted(OPS))
    ap.add_argument("--m", type=int, default=None)
    ap.add_argument("--n", type=int, default=None)
    ap.add_argument("--k", type=int, default=None)
    ap.add_argument("--nmod", type=int, default=None)
    ap.add_argument("--phi", type=float, default=0.5)
    ap.add_argument("--seed", type=int, default=1)
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="target CPU time of the oracle sample")
    ap.add_argument("--ab-calls", type=int, default=50, help="calls per panel mode in the interleaved overlap-on / overlap-off comparison")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    a = ap.parse_args()
    for key in ("m", "n", "k", "nmod"):
        if getattr(a, key) is None:
            setattr(a, key, OPS[a.op][key])
    if a.op == "zherk":
        a.m = a.n
    a.dist = OPS[a.op]["dist"]
    a.metric = OPS[a.op]["metric"]
    return a


def workload_name(a):
    parts = f"(rand-0.5)*exp({a.phi}*randn)" if a.dist == "phi" else "uniform(-1,1)"
    if a.op == "zherk":
        return f"zherk2m complex128 C=A A^H lower n={a.n} k={a.k} nmod={a.nmod} parts={parts}"
    return f"{a.op}2m complex{64 if a.op == 'cgemm' else 128} m={a.m} n={a.n} k={a.k} nmod={a.nmod} parts={parts}"


def host_inputs(a, seed):
    """The synthetic operands on the host (numpy, column-major): A and B; zherk has A only (B is None)."""
    from paper_2609_05419_b200 import inputs
    if a.op == "zherk":
        return inputs.herk_input(a.n, a.k, seed, a.dist, a.phi), None
    dtype = np.complex64 if a.op == "cgemm" else np.complex128
    return inputs.complex_inputs(a.m, a.n, a.k, seed, dist=a.dist, phi=a.phi, dtype=dtype)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_burst=float(d["bf16_tflops"]),
                    bf16_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


# ----------------------------------------------------------------------------------------------- CPU oracle leg
def oracle_operands(a, A, B):
    """Operands of the double-double oracle: complex128 copies (exact for complex64 inputs); zherk multiplies A by A^H."""
    A = np.asfortranarray(A, dtype=np.complex128)
    B = np.asfortranarray(A.conj().T) if a.op == "zherk" else np.asfortranarray(B, dtype=np.complex128)
    return A, B


def time_oracle(a, A, B, seconds):
    """Times the double-double 4M oracle, as it stands, on a bounded sample of entries of the same product (A, B: its operands)."""
    from oracle import direct
    from paper_2609_05419_b200 import inputs
    cores = direct.num_threads()
    rows, cols = (a.n, a.n) if a.op == "zherk" else (a.m, a.n)
    probe = inputs.sample_indices(rows, cols, 2048, seed=11)
    t0 = time.perf_counter()
    direct.zgemm4m_dd_samples(A, B, probe)
    t_probe = max(time.perf_counter() - t0, 1e-6)
    count = int(min(max(len(probe), len(probe) * seconds / t_probe), rows * cols))
    pairs = inputs.sample_indices(rows, cols, count, seed=12)
    t0 = time.perf_counter()
    direct.zgemm4m_dd_samples(A, B, pairs)
    dt = time.perf_counter() - t0
    per_entry = flops_of(a) / (rows * cols)                 # the metric's flop count, spread over the entries of the full result
    return dict(value=per_entry * len(pairs) / dt / 1e12, unit=UNIT, cores=cores, kind="oracle",
                sample=f"{len(pairs)} sampled entries of the {rows}x{cols}x{a.k} product (double-double 4M, {dt:.1f} s)"), dt


def run_reference(a):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    A, B = oracle_operands(a, *host_inputs(a, a.seed))
    per_step = max(2.0, min(a.cpu_seconds, 120.0 / max(a.steps + a.warmup, 1)))
    for _ in range(a.warmup):
        time_oracle(a, A, B, per_step)
    vals, times = [], []
    last = None
    for _ in range(a.steps):
        last, dt = time_oracle(a, A, B, per_step)
        vals.append(last["value"])
        times.append(dt)
    value = float(np.mean(vals))
    last["value"] = value
    line = {"impl": "reference", "metric": a.metric, "value": value, "unit": UNIT, "n_gpus": a.gpus, "steps": a.steps,
            "warmup": a.warmup, "ms_per_step": float(np.mean(times)) * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_name(a), "note": "CPU oracle on host cores; each step is a bounded sample of entries"},
            "cpu_baseline": last,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------- GPU leg
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = str(index)
        try:    # nvidia-smi numbers the GPUs it sees, CUDA the ones it was given: name the device by its PCI address instead
            import torch
            pr = torch.cuda.get_device_properties(index)
            self.index = "%08x:%02x:%02x.0" % (pr.pci_domain_id, pr.pci_bus_id, pr.pci_device_id)
        except Exception:
            pass
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "20"], stdout=self.out, stderr=subprocess.DEVNULL)
            t0 = time.time()                     # wait for the first sample so that the timed region is covered
            while time.time() - t0 < 5.0 and os.path.getsize(self.path) == 0:
                self.out.flush()
                time.sleep(0.02)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, mx, reasons, power = [], [], set(), []
        with open(self.path) as f:
            for line in f:
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    sm.append(float(parts[1]))
                    mx.append(float(parts[2]))
                    power.append(float(parts[3]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        os.unlink(self.path)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        load = [s for s, p in zip(sm, power) if p > 0.5 * max(power)] or sm
        return {"sm_mhz": float(np.median(load)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "power_w_max": float(max(power)), "samples": len(sm)}


def run_ours(a):
    import torch
    import torch.distributed as dist
    from paper_2609_05419_b200 import binding as b

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    b.lib()   # fails loudly if the CUDA library is missing
    m, n, k, nmod = a.m, a.n, a.k, a.nmod
    herk = a.op == "zherk"
    cdtype = torch.complex64 if a.op == "cgemm" else torch.complex128
    esize = 8 if a.op == "cgemm" else 16
    A, B = host_inputs(a, a.seed + rank)                      # every replica its own problem
    # pinned host buffers in column-major order (the transposed view is what the C ABI sees)
    pin = lambda X: torch.from_numpy(np.ascontiguousarray(X.T)).pin_memory()
    hA, hB = pin(A), (None if herk else pin(B))
    hC = torch.zeros((n, m), dtype=cdtype).pin_memory()
    dA, dB = hA.cuda(), (None if herk else hB.cuda())
    dC = torch.zeros((n, m), dtype=cdtype, device="cuda")
    host_form = a.op == "zgemm" and not a.no_e2e              # zgemm2m_host: its workspace is zgemm2m's plus device copies of A, B, C
    ws_op = {"zgemm": b.OP_ZGEMM_HOST if host_form else b.OP_ZGEMM, "cgemm": b.OP_CGEMM, "zherk": b.OP_ZHERK}[a.op]
    ws = torch.zeros(b.workspace_bytes(ws_op, m, n, k, nmod), dtype=torch.uint8, device="cuda")
    b.set_workspace(ws)
    stream = torch.cuda.current_stream()

    def step():
        if a.op == "zgemm":
            b.zgemm2m(dA.t(), dB.t(), dC.t(), nmod, stream)
        elif a.op == "cgemm":
            b.cgemm2m(dA.t(), dB.t(), dC.t(), nmod, stream)
        else:
            b.zherk2m(dA.t(), dC.t(), nmod, stream)

    for _ in range(max(a.warmup, 3)):
        step()
    b.device_status()

    # ---- timed region: device-resident inputs; an event after every step (same stream) gives the per-step times
    sampler = ClockSampler(local)
    b.set_profiling(True)
    barrier()
    sampler.start()
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(a.steps + 1)]
    marks[0].record(stream)
    for i in range(a.steps):
        step()
        marks[i + 1].record(stream)
    barrier()
    clocks = sampler.stop()
    ms_total = max_over_ranks(marks[0].elapsed_time(marks[-1]), world, "cuda")
    per_step = [marks[i].elapsed_time(marks[i + 1]) for i in range(a.steps)]
    phase, calls = b.phase_ms()
    b.set_profiling(False)
    b.device_status()
    launches_per_step, per_phase = b.last_launch_count()
    serial = phase                                      # the phases of a call run one after the other on the call's stream
    # whole calls of the two panel modes, alternating in one loop (same clocks, same temperature for both)
    ab = None
    if a.ab_calls > 0:
        pairs = {8: [], 1: []}
        for _ in range(a.ab_calls):
            for panels in (8, 1):
                b.debug_set_overlap(panels == 8)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                step()
                e1.record(stream)
                pairs[panels].append((e0, e1))
        b.debug_set_overlap(False)
        torch.cuda.synchronize()
        b.device_status()
        t = {p: [x.elapsed_time(y) for x, y in v] for p, v in pairs.items()}
        ab = {"calls_per_mode": a.ab_calls, "overlap_ms_median": float(np.median(t[8])), "overlap_ms_best": float(min(t[8])),
              "serial_ms_median": float(np.median(t[1])), "serial_ms_best": float(min(t[1])),
              "note": "whole calls of the two modes alternating call by call: post-processing of a panel on a second stream beside the "
                      "next panel's GEMMs (gemm2m_debug_set_overlap(1)) against every kernel on the caller's stream, in order (default)"}

    # ---- end to end.  zgemm: the library's call on HOST operands (zgemm2m_host): every step uploads A and B from pinned host
    # memory, runs the whole path and downloads C inside the one C-ABI call (A first, B in column panels whose kernels run
    # while the next panel is on the bus, every finished panel of C down beside the next panel's work).  The other entry
    # points have no host form: their step is upload (pinned, asynchronous), the device call, download, on one stream.
    e2e = None
    if not a.no_e2e:
        def run_e2e(nsteps):
            for _ in range(nsteps):
                if host_form:
                    b.zgemm2m_host(hA.t(), hB.t(), hC.t(), nmod, stream)
                else:
                    dA.copy_(hA, non_blocking=True)
                    if dB is not None:
                        dB.copy_(hB, non_blocking=True)
                    step()
                    hC.copy_(dC, non_blocking=True)

        run_e2e(2)
        b.device_status()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        run_e2e(a.steps)
        e1.record(stream)
        barrier()
        b.device_status()
        ms_e2e = max_over_ranks(e0.elapsed_time(e1), world, "cuda")
        if not bool(torch.equal(hC.cuda(), dC)):           # the end-to-end form must reproduce the device form bit for bit
            raise RuntimeError("end-to-end result and device result disagree")
        e2e = {"value": job_value(flops_of(a), world, ms_e2e / a.steps), "unit": UNIT,
               "h2d_bytes_per_step": int(hA.numel() * esize + (0 if herk else hB.numel() * esize)), "d2h_bytes_per_step": int(hC.numel() * esize),
               "ms_per_step": ms_e2e / a.steps,
               "pipeline": ("one zgemm2m_host call per step on pinned host buffers: upload of A, then per column panel of B upload, residues, "
                            "GEMMs, post-processing and download of that panel of C (copies on two library streams)") if host_form else
                           "per step: asynchronous upload of the operands from pinned host buffers, the device call, download of C; one stream"}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    ms_step = ms_total / a.steps
    value = job_value(flops_of(a), world, ms_step)
    planes = nmod if herk else 2 * min(nmod, 22) + 3 * max(nmod - 22, 0)      # real int8 GEMMs per call
    gemm_launches = max(per_phase[2], 1)               # one launch per panel, each all the real GEMMs of its panel
    gemm_ops = 2.0 * planes * m * n * k / gemm_launches   # int8 multiply-adds x2
    gemm_tops = gemm_ops * gemm_launches / (phase[2] * 1e-3) / 1e12
    int8_peak = INT8_OVER_BF16 * peaks["bf16_sustained"]
    c_kp, c_ldp = (k + 127) // 128 * 128, (m + 15) // 16 * 16
    if herk:
        scan_bytes, pre_bytes, post_bytes = n * k * 16, n * k * (16 + 2 * nmod), n * (n + 1) // 2 * (2 * nmod + 16)
    else:
        scan_bytes, pre_bytes, post_bytes = (m * k + k * n) * esize, (m * k + k * n) * (esize + planes), m * n * (planes + esize)
    sm_ghz = (clocks.get("sm_mhz") or 0.0) / 1000.0
    roofline = {"bound": "tensor", "kernel": "gemm_i8_tcgen05_pair_kernel", "achieved": gemm_tops, "peak": int8_peak, "unit": "TFLOP/s",
                "frac": gemm_tops / int8_peak,
                "traffic": GEMM_DRAM_BYTES_PER_PLANE_BYTE * planes * (m * c_kp + (n * c_kp + n * c_ldp) / gemm_launches),
                "traffic_source": "ncu dram__bytes_read+write of one panel launch at 4096^3, scaled by the plane bytes a launch touches",
                "peak_source": f"2 x {peaks['source']} sustained bf16 cuBLAS rate (int8:bf16 nominal ratio); int8 ops counted as 2 per MAC",
                "frac_of_measured_2x_bf16_sustained": gemm_tops / int8_peak,
                "frac_of_measured_2x_bf16_burst": gemm_tops / (INT8_OVER_BF16 * peaks["bf16_burst"]),
                "frac_of_nominal_4500": gemm_tops / INT8_NOMINAL_TOPS,
                "gemm_ms_x_sm_ghz": phase[2] * sm_ghz if sm_ghz else None,
                "clock_note": "the GEMM phase runs at the board's power limit; gemm_ms_x_sm_ghz (GEMM milliseconds per call times the median "
                              "SM clock sampled under load) compares runs taken at different clocks",
                "launch_ms": phase[2] / gemm_launches, "launches_per_step": gemm_launches, "algorithmic_ops_per_launch": gemm_ops}
    gbs = lambda nbytes, ms: nbytes / (ms * 1e-3) / 1e9 if ms > 0 else None
    phases = {"note": "kernel time per phase and call in the timed region (events recorded by the library around every launch on "
                      "the call's stream; the phases run one after the other)",
              "scan_ms": phase[0], "residues_ms": phase[1], "gemm_ms": phase[2], "post_ms": phase[3], "calls_averaged": calls}
    phases_serial = {"note": "the same phase times as bytes per second: algorithmic bytes of the phase over its kernel time",
                     "scan_ms": serial[0], "residues_ms": serial[1], "gemm_ms": serial[2], "post_ms": serial[3],
                     "scan_gbs": gbs(scan_bytes, serial[0]), "residues_gbs": gbs(pre_bytes, serial[1]), "post_gbs": gbs(post_bytes, serial[3]),
                     "hbm_peak_gbs": peaks["hbm_gbs"], "hbm_peak_source": peaks["source"]}
    for key in ("scan", "residues", "post"):
        g = phases_serial[key + "_gbs"]
        phases_serial[key + "_frac_of_hbm"] = g / peaks["hbm_gbs"] if g else None
    cpu = None
    if not a.no_cpu_baseline:
        cpu, _ = time_oracle(a, *oracle_operands(a, A, B), a.cpu_seconds)
    line = {"metric": a.metric, "value": value, "unit": UNIT, "n_gpus": world, "steps": a.steps, "warmup": max(a.warmup, 3),
            "ms_per_step": ms_step, "ms_per_step_median": float(np.median(per_step)), "ms_per_step_best": float(min(per_step)),
            "ms_per_step_serial": ab["serial_ms_median"] if ab else None, "ms_per_step_overlap": ab["overlap_ms_median"] if ab else None,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8",
            "data": "synthetic",
            "config": {"workload": workload_name(a),
                       "l2": "operands (%.2f GiB) and residue planes exceed the 126 MB L2" % ((m * k + (0 if herk else k * n)) * esize / 2**30),
                       "multi_gpu": "replicas only (no collective on the path)"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * a.steps, "launches_per_step": per_phase,
            "roofline": roofline, "phases": phases, "phases_serial": phases_serial, "panel_overlap_ab": ab, "cpu_baseline": cpu}
    print(json.dumps(line))
    b.set_workspace(None)
    if world > 1:
        dist.destroy_process_group()


def main():
    a = parse()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)


if __name__ == "__main__":
    main()
