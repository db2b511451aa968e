"""Benchmark of the zgemm2m hot path (2M multiplication + Ozaki-II) on B200.

One step = one zgemm2m call (exponent scan, quantise + residues, 2N int8 GEMMs, post-processing) on a synthetic
complex128 problem.  Prints ONE JSON line (rank 0).  See --help for the workload knobs; the defaults are the
headline configuration: m = n = k = 8192, 16 moduli, inputs (rand-0.5)*exp(0.5*randn).

  python bench.py                          # this library, 1 GPU
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

METRIC = "zgemm2m_effective_tflops_8mnk_per_t"
UNIT = "TFLOP/s"
INT8_NOMINAL_TOPS = 4500.0          # dense int8, nominal
INT8_OVER_BF16 = 2.0                # nominal ratio used to turn the measured bf16 peak into an int8 peak
# DRAM bytes (read + write) of a GEMM launch per byte of the int8 planes it touches, from the ncu capture of one panel launch of
# the 4096^3, 16-modulus case (profiles/gemm_i8_tcgen05_pair_4096_nmod16.md): (673.9 + 123.9) MB over 805.3 MB of planes.
GEMM_DRAM_BYTES_PER_PLANE_BYTE = (673.872384e6 + 123.916288e6) / (32 * 4096 * (4096 + 1024 + 1024))


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
    ap.add_argument("--m", type=int, default=8192)
    ap.add_argument("--n", type=int, default=8192)
    ap.add_argument("--k", type=int, default=8192)
    ap.add_argument("--nmod", type=int, default=16)
    ap.add_argument("--phi", type=float, default=0.5)
    ap.add_argument("--seed", type=int, default=1)
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="target CPU time of the oracle sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    return ap.parse_args()


def workload_name(a):
    return f"zgemm2m complex128 m={a.m} n={a.n} k={a.k} nmod={a.nmod} parts=(rand-0.5)*exp({a.phi}*randn)"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_burst=float(d["bf16_tflops"]),
                    bf16_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


# ----------------------------------------------------------------------------------------------- CPU oracle leg
def time_oracle(a, A, B, seconds):
    """Times the double-double 4M oracle, as it stands, on a bounded sample of entries of the same product."""
    from oracle import direct
    from paper_2609_05419_b200 import inputs
    cores = direct.num_threads()
    probe = inputs.sample_indices(a.m, a.n, 2048, seed=11)
    t0 = time.perf_counter()
    direct.zgemm4m_dd_samples(A, B, probe)
    t_probe = max(time.perf_counter() - t0, 1e-6)
    count = int(min(max(len(probe), len(probe) * seconds / t_probe), a.m * a.n))
    pairs = inputs.sample_indices(a.m, a.n, count, seed=12)
    t0 = time.perf_counter()
    direct.zgemm4m_dd_samples(A, B, pairs)
    dt = time.perf_counter() - t0
    flops = 8.0 * a.k * len(pairs)
    return dict(value=flops / dt / 1e12, unit=UNIT, cores=cores, kind="oracle",
                sample=f"{len(pairs)} sampled entries of the {a.m}x{a.n}x{a.k} product (double-double 4M, {dt:.1f} s)"), dt


def run_reference(a):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2609_05419_b200 import inputs
    A, B = inputs.complex_inputs(a.m, a.n, a.k, a.seed, dist="phi", phi=a.phi)
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
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": a.gpus, "steps": a.steps,
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
    from paper_2609_05419_b200 import inputs

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
    A, B = inputs.complex_inputs(m, n, k, a.seed + rank, dist="phi", phi=a.phi)     # every replica its own problem
    # pinned host buffers in column-major order (the transposed view is what the C ABI sees)
    hA = torch.from_numpy(np.ascontiguousarray(A.T)).pin_memory()
    hB = torch.from_numpy(np.ascontiguousarray(B.T)).pin_memory()
    hC = torch.empty((n, m), dtype=torch.complex128).pin_memory()
    dA, dB = hA.cuda(), hB.cuda()
    dC = torch.empty((n, m), dtype=torch.complex128, device="cuda")
    ws_op = b.OP_ZGEMM if a.no_e2e else b.OP_ZGEMM_HOST      # the host form's workspace is zgemm2m's plus device copies of A, B, C
    ws = torch.zeros(b.workspace_bytes(ws_op, m, n, k, nmod), dtype=torch.uint8, device="cuda")
    b.set_workspace(ws)
    stream = torch.cuda.current_stream()

    def step():
        b.zgemm2m(dA.t(), dB.t(), dC.t(), nmod, stream)

    for _ in range(max(a.warmup, 3)):
        step()
    b.device_status()

    # ---- timed region: device-resident inputs, phase events recorded on the same stream
    sampler = ClockSampler(local)
    b.set_profiling(True)
    barrier()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(a.steps):
        step()
    e1.record(stream)
    barrier()
    clocks = sampler.stop()
    ms_total = max_over_ranks(e0.elapsed_time(e1), world, "cuda")
    phase, calls = b.phase_ms()
    b.set_profiling(False)
    b.device_status()
    launches_per_step, per_phase = b.last_launch_count()
    # the same phases strictly one after the other (no panel overlap): what the per-phase bandwidth figures are taken from
    b.debug_set_panels(1)
    b.set_profiling(True)
    for _ in range(3):
        step()
    serial, _ = b.phase_ms()
    b.set_profiling(False)
    b.debug_set_panels(8)
    b.device_status()

    # ---- end to end: the library's call on HOST operands (zgemm2m_host).  Every step uploads A and B from pinned host memory,
    # runs the whole path and downloads C, all inside the one C-ABI call: A goes up first, B in column panels whose kernels
    # run while the next panel is on the bus, and every finished panel of C goes down beside the next panel's work.
    e2e = None
    if not a.no_e2e:
        def run_e2e(nsteps):
            for _ in range(nsteps):
                b.zgemm2m_host(hA.t(), hB.t(), hC.t(), nmod, stream)

        run_e2e(2)
        b.device_status()
        barrier()
        e0.record(stream)
        run_e2e(a.steps)
        e1.record(stream)
        barrier()
        b.device_status()
        ms_e2e = max_over_ranks(e0.elapsed_time(e1), world, "cuda")
        same = bool(torch.equal(hC.cuda(), dC))            # the host form must reproduce the device form bit for bit
        if not same:
            raise RuntimeError("zgemm2m_host and zgemm2m disagree")
        e2e = {"value": job_value(8.0 * m * n * k, world, ms_e2e / a.steps), "unit": UNIT,
               "h2d_bytes_per_step": int(hA.numel() * 16 + hB.numel() * 16), "d2h_bytes_per_step": int(hC.numel() * 16),
               "ms_per_step": ms_e2e / a.steps,
               "pipeline": "one zgemm2m_host call per step on pinned host buffers: upload of A, then per column panel of B "
                           "upload, residues, GEMMs, post-processing and download of that panel of C (copies on two library streams)"}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    ms_step = ms_total / a.steps
    value = job_value(8.0 * m * n * k, world, ms_step)
    gemm_launches = max(per_phase[2], 1)               # one launch per column panel, each all 2N real GEMMs of its panel
    gemm_ops = 2.0 * (2 * nmod) * m * n * k / gemm_launches   # int8 multiply-adds x2
    gemm_tops = gemm_ops * gemm_launches / (phase[2] * 1e-3) / 1e12
    int8_peak = INT8_OVER_BF16 * peaks["bf16_sustained"]
    c_kp, c_ldp = (k + 127) // 128 * 128, (m + 15) // 16 * 16
    pre_bytes = (m * k + k * n) * (16 + 2 * nmod)       # quantise read + residue planes written
    scan_bytes = (m * k + k * n) * 16
    post_bytes = m * n * (2 * nmod + 16)
    roofline = {"bound": "tensor", "kernel": "gemm_i8_tcgen05_pair_kernel", "achieved": gemm_tops, "peak": int8_peak, "unit": "TFLOP/s",
                "frac": gemm_tops / int8_peak,
                "traffic": GEMM_DRAM_BYTES_PER_PLANE_BYTE * 2 * nmod * (m * c_kp + (n * c_kp + n * c_ldp) / gemm_launches),
                "traffic_source": "ncu dram__bytes_read+write of one panel launch at 4096^3, scaled by the plane bytes a launch touches",
                "peak_source": f"2 x {peaks['source']} sustained bf16 cuBLAS rate (int8:bf16 nominal ratio); int8 ops counted as 2 per MAC",
                "frac_of_nominal_4500": gemm_tops / INT8_NOMINAL_TOPS,
                "launch_ms": phase[2] / gemm_launches, "launches_per_step": gemm_launches, "algorithmic_ops_per_launch": gemm_ops}
    gbs = lambda nbytes, ms: nbytes / (ms * 1e-3) / 1e9 if ms > 0 else None
    phases = {"note": "sums of kernel durations per phase in the timed region; post-processing of a column panel runs beside the "
                      "next panel's GEMMs, so the phases add up to more than ms_per_step",
              "scan_ms": phase[0], "residues_ms": phase[1], "gemm_ms": phase[2], "post_ms": phase[3], "calls_averaged": calls}
    phases_serial = {"note": "3 extra calls with the panel overlap switched off (phases strictly sequential)",
                     "scan_ms": serial[0], "residues_ms": serial[1], "gemm_ms": serial[2], "post_ms": serial[3],
                     "scan_gbs": gbs(scan_bytes, serial[0]), "residues_gbs": gbs(pre_bytes, serial[1]), "post_gbs": gbs(post_bytes, serial[3]),
                     "hbm_peak_gbs": peaks["hbm_gbs"], "hbm_peak_source": peaks["source"]}
    cpu = None
    if not a.no_cpu_baseline:
        cpu, _ = time_oracle(a, A, B, a.cpu_seconds)
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": a.steps, "warmup": max(a.warmup, 3),
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8",
            "data": "synthetic",
            "config": {"workload": workload_name(a), "l2": "inputs (2 x %.2f GiB) and residue planes exceed the 126 MB L2" % (m * k * 16 / 2**30),
                       "multi_gpu": "replicas only (no collective on the path)"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * a.steps, "launches_per_step": per_phase,
            "roofline": roofline, "phases": phases, "phases_serial": phases_serial, "cpu_baseline": cpu}
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
