#!/usr/bin/env python
"""Benchmark of the AWE exact integer matrix product on B200.

One "step" is one pass of the whole hot path over one batch: encode A, encode B, the r FP4
GEMMs with the fused integer reconstruction.  The default workload is the one the headline
metric is quoted on: INT8 x INT8 at M = N = K = 8192 with the 6-product encoding.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` is effective exact-INT8 TOPS = 2 M N K / t with inputs
resident in HBM; `e2e` is the same metric through awe_gemm_exact_host with pinned HOST buffers
(host<->device copies inside the timed region); `roofline` describes the dominant kernel (the
FP4 GEMM) against the FP4 tensor peak; `cpu_baseline` is the CPU oracle timed on a bounded
sample of the same workload on this machine's cores.  With --gpus N > 1 (under torchrun) every
rank runs an independent replica of the workload: the path has no exchange step.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "effective exact INT8xINT8 TOPS (2*M*N*K / time), AWE 6-GEMM"
NOMINAL_FP4_TFLOPS = 9000.0          # published dense FP4 peak of one B200 (paper, Section 6.2)
NOMINAL_FP4_OVER_BF16 = 4.0          # 9.0 / 2.25 PFLOP/s nominal
GEMM_TRAFFIC_JSON = os.path.join(ROOT, "profiles", "awe_gemm_kernel_8192_awe6_traffic.json")
GEMM_KERNEL_SOURCES = ["awe_gemm.cu", "gemm_common.cuh", "ptx.cuh"]
BURST_REGION_S = 0.1                 # the power regulator pulls the clock down within 0.1-0.4 s (a 0.39 s run already sits at 1.30 GHz)
MAC_PER_CLK_PER_SM = 16384           # dense FP4: 4 x the 4096 bf16 MAC/clk/SM of the tcgen05 pipe


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def gemm_sources_hash():
    """sha256 over the sources of the product kernel: ties a stored ncu figure to the code it measured."""
    import hashlib
    hsh = hashlib.sha256()
    for f in GEMM_KERNEL_SOURCES:
        hsh.update(open(os.path.join(ROOT, "paper_2609_24519_b200", "csrc", f), "rb").read())
    return hsh.hexdigest()[:16]


def gemm_dram_traffic(M, N, K, encoding):
    """dram__bytes_read.sum + dram__bytes_write.sum of one product launch from the committed ncu
    capture, or None when the capture is of another workload or of older kernel sources."""
    try:
        d = json.load(open(GEMM_TRAFFIC_JSON))
    except Exception:
        return None, "no capture on file"
    if (d.get("M"), d.get("N"), d.get("K"), d.get("encoding")) != (M, N, K, encoding):
        return None, "the capture on file is of another workload"
    if d.get("sources_sha256_16") != gemm_sources_hash():
        return None, "kernel sources changed since the capture on file (%s)" % d.get("summary")
    return int(d["dram_bytes_read"]) + int(d["dram_bytes_write"]), \
        "dram__bytes_read.sum + dram__bytes_write.sum of one launch at this workload (%s)" % d.get("summary")


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed regions run."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting"}

    def __init__(self, index: int, uuid: str = ""):
        self.by_region, self.max_mhz = {}, None
        self._stop = threading.Event()
        self._active = threading.Event()
        self._region = None
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            try:
                self._dev = pynvml.nvmlDeviceGetHandleByUUID(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
            except Exception:
                self._dev = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._dev, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            if self._active.is_set():
                rec = self.by_region.setdefault(self._region, {"mhz": [], "reasons": set(), "power": []})
                try:
                    rec["mhz"].append(nv.nvmlDeviceGetClockInfo(self._dev, nv.NVML_CLOCK_SM))
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self._dev)
                    for bit, name in self.REASONS.items():
                        if mask & bit:
                            rec["reasons"].add(name)
                    rec["power"].append(nv.nvmlDeviceGetPowerUsage(self._dev) / 1000.0)
                except Exception:
                    pass
            time.sleep(0.001)

    def start(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def region(self, name):
        """Samples taken from now on belong to region `name`; None pauses sampling."""
        if name is None:
            self._active.clear()
        else:
            self._region = name
            self._active.set()

    def summary(self, name):
        rec = self.by_region.get(name, {"mhz": [], "reasons": set(), "power": []})
        return {"sm_mhz": statistics.median(rec["mhz"]) if rec["mhz"] else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(rec["reasons"]), "samples": len(rec["mhz"]),
                "power_w_max": max(rec["power"]) if rec["power"] else None}

    def stop(self):
        self._stop.set()
        if self._thread:
            self._thread.join()


def cpu_oracle_sample(A, B, budget_s: float):
    """Time the CPU oracle (plain int64 product) on the first rows of the workload; the number
    of rows is chosen from a 2-row probe so the run takes about budget_s seconds."""
    from oracle import matmul as om
    om.build()
    M, K = A.shape
    N = B.shape[1]
    t0 = time.perf_counter()
    om.matmul_i64_rows(A, B, 0, min(2 * om.threads(), M))
    probe = (time.perf_counter() - t0) / min(2 * om.threads(), M)
    rows = int(max(om.threads(), min(M, budget_s / max(probe, 1e-9))))
    t0 = time.perf_counter()
    c_rows = om.matmul_i64_rows(A, B, 0, rows)
    dt = time.perf_counter() - t0
    return {"value": 2.0 * rows * N * K / dt / 1e12, "unit": "TOPS", "cores": om.threads(), "kind": "oracle",
            "sample": f"rows 0..{rows - 1} of the {M}x{N}x{K} product ({dt:.1f} s)"}, rows, dt, c_rows


def run_reference(args, w, rank):
    """The reference arm is the CPU oracle as it stands, on this machine's cores."""
    if rank != 0:
        return
    from paper_2609_24519_b200 import workloads as wl
    from oracle import matmul as om
    om.build()
    A, B = wl.make_inputs(w)
    per_step = max(0.3, min(3.0, 150.0 / max(1, args.steps + args.warmup)))
    _, rows, dt, _ = cpu_oracle_sample(A, B, per_step)
    for _ in range(args.warmup):
        om.matmul_i64_rows(A, B, 0, rows)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        om.matmul_i64_rows(A, B, 0, rows)
    dt = (time.perf_counter() - t0) / args.steps
    value = 2.0 * rows * w.N * w.K / dt / 1e12
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "TOPS", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int64", "data": "synthetic",
            "config": {"workload": w.name, "M": w.M, "N": w.N, "K": w.K,
                       "note": "CPU oracle; each step is a bounded row sample of the workload"},
            "cpu_baseline": {"value": value, "unit": "TOPS", "cores": om.threads(), "kind": "oracle",
                             "sample": f"rows 0..{rows - 1} of {w.M} per step"},
            "e2e": {"value": value, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--size", type=int, default=8192, help="M = N = K of the headline workload")
    ap.add_argument("--encoding", default="awe6", choices=["awe6", "awe6_alt", "base13", "mixed", "derived"],
                    help="INT8xINT8 record of the timed step (the headline metric is awe6)")
    ap.add_argument("--no-extras", action="store_true", help="skip the context measurements")
    ap.add_argument("--context", default="all",
                    help="comma list of context measurements to run: sustained, base13, mixed, derived, int8, configs, ceiling, "
                         "reconstruct (default: all)")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle baseline")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    from paper_2609_24519_b200 import workloads as wl
    w = wl.headline(args.size)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, w, rank)
        return

    import numpy as np
    import torch
    import torch.distributed as dist

    from paper_2609_24519_b200 import binding as b

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    from paper_2609_24519_b200 import replicas

    def barrier():
        replicas.barrier(dev)

    h = b.awe_create(local_rank)
    enc, enc_name = {"awe6": (b.ENC_INT8_AWE6, "int8_awe6"), "awe6_alt": (b.ENC_INT8_AWE6_ALT, "int8_awe6_alt"),
                     "base13": (b.ENC_INT8_BASE13_9, "int8_base13_9"),
                     "mixed": (b.ENC_INT8_MIXED_FP8_3, "int8_mixed_2fp8_1fp4"),
                     "derived": (b.ENC_INT8_AWE6_DERIVED, "int8_awe6_sum_planes_formed_in_kernel")}[args.encoding]
    M, N, K = w.M, w.N, w.K
    A, B = wl.make_inputs(w)
    dA, dB = torch.from_numpy(A).to(dev), torch.from_numpy(B).to(dev)
    C = torch.empty((M, N), dtype=torch.int32, device=dev)
    nA = b.awe_planes_bytes(enc, 0, b.SIDE_A, M, K)
    ws = torch.empty(b.awe_workspace_bytes(enc, 0, M, N, K), dtype=torch.uint8, device=dev)
    pa, pb = ws[:nA], ws[(nA + 255) // 256 * 256:]
    desc = b.awe_encoding_info(enc)

    def step(events=None):
        if events is not None:
            events[0].record()
        b.awe_encode(h, enc, 0, b.SIDE_A, dA, b.I8, b.ROWMAJOR_RxK, M, K, K, pa)
        b.awe_encode(h, enc, 0, b.SIDE_B, dB, b.I8, b.ROWMAJOR_KxR, N, K, N, pb)
        if events is not None:
            events[1].record()
        b.awe_gemm_planes(h, enc, 0, pa, pb, M, N, K, C, b.C_I32, N)
        if events is not None:
            events[2].record()

    # ---- consistency of the entry points (outside every timed region; the comparison with the CPU
    # oracle happens in the cpu_baseline leg below, on the rows that leg computes anyway)
    step()
    torch.cuda.synchronize()
    parity_ok = True
    # the single-call entry point must give the same matrix as the three calls
    C2 = torch.empty_like(C)
    b.awe_gemm_exact(h, dA, b.I8, dB, b.I8, M, N, K, enc, 0, C2, b.C_I32, ws)
    torch.cuda.synchronize()
    parity_ok = parity_ok and bool(torch.equal(C, C2)) and b.awe_last_device_status(h) == (0, 0)

    sampler = ClockSampler(local_rank, str(getattr(torch.cuda.get_device_properties(dev), "uuid", "")))
    sampler.start()

    # ---- device-resident timing
    for _ in range(args.warmup):
        step()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = b.awe_launch_count(h)
    barrier()
    sampler.region("device_resident")
    t_start.record()
    for i in range(args.steps):
        step(evs[i])
    t_end.record()
    barrier()
    sampler.region(None)
    launches = b.awe_launch_count(h) - launches0
    ops = 2.0 * M * N * K
    ms_total, ops_all_ranks = replicas.aggregate(t_start.elapsed_time(t_end), ops * args.steps, dev)
    ms_step = ms_total / args.steps
    enc_ms = [e[0].elapsed_time(e[1]) for e in evs]
    gemm_ms = [e[1].elapsed_time(e[2]) for e in evs]
    step_ms = [e[0].elapsed_time(e[2]) for e in evs]
    ms_encode, ms_gemm = statistics.mean(enc_ms), statistics.mean(gemm_ms)
    assert b.awe_last_device_status(h) == (0, 0)
    gemm_mhz = b.awe_last_gemm_clock_mhz(h)       # SM clock measured inside the last timed GEMM launch

    # ---- end to end from pinned host buffers through awe_gemm_exact_host
    Ah, Bh = torch.from_numpy(A).pin_memory(), torch.from_numpy(B).pin_memory()
    Ch = torch.empty((M, N), dtype=torch.int32).pin_memory()
    scratch = torch.empty(b.awe_workspace_bytes(enc, 0, M, N, K) + b.awe_host_staging_bytes(enc, 0, M, N, K, b.C_I32),
                          dtype=torch.uint8, device=dev)
    e2e_steps = max(3, min(args.steps, 20))
    for _ in range(3):
        b.awe_gemm_exact_host(h, Ah, b.I8, Bh, b.I8, M, N, K, enc, 0, Ch, b.C_I32, scratch)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.region("e2e")
    e0.record()
    for _ in range(e2e_steps):
        b.awe_gemm_exact_host(h, Ah, b.I8, Bh, b.I8, M, N, K, enc, 0, Ch, b.C_I32, scratch)
    e1.record()
    barrier()
    sampler.region(None)
    ms_e2e_total, ops_e2e_all = replicas.aggregate(e0.elapsed_time(e1), ops * e2e_steps, dev)
    ms_e2e = ms_e2e_total / e2e_steps
    parity_ok = parity_ok and bool(torch.equal(Ch, C.cpu()))
    sampler.stop()
    clocks = sampler.summary("device_resident")
    clocks["sm_mhz_in_gemm_kernel"] = gemm_mhz
    clocks["e2e_region"] = sampler.summary("e2e")
    clocks["note"] = ("sm_mhz, reasons, power: NVML samples (1 ms apart) during the device-resident timed region; "
                      "e2e_region: the same for the host-buffer region; sm_mhz_in_gemm_kernel: SM cycles / wall "
                      "time measured inside the last timed GEMM launch")

    sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
    peaks = measured_peaks()
    # Denominator: the peaks file has no FP4 entry, so the measured bf16 figure is scaled by the nominal
    # fp4 : bf16 ratio -- the burst figure when the timed region is too short for the power regulator to
    # act, the sustained one for a long region.  Both fractions are printed by name as well.
    region_s = ms_total * 1e-3
    burst = region_s < BURST_REGION_S
    peak_key = "bf16_tflops" if burst else "bf16_tflops_sustained"
    fp4_peak = peaks[peak_key] * NOMINAL_FP4_OVER_BF16
    gemm_tflops = desc.r * ops / (ms_gemm * 1e-3) / 1e12
    plane_bytes = b.awe_planes_bytes(enc, 0, b.SIDE_A, M, K) + b.awe_planes_bytes(enc, 0, b.SIDE_B, N, K)
    # an FP8 product runs at half the FP4 peak: the peak of a record is its flops over its ideal time
    fp4_equiv = sum(2 if desc.fp8[k] else 1 for k in range(desc.r))
    fmt_scale = desc.r / fp4_equiv  # 1 for FP4-only records
    fp4_peak = fp4_peak * fmt_scale
    traffic, traffic_note = gemm_dram_traffic(M, N, K, args.encoding)
    line = {
        "metric": METRIC, "value": ops_all_ranks / (ms_total * 1e-3) / 1e12, "unit": "TOPS", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "e2m1 (fp4) operands, f32 accumulate, int32 reconstruction",
        "data": "synthetic",
        "config": {"workload": w.name, "M": M, "N": N, "K": K, "encoding": enc_name, "fp4_gemms": desc.r - sum(desc.fp8[k] for k in range(desc.r)),
                   "fp8_gemms": sum(desc.fp8[k] for k in range(desc.r)),
                   "inputs": "int8 uniform [-128,127], numpy default_rng(seed=6)", "output": "int32",
                   "l2": "no flush: per-step working set (%d+%d MiB in, %d MiB planes, %d MiB out) exceeds the 126 MB L2"
                         % (M * K >> 20, K * N >> 20, plane_bytes >> 20, M * N * 4 >> 20),
                   "parallelism": "replicas only (no exchange step)" if world > 1 else "single GPU"},
        "clocks": clocks,
        "e2e": {"value": ops_e2e_all / (ms_e2e_total * 1e-3) / 1e12, "unit": "TOPS", "ms_per_step": ms_e2e,
                "steps": e2e_steps, "h2d_bytes_per_step": int(A.nbytes + B.nbytes), "d2h_bytes_per_step": int(M * N * 4)},
        "gpu_launches": int(launches),
        "parity": "3-call path == awe_gemm_exact == host path" if parity_ok else "MISMATCH between entry points",
        "kernels_ms": {"encode_a_plus_b": ms_encode, "gemm_and_reconstruction": ms_gemm,
                       "per_step_stats": {name: {"mean": statistics.mean(v), "median": statistics.median(v), "best": min(v)}
                                          for name, v in (("encode_a_plus_b", enc_ms), ("gemm_and_reconstruction", gemm_ms),
                                                          ("step", step_ms))}},
        "roofline": {"bound": "tensor", "achieved": gemm_tflops, "peak": fp4_peak, "unit": "TFLOP/s",
                     "frac": gemm_tflops / fp4_peak, "traffic": traffic, "traffic_note": traffic_note,
                     "kernel": "awe_gemm_kernel", "flops_per_launch": desc.r * ops,
                     "peak_source": "%s %s %.1f TFLOP/s x nominal fp4:bf16 ratio 4 (timed region %.3f s: %s)" %
                                    (peaks["source"], peak_key, peaks[peak_key], region_s,
                                     "burst" if burst else "sustained"),
                     "frac_of_sustained_peak": gemm_tflops / (peaks["bf16_tflops_sustained"] * NOMINAL_FP4_OVER_BF16 * fmt_scale),
                     "frac_of_nominal_9pflops": gemm_tflops / (NOMINAL_FP4_TFLOPS * fmt_scale),
                     "frac_of_pipe_peak_at_delivered_clock":
                         gemm_tflops / (fmt_scale * MAC_PER_CLK_PER_SM * 2 * sm_count * gemm_mhz * 1e6 / 1e12) if gemm_mhz else None,
                     "frac_of_burst_peak": gemm_tflops / (peaks["bf16_tflops"] * NOMINAL_FP4_OVER_BF16 * fmt_scale)},
        "encode_roofline": {"bound": "hbm", "achieved": (M * K + K * N + plane_bytes) / (ms_encode * 1e-3) / 1e9,
                            "peak": peaks["hbm_gbs"], "unit": "GB/s"},
    }
    line["encode_roofline"]["frac"] = line["encode_roofline"]["achieved"] / peaks["hbm_gbs"]

    def want(name):
        return args.context == "all" or name in args.context.split(",")

    # the context measurements are single-GPU work: in a multi-GPU run every rank finishes at the same time
    if rank == 0 and world == 1 and not args.no_extras:
        ctx = {}
        if want("sustained"):
            # the same step 300 times back to back (about 0.4 s): long enough for the power regulator to settle,
            # reported beside the burst figure of the timed region above
            for _ in range(3):
                step()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(300):
                step()
            e1.record()
            torch.cuda.synchronize()
            ms300 = e0.elapsed_time(e1) / 300
            ctx["sustained_300_steps"] = {"TOPS": ops / (ms300 * 1e-3) / 1e12, "ms_per_step": ms300,
                                          "sm_mhz_in_gemm_kernel": b.awe_last_gemm_clock_mhz(h)}
            time.sleep(1.0)  # let the part cool before the next short measurement
        if want("base13"):
            # prior-work 9-GEMM base-13 scheme through the same kernels, same inputs
            enc9 = b.ENC_INT8_BASE13_9
            ws9 = torch.empty(b.awe_workspace_bytes(enc9, 0, M, N, K), dtype=torch.uint8, device=dev)
            C9 = torch.empty_like(C)
            for _ in range(2):
                b.awe_gemm_exact(h, dA, b.I8, dB, b.I8, M, N, K, enc9, 0, C9, b.C_I32, ws9)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(5):
                b.awe_gemm_exact(h, dA, b.I8, dB, b.I8, M, N, K, enc9, 0, C9, b.C_I32, ws9)
            e1.record()
            torch.cuda.synchronize()
            ctx["base13_9gemm_TOPS"] = ops / (e0.elapsed_time(e1) / 5 * 1e-3) / 1e12
            ctx["base13_equals_awe6"] = bool(torch.equal(C9, C))
            parity_ok = parity_ok and ctx["base13_equals_awe6"]
            del ws9, C9
        if want("mixed"):
            # mixed 2 x FP8 + 1 x FP4 construction (Appendix A) on the same inputs: whole call and its product kernel
            encm = b.ENC_INT8_MIXED_FP8_3
            wsm = torch.empty(b.awe_workspace_bytes(encm, 0, M, N, K), dtype=torch.uint8, device=dev)
            Cm = torch.empty_like(C)
            for _ in range(3):
                b.awe_gemm_exact(h, dA, b.I8, dB, b.I8, M, N, K, encm, 0, Cm, b.C_I32, wsm)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(10):
                b.awe_gemm_exact(h, dA, b.I8, dB, b.I8, M, N, K, encm, 0, Cm, b.C_I32, wsm)
            e1.record()
            torch.cuda.synchronize()
            ctx["mixed_2fp8_1fp4_TOPS"] = ops / (e0.elapsed_time(e1) / 10 * 1e-3) / 1e12
            nAm = b.awe_planes_bytes(encm, 0, b.SIDE_A, M, K)
            pam, pbm = wsm[:nAm], wsm[(nAm + 255) // 256 * 256:]
            e0.record()
            for _ in range(10):
                b.awe_gemm_planes(h, encm, 0, pam, pbm, M, N, K, Cm, b.C_I32, N, 0)
            e1.record()
            torch.cuda.synchronize()
            ctx["mixed_2fp8_1fp4_products_ms"] = e0.elapsed_time(e1) / 10
            ctx["mixed_sm_mhz"] = b.awe_last_gemm_clock_mhz(h)
            ctx["mixed_equals_awe6"] = bool(torch.equal(Cm, C))
            parity_ok = parity_ok and ctx["mixed_equals_awe6"]
            del wsm, Cm, pam, pbm
        if want("derived") and args.encoding != "derived":
            # the same record with its sum planes formed inside the product kernel (Section 6.1's alternative)
            encd = b.ENC_INT8_AWE6_DERIVED
            wsd = torch.empty(b.awe_workspace_bytes(encd, 0, M, N, K), dtype=torch.uint8, device=dev)
            Cd = torch.empty_like(C)
            nAd = b.awe_planes_bytes(encd, 0, b.SIDE_A, M, K)
            pad, pbd = wsd[:nAd], wsd[(nAd + 255) // 256 * 256:]
            e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            for it_ in range(4):            # the first pass warms up, the last three are timed
                if it_ == 1:
                    torch.cuda.synchronize()
                    enc_d, prod_d = [], []
                e0.record()
                b.awe_encode(h, encd, 0, b.SIDE_A, dA, b.I8, b.ROWMAJOR_RxK, M, K, K, pad)
                b.awe_encode(h, encd, 0, b.SIDE_B, dB, b.I8, b.ROWMAJOR_KxR, N, K, N, pbd)
                e1.record()
                b.awe_gemm_planes(h, encd, 0, pad, pbd, M, N, K, Cd, b.C_I32, N, 0)
                e2.record()
                torch.cuda.synchronize()
                if it_ >= 1:
                    enc_d.append(e0.elapsed_time(e1))
                    prod_d.append(e1.elapsed_time(e2))
            ctx["sum_planes_formed_in_kernel"] = {
                "encode_a_plus_b_ms": statistics.mean(enc_d), "products_ms": statistics.mean(prod_d),
                "TOPS": ops / ((statistics.mean(enc_d) + statistics.mean(prod_d)) * 1e-3) / 1e12,
                "plane_bytes": int(b.awe_workspace_bytes(encd, 0, M, N, K)), "equals_awe6": bool(torch.equal(Cd, C))}
            parity_ok = parity_ok and ctx["sum_planes_formed_in_kernel"]["equals_awe6"]
            del wsd, Cd, pad, pbd
        if want("int8"):
            # INT8 tensor-core GEMM of the same product (library reference point)
            try:
                for _ in range(2):
                    Ci = torch._int_mm(dA, dB)
                torch.cuda.synchronize()
                e0.record()
                for _ in range(5):
                    Ci = torch._int_mm(dA, dB)
                e1.record()
                torch.cuda.synchronize()
                ctx["int8_tensor_core_gemm_TOPS"] = ops / (e0.elapsed_time(e1) / 5 * 1e-3) / 1e12
                ctx["int8_gemm_equals_awe6"] = bool(torch.equal(Ci, C))
                parity_ok = parity_ok and ctx["int8_gemm_equals_awe6"]
                del Ci
            except Exception as ex:  # library reference point only
                ctx["int8_tensor_core_gemm_TOPS"] = None
                ctx["int8_gemm_error"] = str(ex)[:100]
        # the other configurations, device-timed through awe_gemm_exact (context only; their parity is
        # covered by the GPU tests).  Inputs are drawn on the device from a seeded torch generator.
        if want("configs") and (M, N, K) == (8192, 8192, 8192):
            gen = torch.Generator(device=dev)
            gen.manual_seed(7)

            def timed(enc_, mod_, a_, a_dt_, b_, out_dt_, tdt_, m_, n_, k_, iters=5):
                ws_ = torch.empty(b.awe_workspace_bytes(enc_, mod_, m_, n_, k_), dtype=torch.uint8, device=dev)
                c_ = torch.empty((m_, n_), dtype=tdt_, device=dev)
                for _ in range(2):
                    b.awe_gemm_exact(h, a_, a_dt_, b_, b.I8, m_, n_, k_, enc_, mod_, c_, out_dt_, ws_)
                torch.cuda.synchronize()
                e0.record()
                for _ in range(iters):
                    b.awe_gemm_exact(h, a_, a_dt_, b_, b.I8, m_, n_, k_, enc_, mod_, c_, out_dt_, ws_)
                e1.record()
                torch.cuda.synchronize()
                return e0.elapsed_time(e1) / iters

            a4 = torch.randint(-8, 8, (8192, 8192), dtype=torch.int8, device=dev, generator=gen)
            ms = timed(b.ENC_INT4xINT8_AWE4, 0, a4, b.I4_IN_I8, dB, b.C_I32, torch.int32, 8192, 8192, 8192)
            ctx["int4xint8_awe4_8192_TOPS"] = ops / (ms * 1e-3) / 1e12
            del a4
            ax = torch.randint(0, 2, (4096, 16384), dtype=torch.int8, device=dev, generator=gen) * 255 - 128
            bx = torch.randint(0, 2, (16384, 4096), dtype=torch.int8, device=dev, generator=gen) * 255 - 128
            ms = timed(b.ENC_INT8_AWE6, 0, ax.to(torch.int8), b.I8, bx.to(torch.int8), b.C_I64, torch.int64, 4096, 4096,
                       16384)
            ctx["worst_case_4096x4096x16384_int64_TOPS"] = 2.0 * 4096 * 4096 * 16384 / (ms * 1e-3) / 1e12
            del ax, bx
            # width-12 integers (FP16 significands), 12 products, 64-bit reconstruction
            a12 = torch.randint(-2047, 2048, (8192, 8192), dtype=torch.int16, device=dev, generator=gen)
            b12 = torch.randint(-2047, 2048, (8192, 8192), dtype=torch.int16, device=dev, generator=gen)
            ws12 = torch.empty(b.awe_workspace_bytes(b.ENC_FP16SIG_AWE12, 0, 8192, 8192, 8192), dtype=torch.uint8,
                               device=dev)
            c12 = torch.empty((8192, 8192), dtype=torch.int64, device=dev)
            for _ in range(2):
                b.awe_gemm_exact(h, a12, b.I16, b12, b.I16, 8192, 8192, 8192, b.ENC_FP16SIG_AWE12, 0, c12, b.C_I64, ws12)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(3):
                b.awe_gemm_exact(h, a12, b.I16, b12, b.I16, 8192, 8192, 8192, b.ENC_FP16SIG_AWE12, 0, c12, b.C_I64, ws12)
            e1.record()
            torch.cuda.synchronize()
            ctx["fp16_significand_awe12_8192_TOPS"] = ops / (e0.elapsed_time(e1) / 3 * 1e-3) / 1e12
            # the other significand rows of the paper's table of native formats: FP8 (3 products), BF16 (8)
            for key, enc_s, dt_s, lo, hi, tdt_in, out_s, tdt_out in (
                    ("fp8_significand_3_8192_TOPS", b.ENC_FP8SIG_3, b.I5_IN_I8, -15, 16, torch.int8, b.C_I32, torch.int32),
                    ("bf16_significand_8_8192_TOPS", b.ENC_BF16SIG_8, b.I9_IN_I16, -255, 256, torch.int16, b.C_I32,
                     torch.int32)):
                a_s = torch.randint(lo, hi, (8192, 8192), dtype=tdt_in, device=dev, generator=gen)
                b_s = torch.randint(lo, hi, (8192, 8192), dtype=tdt_in, device=dev, generator=gen)
                ws_s = torch.empty(b.awe_workspace_bytes(enc_s, 0, 8192, 8192, 8192), dtype=torch.uint8, device=dev)
                c_s = torch.empty((8192, 8192), dtype=tdt_out, device=dev)
                for _ in range(2):
                    b.awe_gemm_exact(h, a_s, dt_s, b_s, dt_s, 8192, 8192, 8192, enc_s, 0, c_s, out_s, ws_s)
                torch.cuda.synchronize()
                e0.record()
                for _ in range(5):
                    b.awe_gemm_exact(h, a_s, dt_s, b_s, dt_s, 8192, 8192, 8192, enc_s, 0, c_s, out_s, ws_s)
                e1.record()
                torch.cuda.synchronize()
                ctx[key] = ops / (e0.elapsed_time(e1) / 5 * 1e-3) / 1e12
                del a_s, b_s, ws_s, c_s
            del a12, b12, ws12, c12
            RNS_SET_FP64 = b.awe_wide_moduli()
            total_ms, prods = 0.0, 0
            for m_ in RNS_SET_FP64:
                lo = -(m_ // 2)
                am = torch.randint(lo, lo + m_, (8192, 8192), dtype=torch.int8, device=dev, generator=gen)
                bm = torch.randint(lo, lo + m_, (8192, 8192), dtype=torch.int8, device=dev, generator=gen)
                total_ms += timed(b.ENC_MOD_M, m_, am, b.I8, bm, b.C_RES_I16, torch.int16, 8192, 8192, 8192, iters=2)
                prods += b.awe_encoding_info(b.ENC_MOD_M, m_).r
                del am, bm
            ctx["residue_22_moduli_8192_total_ms"] = total_ms
            ctx["residue_22_moduli_fp4_gemms"] = prods
            # width-54 integers (the FP64 significand) through the residue number system + CRT
            B53 = 2 ** 53 - 1
            aw = torch.randint(-B53, B53 + 1, (8192, 8192), dtype=torch.int64, device=dev, generator=gen)
            bw = torch.randint(-B53, B53 + 1, (8192, 8192), dtype=torch.int64, device=dev, generator=gen)
            wsw = torch.empty(b.awe_wide_workspace_bytes(8192, 8192, 8192), dtype=torch.uint8, device=dev)
            cw = torch.empty((8192, 8192, 2), dtype=torch.int64, device=dev)
            nmod = len(RNS_SET_FP64)
            ra = torch.empty((nmod, 8192 * 8192), dtype=torch.int8, device=dev)
            rc = torch.empty((nmod, 8192 * 8192), dtype=torch.int16, device=dev)
            for _ in range(2):
                b.awe_gemm_exact_wide(h, aw, bw, 8192, 8192, 8192, 54, cw, wsw)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(3):
                b.awe_gemm_exact_wide(h, aw, bw, 8192, 8192, 8192, 54, cw, wsw)
            e1.record()
            torch.cuda.synchronize()
            ms_wide = e0.elapsed_time(e1) / 3
            e0.record()
            for _ in range(3):
                b.awe_wide_residues(h, aw, 8192 * 8192, ra)
            e1.record()
            torch.cuda.synchronize()
            ms_res = e0.elapsed_time(e1) / 3
            e0.record()
            for _ in range(3):
                b.awe_wide_crt(h, rc, 8192 * 8192, cw)
            e1.record()
            torch.cuda.synchronize()
            ms_crt = e0.elapsed_time(e1) / 3
            ctx["wide_int54_8192"] = {"total_ms": ms_wide, "effective_TOPS": ops / (ms_wide * 1e-3) / 1e12,
                                      "residues_one_operand_ms": ms_res, "crt_ms": ms_crt,
                                      "residues_GBs": 8192 * 8192 * (8 + nmod) / (ms_res * 1e-3) / 1e9,
                                      "crt_GBs": 8192 * 8192 * (2 * nmod + 16) / (ms_crt * 1e-3) / 1e9}
            del aw, bw, wsw, cw, ra, rc
        if want("ceiling") and (M, N, K) == (8192, 8192, 8192):
            # FP4 MMA ceiling of this kernel on this part: one raw product on all-zero planes, which
            # draws too little power to be capped, so it shows the structural limit at ~max clock
            kz = 65536
            pz = torch.zeros((8192, kz // 2), dtype=torch.uint8, device=dev)
            pzo = torch.empty((8192, 8192), dtype=torch.float32, device=dev)
            time.sleep(1.5)                      # let the power regulator forget the runs above
            for _ in range(100):
                b.awe_fp4_product_raw(h, pz, pz, 8192, 8192, kz, pzo, 8192)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(10):
                b.awe_fp4_product_raw(h, pz, pz, 8192, 8192, kz, pzo, 8192)
            e1.record()
            torch.cuda.synchronize()
            ceil_tflops = 2.0 * 8192 * 8192 * kz / (e0.elapsed_time(e1) / 10 * 1e-3) / 1e12
            ctx["fp4_ceiling_zero_data_TFLOPs"] = ceil_tflops
            ctx["fp4_ceiling_clock_mhz"] = b.awe_last_gemm_clock_mhz(h)
            line["roofline"]["frac_of_measured_fp4_ceiling"] = gemm_tflops / (ceil_tflops * fmt_scale)
            del pz, pzo
        if want("reconstruct") and (M, N, K) == (8192, 8192, 8192):
            pzo = torch.empty((8192, 8192), dtype=torch.int32, device=dev)
            # stand-alone reconstruction (HBM pass): 6 FP32 product matrices -> int32
            P6 = torch.zeros((6, 8192, 8192), dtype=torch.float32, device=dev)
            for _ in range(2):
                b.awe_reconstruct(h, b.ENC_INT8_AWE6, 0, P6, 8192 * 8192, 8192, 8192, 8192, pzo, b.C_I32, 8192)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(5):
                b.awe_reconstruct(h, b.ENC_INT8_AWE6, 0, P6, 8192 * 8192, 8192, 8192, 8192, pzo, b.C_I32, 8192)
            e1.record()
            torch.cuda.synchronize()
            ctx["standalone_reconstruct_GBs"] = 8192 * 8192 * 28 / (e0.elapsed_time(e1) / 5 * 1e-3) / 1e9
            del P6, pzo
        ctx["paper_theoretical_TOPS"] = "1500 (9.0 PFLOPS / 6, published peak, not a measurement; B200)"
        line["context"] = ctx

    if rank == 0 and world == 1 and not args.no_cpu:
        base, n_rows, _, c_rows = cpu_oracle_sample(A, B, 12.0)
        line["cpu_baseline"] = base
        same = bool(np.array_equal(c_rows, C[:n_rows].cpu().numpy().astype(np.int64)))
        line["parity"] += ("; GPU rows 0..%d bit-exact vs the CPU oracle" % (n_rows - 1)) if same else \
            "; MISMATCH vs the CPU oracle"
        parity_ok = parity_ok and same
        # the textbook (i, j, k) loop nest on one thread, once, at 1024^3
        from oracle import matmul as om
        n1 = min(1024, M, N, K)
        t0 = time.perf_counter()
        c_naive = om.matmul_i64_ijk(A[:n1, :n1], B[:n1, :n1])
        dt = time.perf_counter() - t0
        line["cpu_baseline"]["naive"] = {"value": 2.0 * n1 ** 3 / dt / 1e12, "unit": "TOPS", "cores": 1,
                                         "kind": "oracle, textbook i-j-k loop nest",
                                         "sample": "%d^3 corner of the workload (%.1f s)" % (n1, dt)}
        del c_naive

    elif rank == 0:
        line["cpu_baseline"] = None

    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()
    if not parity_ok:
        raise SystemExit("bench.py: parity mismatch (see the `parity` field)")


if __name__ == "__main__":
    main()
