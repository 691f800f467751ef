#!/usr/bin/env python
"""Benchmark of the emulated DGEMM hot path (Ozaki scheme II on FP4 tensor cores).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--size 16384] [--moduli 19]
    python bench.py --impl reference ...     # times the CPU oracle on a bounded sample

One step = one ozk_dgemm (exponent scan, limb encoding, limb GEMM, CRT) over one pair of
seeded synthetic FP64 matrices.  `value` is the whole-job effective FP64 rate 2MNK/t with the
inputs resident in HBM; `e2e` is the same metric through the C ABI with host buffers, the
host-to-device copies of A and B and the device-to-host copy of C inside the timed region.
With N > 1 every rank runs an independent replica of the same problem (the path has no
exchange step); the time is the maximum over ranks and the value the sum of the work.
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "effective FP64 TFLOPS (2MNK/t), Ozaki scheme II on FP4, end to end incl. preprocessing"
UNIT = "TFLOP/s"
PAPER_TOTAL_TFLOPS = {4096: 10.81, 8192: 13.52, 16384: 15.26}   # the paper's end-to-end numbers, L = 19, other GPU
FP4_PER_BF16 = 4.0                                               # nominal dense FP4 : BF16 ratio on B200
NOMINAL_FP4_TFLOPS = 9000.0                                      # B200 dense FP4 (NVIDIA's doubled figures are 2:4 sparsity)
SM_COUNT = 148
# DRAM traffic of one limb-GEMM launch comes from an ncu capture recorded in this file together with a hash of the
# kernel source it was taken from; a capture of other source is not reported
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "limb_gemm_dram_traffic.json")
GEMM_SOURCES = ["paper_2608_06812_b200/csrc/ozk_gemm.cu", "paper_2608_06812_b200/csrc/ozk_ptx.cuh"]
KERNELS_PER_STEP = 8   # lut, scan_rows, scan_cols, shifts of both operands, encode_rows, encode_cols, limb GEMM, CRT


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--size", type=int, default=16384, help="M = N = K")
    ap.add_argument("--shape", default=None, help="M,N,K of a non-square run (scheme II only; overrides --size; the headline "
                    "metric is quoted on the square default)")
    ap.add_argument("--moduli", type=int, default=19)
    ap.add_argument("--phi", type=float, default=1.0)
    ap.add_argument("--max-bits", type=int, default=53, help="width cap of the converted integers; values above 53 time the "
                    "extended-capacity entry point ozk_dgemm_ext (not the paper's method, not the headline)")
    ap.add_argument("--impl", default="ozk", choices=["ozk", "reference"])
    ap.add_argument("--scheme", default="oz2", choices=["oz2", "oz1", "i8"],
                    help="oz2 = Ozaki scheme II (the headline path); oz1 = Ozaki scheme I, 15 x 15 limbs; "
                         "i8 = INT8 x INT8 -> INT32 GEMM on FP4 limbs (reports integer TOP/s)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-fp64-context", action="store_true")
    ap.add_argument("--karatsuba", action="store_true", help="switch the partial Karatsuba variant on (68 instead of 75 limb products "
                    "at 19 moduli; a measured loss, not the default)")
    ap.add_argument("--launcher-selftest", action="store_true", help="CPU-only check of the multi-rank launch and reduction (no GPU work)")
    return ap.parse_args()


def gemm_source_hash() -> str:
    import hashlib
    h = hashlib.sha256()
    for rel in GEMM_SOURCES:
        h.update(open(os.path.join(ROOT, rel), "rb").read())
    return h.hexdigest()


def recorded_traffic(M: int, N: int, K: int, L: int):
    """(bytes per launch or None, note): the ncu DRAM read + write bytes of one limb-GEMM launch at this size, if a
    capture of the current kernel source is on record."""
    try:
        rec = json.load(open(TRAFFIC_FILE))
    except (OSError, ValueError):
        return None, "no capture on record"
    for c in rec.get("captures", []):
        if [c.get("M"), c.get("N"), c.get("K"), c.get("moduli")] == [M, N, K, L]:
            if c.get("gemm_source_sha256") != gemm_source_hash():
                return None, "the capture on record is of other kernel source"
            return float(c["dram_read_bytes"]) + float(c["dram_write_bytes"]), c.get("command", "")
    return None, "no capture of this size on record"


def workload_name(n: int, L: int, phi: float, shape=None) -> str:
    dims = f"M=N=K={n} FP64 square" if shape is None else "M,N,K=%d,%d,%d FP64" % tuple(shape)
    return f"{dims}, (U-0.5)*exp({phi:g}*N(0,1)), seeds 0/1, Ozaki-II {L} moduli"


# ---------------------------------------------------------------------------------------------
# measured peaks, clocks
# ---------------------------------------------------------------------------------------------
def measured_peaks() -> dict:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"source": "measured", "hbm_gbs": d["hbm_gbs"], "bf16_burst": d["bf16_tflops"],
                "bf16_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"])}
    return {"source": "fallback", "hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0}


class ClockSampler:
    """nvidia-smi clock and throttle-reason samples while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.gpu_index)], stdout=self.file, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.file.flush()
        rows = [r.split(", ") for r in open(self.file.name).read().strip().splitlines() if r.strip()]
        os.unlink(self.file.name)
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1])); smax.append(float(r[2])); power.append(float(r[3]))
            except ValueError:
                continue
            for name, flag in zip(names, r[5:9]):
                if flag.strip().lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(smax), "power_w_max": max(power),
                "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------------------------
# CPU oracle legs
# ---------------------------------------------------------------------------------------------
def threads_used(cpu_seconds: float, wall_seconds: float) -> int:
    """Threads a timed region kept busy on average (its process CPU time over its wall time): the big-integer loops
    of the oracle are single-threaded Python, only its float64 matrix products use the BLAS thread pool."""
    return max(1, int(round(cpu_seconds / max(wall_seconds, 1e-9))))


def oracle_sample_tflops(A: np.ndarray, B: np.ndarray, L: int, block: int, repeats: int = 1) -> tuple[float, float, str, int]:
    """Times the CPU oracle, as it stands, on a block x block corner of the output (full K).
    Returns (TFLOP/s, seconds per run, description of the sample, threads used)."""
    from oracle import ozaki2
    M, K = A.shape
    b = min(block, M, B.shape[1])
    As, Bs = np.ascontiguousarray(A[:b]), np.ascontiguousarray(B[:, :b])
    best, threads = float("inf"), 1
    for _ in range(repeats):
        t0, c0 = time.perf_counter(), time.process_time()
        ozaki2.dgemm(As, Bs, L)
        wall, cpu = time.perf_counter() - t0, time.process_time() - c0
        if wall < best:
            best, threads = wall, threads_used(cpu, wall)
    sample = f"oracle.ozaki2.dgemm on the {b}x{b} leading output block, full K={K} ({2.0 * b * b * K:.3g} flop-equivalents)"
    return 2.0 * b * b * K / best / 1e12, best, sample, threads


def oracle_full_runs(L: int, phi: float) -> dict:
    """Whole-matrix oracle runs at small sizes (the scheme-II pipeline at 256^3 and 1024^3, the exact fl(AB) at
    256^3), each timed once: effective FP64 GFLOP/s, seconds, threads."""
    from oracle import exact, ozaki2
    from paper_2608_06812_b200 import inputs
    out = {}
    for name, n, fn in (("ozaki2_256", 256, lambda a, b: ozaki2.dgemm(a, b, L)), ("ozaki2_1024", 1024, lambda a, b: ozaki2.dgemm(a, b, L)),
                        ("exact_fl_matmul_256", 256, exact.fl_matmul)):
        a, b = inputs.lognormal_matrix(n, n, phi, seed=0), inputs.lognormal_matrix(n, n, phi, seed=1)
        t0, c0 = time.perf_counter(), time.process_time()
        fn(a, b)
        wall, cpu = time.perf_counter() - t0, time.process_time() - c0
        out[name] = {"gflops": 2.0 * n ** 3 / wall / 1e9, "seconds": wall, "cores": threads_used(cpu, wall)}
    return out


def run_reference(args, rank: int, world: int) -> None:
    """--impl reference: the CPU oracle on this arm's workload, rank 0 only."""
    if rank != 0:
        return
    from paper_2608_06812_b200 import inputs
    n, L = args.size, args.moduli
    block = 128
    A = inputs.lognormal_matrix(block, n, args.phi, seed=0)          # 128 rows / columns of the workload's law and seeds
    B = inputs.lognormal_matrix(n, block, args.phi, seed=1)
    for _ in range(min(args.warmup, 1)):
        oracle_sample_tflops(A, B, L, block)
    secs = []
    for _ in range(args.steps):
        tf, s, sample, threads = oracle_sample_tflops(A, B, L, block)
        secs.append(s)
    t = statistics.mean(secs)
    value = 2.0 * block * block * n / t / 1e12
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * t, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "int64/f64 (CPU oracle)", "data": "synthetic",
            "config": {"workload": workload_name(n, L, args.phi), "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample, "host_cpus": os.cpu_count()},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------
# multi-rank reduction (replicas): max of the times, sum of the work
# ---------------------------------------------------------------------------------------------
def reduce_over_ranks(ms_per_step: float, flops_per_step: float, dist=None, device=None) -> tuple[float, float]:
    """Returns (max over ranks of ms_per_step, sum over ranks of flops_per_step)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return ms_per_step, flops_per_step
    import torch
    t = torch.tensor([ms_per_step], dtype=torch.float64, device=device)
    f = torch.tensor([flops_per_step], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(f, op=dist.ReduceOp.SUM)
    return float(t.item()), float(f.item())


# ---------------------------------------------------------------------------------------------
# the GPU arm
# ---------------------------------------------------------------------------------------------
def run_int8(args) -> None:
    """INT8 GEMM emulated on FP4 (9 limb products): device-resident timing, one JSON line."""
    import torch
    from paper_2608_06812_b200 import binding as ozk
    from paper_2608_06812_b200 import inputs
    n = args.size
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    stream = torch.cuda.current_stream().cuda_stream
    dA = torch.from_numpy(np.ascontiguousarray(inputs.int8_matrix(n, n, seed=0).T)).to(dev)
    dB = torch.from_numpy(np.ascontiguousarray(inputs.int8_matrix(n, n, seed=1).T)).to(dev)
    dC = torch.empty((n, n), dtype=torch.int32, device=dev)
    ws = torch.empty(ozk.ozk_igemm_i8_workspace_bytes(n, n, n), dtype=torch.uint8, device=dev)
    ozk.check(ozk.ozk_set_workspace(ws.data_ptr(), ws.numel()), "ozk_set_workspace")

    def step():
        ozk.check(ozk.ozk_igemm_i8(n, n, n, dA.data_ptr(), n, dB.data_ptr(), n, dC.data_ptr(), n, stream), "ozk_igemm_i8")
    for _ in range(max(args.warmup, 3)):
        step()
    ozk.check(ozk.ozk_get_async_status(stream), "status")
    sampler = ClockSampler(0)
    sampler.start()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0.record()
    for _ in range(args.steps):
        step()
    t1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = t0.elapsed_time(t1) / args.steps
    ops = 2.0 * n ** 3
    print(json.dumps({"metric": "INT8 x INT8 -> INT32 GEMM emulated on FP4 limbs, 2MNK/t", "value": ops / (ms * 1e-3) / 1e12,
                      "unit": "TOP/s", "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms,
                      "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "fp4_e2m1 (fp32 accumulate, int32 out)",
                      "data": "synthetic", "config": {"workload": f"M=N=K={n} int8 uniform on [-128,127], seeds 0/1"},
                      "clocks": clocks, "gpu_launches": 3 * args.steps,
                      "fp4_tflops_executed_9_products": 9 * ops / (ms * 1e-3) / 1e12}), flush=True)


def run_ozk(args, rank: int, local_rank: int, world: int) -> None:
    import torch
    import torch.distributed as dist
    from paper_2608_06812_b200 import binding as ozk
    from paper_2608_06812_b200 import inputs

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1 and not dist.is_initialized():
        dist.init_process_group("nccl", device_id=dev)

    n, L = args.size, args.moduli
    M = N = K = n
    shape = None
    if args.shape and args.scheme == "oz2":
        shape = [int(v) for v in args.shape.split(",")]
        M, N, K = shape
        n = None                                          # no square-size table applies
    stream = torch.cuda.current_stream().cuda_stream
    A = inputs.lognormal_matrix(M, K, args.phi, seed=0)
    B = inputs.lognormal_matrix(K, N, args.phi, seed=1)
    # column-major storage = the transpose in C order
    hA = torch.from_numpy(np.ascontiguousarray(A.T)).pin_memory()
    hB = torch.from_numpy(np.ascontiguousarray(B.T)).pin_memory()
    hC = torch.empty((N, M), dtype=torch.float64).pin_memory()
    dA, dB = hA.to(dev), hB.to(dev)
    dC = torch.empty((N, M), dtype=torch.float64, device=dev)
    oz1 = args.scheme == "oz1"
    if args.karatsuba:
        ozk.check(ozk.ozk_stage_set_karatsuba(True), "ozk_stage_set_karatsuba")
    ws_bytes = ozk.ozk_dgemm_oz1_workspace_bytes(M, N, K) if oz1 else ozk.ozk_dgemm_workspace_bytes(M, N, K, L)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    ozk.check(ozk.ozk_set_workspace(ws.data_ptr(), ws.numel()), "ozk_set_workspace")
    ozk.check(ozk.ozk_stage_timing_enable(not oz1), "ozk_stage_timing_enable")

    def step():
        if oz1:
            ozk.check(ozk.ozk_dgemm_oz1(M, N, K, dA.data_ptr(), M, dB.data_ptr(), K, dC.data_ptr(), M, stream), "ozk_dgemm_oz1")
        elif args.max_bits != 53:
            ozk.check(ozk.ozk_dgemm_ext(M, N, K, dA.data_ptr(), M, dB.data_ptr(), K, dC.data_ptr(), M, L, args.max_bits, stream),
                      "ozk_dgemm_ext")
        else:
            ozk.check(ozk.ozk_dgemm(M, N, K, dA.data_ptr(), M, dB.data_ptr(), K, dC.data_ptr(), M, L, stream), "ozk_dgemm")

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    ozk.check(ozk.ozk_get_async_status(stream), "ozk_get_async_status")
    ozk.check(ozk.ozk_stage_timing_enable(not oz1), "ozk_stage_timing_enable")   # forget the warm-up calls

    # ---- device-resident timing: exactly `steps` steps between two barriers -----------------
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    stage_acc = np.zeros(3)
    barrier()
    ev[0].record()
    for i in range(args.steps):
        step()
        ev[i + 1].record()
    barrier()
    # per-stage CUDA events the library recorded on this stream inside the timed steps (a ring of the
    # last 64 calls), read after the region so that no step waits for the host
    gemm_cycles = (0, 0, 0)
    if not oz1:
        stage_acc = np.array(ozk.ozk_stage_timing_read()) * args.steps
        gemm_cycles = ozk.ozk_stage_gemm_cycles()      # the last timed step's limb GEMM (first CTA pair's issuing thread)
    total_ms = ev[0].elapsed_time(ev[args.steps])
    clocks = sampler.stop() if rank == 0 else None
    ozk.check(ozk.ozk_get_async_status(stream), "ozk_get_async_status")
    per_step = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)]
    stage_acc /= args.steps
    ms_per_step = total_ms / args.steps
    flops = 2.0 * M * N * K

    # ---- end to end with host buffers -----------------------------------------------------
    e2e = None
    if not args.no_e2e and not (not oz1 and (K > ozk.OZK_CHUNK_K or args.max_bits != 53)):   # the host-buffer entry point takes one k range
        # the library's host-buffer entry point: A and B start in pinned host memory, C ends there; the copies
        # are inside the timed region (and overlap the stages inside the library)
        host_ws = ozk.ozk_dgemm_host_workspace_bytes(M, N, K, L) if not oz1 else 0
        if not oz1 and host_ws > ws.numel():
            ws_host = torch.empty(host_ws, dtype=torch.uint8, device=dev)
            ozk.check(ozk.ozk_set_workspace(ws_host.data_ptr(), ws_host.numel()), "ozk_set_workspace")

        def e2e_step():
            if oz1:
                dA.copy_(hA, non_blocking=True)
                dB.copy_(hB, non_blocking=True)
                step()
                hC.copy_(dC, non_blocking=True)
            else:
                ozk.check(ozk.ozk_dgemm_host(M, N, K, hA.data_ptr(), M, hB.data_ptr(), K, hC.data_ptr(), M, L, stream), "ozk_dgemm_host")
        e2e_step()
        barrier()
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(args.steps):
            e2e_step()
        t1.record()
        barrier()
        e2e_ms = t0.elapsed_time(t1) / args.steps
        e2e_ms, e2e_flops = reduce_over_ranks(e2e_ms, flops, dist if world > 1 else None, dev)
        e2e = {"value": e2e_flops / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": int(hA.numel() * 8 + hB.numel() * 8), "d2h_bytes_per_step": int(hC.numel() * 8)}

    ms_max, flops_all = reduce_over_ranks(ms_per_step, flops, dist if world > 1 else None, dev)
    value = flops_all / (ms_max * 1e-3) / 1e12

    if rank != 0:
        return
    peaks = measured_peaks()
    if oz1:
        line = {"metric": METRIC.replace("scheme II", "scheme I (15 x 15 limbs)"), "value": value, "unit": UNIT, "n_gpus": world,
                "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_max, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "fp4_e2m1 (fp32 accumulate, multiword integer reduction)",
                "data": "synthetic", "config": {"workload": workload_name(n, L, args.phi).replace(f"Ozaki-II {L} moduli", "Ozaki-I p=q=15"),
                                                "l2": "inputs larger than L2" if M * K * 8 > (126 << 20) else "inputs fit L2"},
                "clocks": clocks, "e2e": e2e, "gpu_launches": 8 * args.steps,
                "fp4_tflops_executed_240_products": 2.0 * 240 * M * N * K / (ms_max * 1e-3) / 1e12, "per_step_ms": per_step}
        print(json.dumps(line), flush=True)
        return
    gemm_ms = float(stage_acc[1])
    k_ranges = max(1, -(-((K + 255) // 256 * 256) // ozk.OZK_CHUNK_K))   # one limb GEMM + one residue add per extra k range
    # both limb-GEMM kernels skip the 13^2 term of modulus 169: executed = required = 4L - 1 products
    pair = ((N + 127) // 128 * 128) % 256 == 0 and os.environ.get("OZK_GEMM_PAIR", "1") != "0"
    executed = 4 * L - 1 if ozk.ozk_get_moduli(L)[0] == 169 else 4 * L
    # K up to 1792 takes the two-accumulator kernel (b0 beta + b1 gamma: four products for every modulus)
    gamma = pair and not args.karatsuba and 0 < K <= 1792 and os.environ.get("OZK_GEMM_GAMMA", "1") != "0"
    if gamma:
        executed = 4 * L
    if args.karatsuba and pair:
        executed -= sum(1 for l in range(L) if l == 11 or l >= 13)      # three products for the Karatsuba moduli
    fp4_flops_exec = 2.0 * executed * M * N * K
    fp4_flops_req = 2.0 * (4 * L - 1) * M * N * K        # the 13^2 term of modulus 169 is not required
    achieved = fp4_flops_exec / (gemm_ms * 1e-3) / 1e12
    proxy_sustained = peaks["bf16_sustained"] * FP4_PER_BF16
    traffic, traffic_note = recorded_traffic(M, N, K, L)
    # per-cycle view: executed multiply-adds per SM and clock at the SM clock sampled during the timed region, against
    # the nominal 9000 TFLOP/s at the maximum clock; and the share of its clocks the issuing thread of the first CTA
    # pair spent issuing rather than waiting (counters of the last launch, read after the region)
    per_cycle = None
    if clocks and clocks.get("sm_mhz") and pair:
        mac_per_clk_sm = fp4_flops_exec / 2.0 / k_ranges / (SM_COUNT * gemm_ms / k_ranges * 1e-3 * clocks["sm_mhz"] * 1e6)
        nominal_mac = NOMINAL_FP4_TFLOPS * 1e12 / 2.0 / (SM_COUNT * clocks["sm_max_mhz"] * 1e6)
        clk_total, clk_tmem, clk_operands = gemm_cycles
        # 16384 multiply-adds per SM and clock is what the tensor pipe does when ncu shows it 100 % active (calibrated on a
        # capture with K = 16384 tiles: 14 876 per clock at 91.3 % sm__pipe_tensor_cycles_active, see profiles/)
        per_cycle = {"mac_per_clk_per_sm": mac_per_clk_sm, "nominal_mac_per_clk_per_sm": nominal_mac, "frac": mac_per_clk_sm / nominal_mac,
                     "pipe_mac_per_clk_per_sm": 16384, "frac_of_pipe": mac_per_clk_sm / 16384.0,
                     "sm_mhz": clocks["sm_mhz"], "gemm_ms_x_sm_mhz": gemm_ms * clocks["sm_mhz"],
                     "issue_thread": {"clocks": clk_total, "waiting_for_tensor_memory": clk_tmem, "waiting_for_operands": clk_operands,
                                      "issuing_frac": (1.0 - (clk_tmem + clk_operands) / clk_total) if clk_total > 0 else None}}
    roofline = {"bound": "tensor", "kernel": "residue_gemm_gamma_kernel" if gamma else ("residue_gemm_pair_kernel" if pair else "limb_gemm_kernel"),
                "achieved": achieved,
                "peak": NOMINAL_FP4_TFLOPS, "unit": "TFLOP/s", "frac": achieved / NOMINAL_FP4_TFLOPS, "traffic": traffic,
                "traffic_source": traffic_note,
                "peak_source": "nominal dense FP4 of B200 (no FP4 peak is measured on this pool; the measured BF16 proxies follow)",
                "achieved_required_count": fp4_flops_req / (gemm_ms * 1e-3) / 1e12,
                "frac_of_4x_measured_bf16_sustained": achieved / proxy_sustained,
                "frac_of_4x_measured_bf16_burst": achieved / (peaks["bf16_burst"] * FP4_PER_BF16),
                "measured_bf16": {"source": peaks["source"], "sustained_tflops": peaks["bf16_sustained"], "burst_tflops": peaks["bf16_burst"]},
                "ms_per_launch": gemm_ms / k_ranges, "launches_per_step": k_ranges, "per_cycle": per_cycle}
    pre_bytes = (16 + L) * (M * K + K * N)               # scan read + convert read + one byte (two nibbles) per modulus
    crt_bytes = (L + 8) * M * N
    stages = {"preprocess_ms": float(stage_acc[0]), "limb_gemm_ms": gemm_ms, "crt_ms": float(stage_acc[2]),
              "preprocess_gbs": pre_bytes / (stage_acc[0] * 1e-3) / 1e9, "crt_gbs": crt_bytes / (stage_acc[2] * 1e-3) / 1e9,
              "hbm_peak_gbs": peaks["hbm_gbs"], "per_step_ms": per_step}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_max, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": (value / world / PAPER_TOTAL_TFLOPS[n]) if (n in PAPER_TOTAL_TFLOPS and L == 19 and args.max_bits == 53) else None,
            "dtype": "fp4_e2m1 (fp32 accumulate, integer CRT)", "data": "synthetic",
            "config": {"workload": workload_name(n, L, args.phi, shape), "l2": "inputs (%.2f + %.2f GiB) %s" % (M * K * 8 / 2 ** 30, K * N * 8 / 2 ** 30, "larger than L2" if (M * K + K * N) * 8 > (126 << 20) else "fit L2: not a valid timing size"),
                       "parallelism": "replicas" if world > 1 else "single GPU", "moduli": L, "karatsuba": bool(args.karatsuba),
                       "integer_bits": ozk.ozk_capacity_bits_ext(K, L, args.max_bits)},
            "clocks": clocks, "e2e": e2e, "gpu_launches": (KERNELS_PER_STEP + 2 * (k_ranges - 1)) * args.steps, "roofline": roofline, "stages": stages}

    if not args.no_fp64_context:
        try:
            x = torch.matmul(dB, dA)                      # native FP64 GEMM on the same GPU (C^T = B^T A^T): context only
            torch.cuda.synchronize()
            t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
            t0.record(); x = torch.matmul(dB, dA); t1.record(); torch.cuda.synchronize()
            line["native_fp64_tflops_context"] = flops / (t0.elapsed_time(t1) * 1e-3) / 1e12
            del x
        except Exception as exc:                          # out of memory on small boxes: context is optional
            line["native_fp64_tflops_context"] = f"unavailable: {type(exc).__name__}"
    if not args.no_fp64_context and world == 1:
        # the limb GEMM's own rate when the operands do not toggle (A = 0: every A-side nibble is zero), the counterpart of the
        # paper's single-kernel rate R (Section 7.4): what the same launch does when the 1 kW power cap does not bind
        try:
            dZ = torch.zeros_like(dA)
            for _ in range(2):
                ozk.check(ozk.ozk_dgemm(M, N, K, dZ.data_ptr(), M, dB.data_ptr(), K, dC.data_ptr(), M, L, stream), "ozk_dgemm")
            torch.cuda.synchronize()
            ozk.ozk_stage_timing_read()
            for _ in range(2):
                ozk.check(ozk.ozk_dgemm(M, N, K, dZ.data_ptr(), M, dB.data_ptr(), K, dC.data_ptr(), M, L, stream), "ozk_dgemm")
            torch.cuda.synchronize()
            own_ms = float(ozk.ozk_stage_timing_read()[1])
            own = fp4_flops_exec / (own_ms * 1e-3) / 1e12
            line["roofline"]["own_kernel_constant_operands"] = {"ms_per_launch": own_ms, "tflops": own, "frac_of_nominal": own / NOMINAL_FP4_TFLOPS,
                                                                "achieved_over_this": achieved / own}
            del dZ
        except Exception as exc:
            line["roofline"]["own_kernel_constant_operands"] = f"unavailable: {type(exc).__name__}"
    if not args.no_cpu_baseline and world == 1:            # the oracle leg runs on rank 0 of a single-GPU run only
        tf, secs, sample, threads = oracle_sample_tflops(A, B, L, 512)
        line["cpu_baseline"] = {"value": tf, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample, "seconds": secs,
                                "host_cpus": os.cpu_count(), "full_runs": oracle_full_runs(L, args.phi)}
    print(json.dumps(line), flush=True)


def launcher_selftest(rank: int, world: int) -> None:
    """CPU check of the multi-rank plumbing (gloo, no GPU, no kernels): every rank contributes a made-up step
    time and flop count, rank 0 prints the reduced line."""
    import torch.distributed as dist
    if world > 1:
        dist.init_process_group("gloo")
    ms, flops = reduce_over_ranks(10.0 + rank, 1e12, dist if world > 1 else None, None)
    if rank == 0:
        print(json.dumps({"selftest": "launcher", "n_gpus": world, "ms_per_step": ms, "value": flops / (ms * 1e-3) / 1e12}), flush=True)
    if world > 1:
        dist.destroy_process_group()


def spawn_ranks(n: int) -> int:
    """`python bench.py --gpus N` without a launcher: start N ranks of this script on this node with torch's
    launcher (one process per GPU, rendezvous on 127.0.0.1) and pass their output through."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    args = parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl != "reference":
        sys.exit(spawn_ranks(args.gpus))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.launcher_selftest:
        launcher_selftest(rank, world)
        return
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if args.scheme == "i8":
        if rank == 0:
            run_int8(args)
        return
    run_ozk(args, rank, local_rank, world)
    if world > 1:
        import torch.distributed as dist
        if dist.is_initialized():
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
