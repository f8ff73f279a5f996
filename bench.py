#!/usr/bin/env python
"""Benchmark of the bf16 GEMM lineage on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--no-extras]

A "step" is one pass of the hot path: one C <- A.B at the headline workload
(8192^3, row-major bf16 A and B, fp32 accumulation, bf16 C - the compute-bound
configuration) through the top lineage rung (tcgen05), called through the C ABI.
Inputs are seeded synthetic data already resident in HBM; A+B+C (384 MiB) exceed
the L2, so no flush is needed between iterations.  One JSON line is printed by
rank 0.  With N > 1 every rank runs an independent GEMM (weak scaling, no
data-path collective); timing is the max over ranks of CUDA-event time.

`--impl reference` times the CPU oracle (plain fp64 triple loop) on a bounded
row slab of the same workload on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

METRIC = "bf16 GEMM TFLOP/s per lineage rung and % of B200 BF16 peak (or HBM GB/s)"
WORKLOADS = {
    "c1": "c1: M=N=K=256, row-major, U[-1,1) bf16, fp32 C",
    "c2": "c2: M=1000 N=1001 K=999, row-major, unaligned leading dimensions, U[-1,1) bf16, fp32 C",
    "c3": "c3: M=N=K=4096, B column-major, N(0,1) bf16, fp32 accumulate, bf16 C",
    "c4": "c4: M=N=K=8192, row-major A and B, N(0,1/sqrt(K)) bf16, fp32 accumulate, bf16 C",
    "c5": "c5: M=16 N=8192 K=8192, row-major, N(0,1) x N(0,0.02) bf16, fp32 C (weight streaming)",
}
WORKLOAD = WORKLOADS["c4"]
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def measured_traffic(workload: str, variant: int):
    """DRAM bytes per launch of the dominant kernel from the stored profiler capture of this workload, or None.

    The figure is not measured by this program (it never runs under a profiler): it is read from the record kept
    beside the profiler summaries, which names the capture and the commit it was taken at."""
    try:
        rec = json.loads((ROOT / "profiles" / "traffic.json").read_text()).get(workload)
        if rec and int(rec.get("variant", -1)) == variant:
            return float(rec["dram_bytes_per_launch"])
    except Exception:
        pass
    return None

VARIANT_NAMES = ["naive", "tiled", "vectorized", "pipelined", "tcgen05", "mma_sync"]
LINEAGE_ORDER = [0, 1, 2, 3, 5, 4]     # rung 3.5 (mma.sync, variant id 5) sits between rungs 3 and 4


def load_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            d = json.loads(p.read_text())
            return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


# ---------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in self.REASONS.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.004)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ---------------------------------------------------------------------------- reference arm (CPU oracle)
def oracle_sample_seconds(case, rows: int, repeat: int = 1):
    """Seconds the oracle needs for the first `rows` rows of C (C only, all host cores)."""
    import numpy as np
    from oracle import gemm_oracle as orc
    A_sub = np.ascontiguousarray(case.A[:rows])
    best = None
    for _ in range(repeat):
        t0 = time.perf_counter()
        orc.gemm(rows, case.N, case.K, A_sub, case.lda, case.B, case.ldb, case.b_col_major, want_S=False)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    return best


def cpu_baseline(case, budget_s: float = 12.0):
    """Times the oracle, as it stands, on a bounded row slab sized for ~budget_s of CPU work."""
    from oracle import gemm_oracle as orc
    probe_rows = min(case.M, 16)
    t_probe = oracle_sample_seconds(case, probe_rows)
    rows = int(max(probe_rows, min(case.M, budget_s / max(t_probe, 1e-6) * probe_rows)))
    rows = max(16, (rows // 16) * 16) if case.M >= 16 else case.M
    t = oracle_sample_seconds(case, rows)
    flops = 2.0 * rows * case.N * case.K
    return {"value": flops / t / 1e12, "unit": "TFLOP/s", "cores": orc.host_threads(), "kind": "oracle",
            "sample": f"first {rows} of {case.M} rows of C at the full N={case.N}, K={case.K} "
                      f"(fp64 triple loop, {t:.2f} s)", "seconds": t, "rows": rows}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from paper_2605_28213_b200 import inputs as gen
    from oracle import gemm_oracle as orc
    case = gen.make_config("c4", 1)
    # one step = a slab sized so that warmup + steps stay within a few minutes
    t_probe = oracle_sample_seconds(case, 16)
    total_steps = max(1, args.steps + args.warmup)
    per_step_budget = min(10.0, 150.0 / total_steps)
    rows = int(max(16, min(case.M, per_step_budget / max(t_probe, 1e-6) * 16)) // 16 * 16)
    for _ in range(args.warmup):
        oracle_sample_seconds(case, rows)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_sample_seconds(case, rows)
    dt = (time.perf_counter() - t0) / max(1, args.steps)
    value = 2.0 * rows * case.N * case.K / dt / 1e12
    sample = f"each step = first {rows} of {case.M} rows of C at the full N and K (fp64 triple loop)"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample": sample},
            "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": orc.host_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)
    return 0


# ---------------------------------------------------------------------------- multi-rank helpers
def max_over_ranks(value: float, world: int, device=None) -> float:
    """MAX all-reduce of a per-rank scalar (elapsed time); identity for one rank."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tflops(flops_per_rank: float, world: int, seconds_per_step: float) -> float:
    """Aggregate over all ranks: every rank does flops_per_rank of work per step (weak scaling)."""
    return flops_per_rank * world / seconds_per_step / 1e12


# ---------------------------------------------------------------------------- GPU arm
class DeviceProblem:
    """A configuration resident in HBM plus its handle."""

    def __init__(self, case, kb, torch, device):
        self.case, self.torch = case, torch
        self.A = torch.from_numpy(case.A.view("int16")).to(device)
        self.B = torch.from_numpy(case.B.view("int16")).to(device)
        self.C = torch.empty((case.M, case.ldc), dtype=torch.int16 if case.c_bf16 else torch.float32, device=device)
        self.gemm = kb.Gemm(device.index, b_col_major=case.b_col_major, c_bf16=case.c_bf16)
        # the C-ABI call with everything marshalled once: addresses and the stream handle (every timed launch goes
        # to torch's current stream of this moment) - the short configurations are as long as a Python attribute walk
        self._run, self._h = kb.klineage_gemm_run, self.gemm._h
        self._ptrs = (self.A.data_ptr(), self.B.data_ptr(), self.C.data_ptr())
        self._stream = torch.cuda.current_stream(device).cuda_stream

    def run(self, variant, B=None):
        c = self.case
        a, b, cc = self._ptrs
        self._run(self._h, c.M, c.N, c.K, a, c.lda, b if B is None else B.data_ptr(), c.ldb, cc, c.ldc, variant,
                  self._stream)

    def time(self, variant, reps, warmup, flush=None, rotate=None):
        """Median and min milliseconds of single launches (events around each launch)."""
        torch = self.torch
        for i in range(warmup):
            self.run(variant, None if not rotate else rotate[i % len(rotate)])
        torch.cuda.synchronize()
        times = []
        for i in range(reps):
            if flush is not None:
                flush.fill_(i)                      # evict L2 outside the timed interval
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            self.run(variant, None if not rotate else rotate[i % len(rotate)])
            e1.record()
            e1.synchronize()
            times.append(e0.elapsed_time(e1))
        return statistics.median(times), min(times)


def smoke_check(prob, variant, result=None):
    """Sampled parity of the timed configuration against the oracle before any number is reported.

    result: an M x ldc matrix to check instead of running the device call (the host-operand call's C)."""
    import numpy as np
    from oracle import gemm_oracle as orc
    from paper_2605_28213_b200 import inputs as gen
    c = prob.case
    rows = np.array(sorted({(r * 977 + 13) % c.M for r in range(8)}))
    C_ref, S = orc.gemm(len(rows), c.N, c.K, np.ascontiguousarray(c.A[rows]), c.lda, c.B, c.ldb, c.b_col_major)
    if result is None:
        prob.run(variant)
        prob.torch.cuda.synchronize()
        result = prob.C
    got = result[rows.tolist()][:, :c.N].cpu().numpy()
    vals = gen.bf16_bits_to_f32(got.view(np.uint16)).astype(np.float64) if c.c_bf16 else got.astype(np.float64)
    bound = orc.bound_bf16(c.K, S, C_ref) if c.c_bf16 else orc.bound_f32(c.K, S)
    return bool(np.all(np.abs(vals - C_ref) <= bound))


def run_gpu(args):
    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2605_28213_b200 import binding as kb
    from paper_2605_28213_b200 import inputs as gen

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    peaks, peak_kind = load_peaks()

    case = gen.make_config(args.workload, 1 + rank)
    prob = DeviceProblem(case, kb, torch, device)
    V = args.variant
    parity_ok = smoke_check(prob, V) if rank == 0 else True
    # A workload whose operands fit the L2 (c5: 129 MiB of weights) rotates over distinct
    # B buffers so that no iteration replays a warm L2.
    small = case.algorithmic_bytes < (300 << 20)
    rot = [prob.B] + ([prob.B.clone() for _ in range(3)] if small else [])

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(3, args.warmup)):
        prob.run(V, rot[i % len(rot)])
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clocks:
        e0.record()
        for i in range(args.steps):
            prob.run(V, rot[i % len(rot)])
        e1.record()
        barrier()
    ms = max_over_ranks(e0.elapsed_time(e1), world, device)
    code, kid = prob.gemm.device_status()
    ms_per_step = ms / args.steps
    tflops = whole_job_tflops(case.flops, world, ms_per_step * 1e-3)

    # ---- end to end: the library's host-operand call (klineage_gemm_run_host) on pinned host buffers - every
    # step copies A and B to the device, multiplies and copies C back, the three overlapped slab by slab inside
    # the library; the step ends when the stream has passed the last copy back
    hA = torch.from_numpy(case.A.view("int16")).pin_memory()
    hB = torch.from_numpy(case.B.view("int16")).pin_memory()
    hC = torch.zeros_like(prob.C, device="cpu").pin_memory()
    e2e_steps = max(2, min(args.steps, 5))
    scratch_bytes = prob.gemm.host_scratch_bytes(case.M, case.N, case.K)
    scratch = torch.empty(scratch_bytes, dtype=torch.uint8, device=device)

    def e2e_step():
        prob.gemm.run_host(hA, hB, hC, case.M, case.N, case.K, case.lda, case.ldb, case.ldc, scratch, scratch_bytes, V)
        torch.cuda.current_stream().synchronize()

    e2e_step()
    e2e_ok = smoke_check(prob, V, result=hC)          # the host-operand call's C against the oracle, sampled rows
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    barrier()
    e2e_s = max_over_ranks((time.perf_counter() - t0) / e2e_steps, world, device)
    e2e = {"value": whole_job_tflops(case.flops, world, e2e_s), "unit": "TFLOP/s",
           "h2d_bytes_per_step": int(hA.numel() * 2 + hB.numel() * 2), "d2h_bytes_per_step": int(hC.numel() * hC.element_size()),
           "steps": e2e_steps, "call": "klineage_gemm_run_host (pinned host A, B, C; copies overlapped with row slabs)",
           "parity_checked": e2e_ok}
    del scratch

    # kernels of this library per step: the GEMM kernel, plus one repack kernel when an operand breaks TMA's
    # alignment rules and the tcgen05 rung copies it into the workspace (kernel-id flag 64)
    launches_per_step = 1
    if V == 4 and (kid - 400) & 64:
        launches_per_step += 1            # one repack launch copies whichever operands need it
    line = {
        "metric": METRIC, "value": tflops, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16 inputs, fp32 accumulate (tcgen05.mma kind::f16), bf16 C",
        "data": "synthetic",
        "config": {"workload": WORKLOADS[args.workload], "variant": f"{VARIANT_NAMES[V]} (rung {V})",
                   "parallelism": f"{world} independent GEMMs",
                   "l2": (f"{len(rot)} distinct B buffers rotated ({len(rot) * case.B.nbytes >> 20} MiB > L2); no flush"
                          if small else "A+B+C = 384 MiB exceed the 126 MB L2; no flush between iterations")},
        "clocks": clocks.summary(), "e2e": e2e, "gpu_launches": args.steps * launches_per_step,
        "parity_checked": parity_ok, "device_status": code, "kernel_id": kid,
    }
    per_gpu = tflops / world
    if args.workload == "c5":
        gbs = case.algorithmic_bytes / (ms_per_step * 1e-3) / 1e9
        line["roofline"] = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                            "frac": gbs / peaks["hbm_gbs"], "traffic": measured_traffic("c5", V),
                            "peak_source": f"{peak_kind} (copy bandwidth)", "frac_of_nominal_8000": gbs / 8000.0,
                            "algorithmic_bytes_per_launch": case.algorithmic_bytes}
    else:
        line["roofline"] = {"bound": "tensor", "achieved": per_gpu, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                            "frac": per_gpu / peaks["bf16_tflops"],
                            "traffic": measured_traffic(args.workload, V),
                            "peak_source": f"{peak_kind} (burst cuBLAS bf16)",
                            "frac_of_sustained": per_gpu / peaks["bf16_tflops_sustained"],
                            "frac_of_nominal_2250": per_gpu / 2250.0,
                            "kernel": "r4_pair_kernel" if (kid - 400) & 32 else VARIANT_NAMES[V],
                            "flops_per_launch": case.flops}

    if rank == 0 and world == 1 and not args.no_extras and (args.workload, V) == ("c4", 4):
        line["lineage"] = lineage_table(prob, kb, gen, torch, device, peaks)
        line["cpu_baseline"] = cpu_baseline(case)
    if world > 1:
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line), flush=True)
    return 0 if (parity_ok and e2e_ok and code == 0) else 1


def run_partitioned(args):
    """--partition n: ONE GEMM partitioned by columns over the ranks, all-gather fused into the epilogue.

    Every rank holds A and its column slice of B, multiplies them on the tcgen05 rung and its epilogue stores the
    result slice into every rank's full-width C (peer stores only; no operand is loaded from a peer, no collective
    follows).  Strong scaling: the job is one product whatever the number of ranks.  A step ends, for the timing,
    when every rank's launch has completed (barrier + synchronize after the loop); every rank then checks sampled
    rows of ITS OWN C - which all ranks wrote - against the oracle."""
    import numpy as np
    import torch
    import torch.distributed as dist
    from oracle import gemm_oracle as orc
    from paper_2605_28213_b200 import binding as kb
    from paper_2605_28213_b200 import inputs as gen
    from paper_2605_28213_b200 import npart

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    peaks, peak_kind = load_peaks()
    case = gen.make_config(args.workload, 1)                  # the same problem on every rank
    n0, n1 = npart.column_slice(case.N, world, rank)
    B_slice = np.ascontiguousarray(case.B[n0:n1, :] if case.b_col_major else case.B[:, n0:n1])
    ldb = case.K if case.b_col_major else max(n1 - n0, 1)
    A = torch.from_numpy(case.A.view("int16")).to(device)
    Bs = torch.from_numpy(B_slice.view("int16")).to(device)
    shared = npart.SharedC(case.M, case.ldc, torch.int16 if case.c_bf16 else torch.float32, device, world, rank)
    shared.local.zero_()
    gemm = kb.Gemm(local, b_col_major=case.b_col_major, c_bf16=case.c_bf16)
    part = npart.NPartitionedGemm(gemm, world, rank, case.N, shared.ptrs, case.ldc)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    barrier()
    for _ in range(max(3, args.warmup)):
        npart.partitioned_step(part, A, Bs, case.M, case.K, case.lda, ldb, args.variant)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clocks:
        e0.record()
        for _ in range(args.steps):
            npart.partitioned_step(part, A, Bs, case.M, case.K, case.lda, ldb, args.variant)
        e1.record()
        barrier()
    ms = max_over_ranks(e0.elapsed_time(e1), world, device) / args.steps
    code, kid = gemm.device_status()
    rows = np.array(sorted({(r * 977 + 13 + 31 * rank) % case.M for r in range(8)}))
    C_ref, S = orc.gemm(len(rows), case.N, case.K, np.ascontiguousarray(case.A[rows]), case.lda, case.B, case.ldb,
                        case.b_col_major)
    got = shared.local[rows.tolist()][:, :case.N].cpu().numpy()
    vals = gen.bf16_bits_to_f32(got.view(np.uint16)).astype(np.float64) if case.c_bf16 else got.astype(np.float64)
    bound = orc.bound_bf16(case.K, S, C_ref) if case.c_bf16 else orc.bound_f32(case.K, S)
    ok = bool(np.all(np.abs(vals - C_ref) <= bound)) and code == 0
    ok_all = max_over_ranks(0.0 if ok else 1.0, world, device) == 0.0
    tflops = case.flops / (ms * 1e-3) / 1e12
    celt = 2 if case.c_bf16 else 4
    line = {
        "metric": METRIC, "value": tflops, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": True, "scaling": "strong",
        "vs_baseline": None, "dtype": "bf16 inputs, fp32 accumulate (tcgen05.mma kind::f16), bf16 C", "data": "synthetic",
        "config": {"workload": WORKLOADS[args.workload], "variant": f"{VARIANT_NAMES[args.variant]} (rung {args.variant})",
                   "parallelism": f"one GEMM partitioned by columns over {world} ranks; every rank's epilogue stores its "
                                  f"slice into all {world} C matrices (peer stores, rendezvous: {shared.how})",
                   "l2": "A + B slice + C exceed the L2; no flush between iterations"},
        "clocks": clocks.summary(), "gpu_launches": args.steps * world, "parity_checked": ok_all, "device_status": code,
        "kernel_id": kid, "e2e": None,
        "exchange": {"bytes_stored_to_peers_per_rank_per_step": int((world - 1) * case.M * (n1 - n0) * celt),
                     "bound_note": "stores leave over NVLink at <= 770 GB/s per direction (measured peer copy)"},
        "roofline": {"bound": "tensor", "achieved": tflops / world, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                     "frac": tflops / world / peaks["bf16_tflops"], "traffic": None,
                     "peak_source": f"{peak_kind} (burst cuBLAS bf16)", "flops_per_launch": case.flops / world},
    }
    if world > 1:
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line), flush=True)
    return 0 if ok_all else 1


def run_shape(args):
    """--shape MxNxK: one ad-hoc product (row-major bf16 operands N(0, 1/sqrt(K)), bf16 C) through the chosen rung;
    a profiling aid - the profiler summaries of shapes outside the five configurations name this command."""
    import numpy as np
    import torch
    from paper_2605_28213_b200 import binding as kb
    from paper_2605_28213_b200 import inputs as gen
    M, N, K = (int(x) for x in args.shape.lower().split("x"))
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    case = gen.make_case(M, N, K, seed=1, dist_a="normal", dist_b="normal", sigma_b=K ** -0.5, c_bf16=True,
                         name=f"shape{M}x{N}x{K}")
    prob = DeviceProblem(case, kb, torch, device)
    ok = smoke_check(prob, args.variant)
    for _ in range(max(3, args.warmup)):
        prob.run(args.variant)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        prob.run(args.variant)
    e1.record()
    e1.synchronize()
    us = e0.elapsed_time(e1) / args.steps * 1e3
    code, kid = prob.gemm.device_status()
    print(json.dumps({"shape": [M, N, K], "variant": VARIANT_NAMES[args.variant], "us_per_launch_back_to_back": us,
                      "tflops": case.flops / us / 1e6, "kernel_id": kid, "device_status": code, "parity_checked": ok}),
          flush=True)
    return 0 if ok and code == 0 else 1


def lineage_table(prob_c4, kb, gen, torch, device, peaks):
    """Per-rung throughput at 8192^3 and 4096^3, and the HBM-bound skinny shape for every rung."""
    out = {}
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
    reps = {0: (1, 2), 1: (2, 5), 2: (2, 5), 3: (2, 5), 5: (3, 10), 4: (5, 30)}          # (warmup, reps)
    c4 = prob_c4.case
    rows = {}
    for v in LINEAGE_ORDER:
        w, r = reps[v]
        med, mn = prob_c4.time(v, r, w)
        rows[VARIANT_NAMES[v]] = {"ms_median": med, "ms_min": mn, "tflops": c4.flops / (med * 1e-3) / 1e12,
                                  "frac_bf16_peak": c4.flops / (med * 1e-3) / 1e12 / peaks["bf16_tflops"],
                                  "kernel_id": prob_c4.gemm.last_kernel_id()}
    out["c4_8192^3"] = rows

    c3 = gen.make_config("c3", 1)
    p3 = DeviceProblem(c3, kb, torch, device)
    rows = {}
    for v in LINEAGE_ORDER:
        w, r = reps[v]
        med, mn = p3.time(v, r * 2, w, flush=flush)
        rows[VARIANT_NAMES[v]] = {"ms_median": med, "ms_min": mn, "tflops": c3.flops / (med * 1e-3) / 1e12,
                                  "frac_bf16_peak": c3.flops / (med * 1e-3) / 1e12 / peaks["bf16_tflops"],
                                  "kernel_id": p3.gemm.last_kernel_id()}
    out["c3_4096^3_Bcol"] = rows
    # AddMM at the same shape (the paper's held-out AddMM instance is 4096^3): bias epilogue fused, top rungs only
    bias = torch.from_numpy(gen.draw((1, c3.N), "normal", 1, 2)[0].view("int16")).to(device)
    rows = {}
    for v in (5, 4):
        times = []
        for i in range(13):
            flush.fill_(i)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            p3.gemm.run_addmm(p3.A, p3.B, bias, p3.C, c3.M, c3.N, c3.K, c3.lda, c3.ldb, c3.ldc, v)
            e1.record()
            e1.synchronize()
            times.append(e0.elapsed_time(e1))
        med = statistics.median(times[3:])
        rows[VARIANT_NAMES[v]] = {"ms_median": med, "tflops": c3.flops / (med * 1e-3) / 1e12,
                                  "frac_bf16_peak": c3.flops / (med * 1e-3) / 1e12 / peaks["bf16_tflops"],
                                  "kernel_id": p3.gemm.last_kernel_id()}
    out["addmm_4096^3_Bcol"] = rows
    # Autotuner of the tcgen05 rung: every candidate plan timed on the operands (fresh handles, so that no
    # pin leaks into the rows above and below), and the paper's held-out MM 2048^3 instance beside c3 and c4.
    mm2k = gen.make_case(2048, 2048, 2048, seed=1, dist_a="normal", dist_b="normal", c_bf16=True, name="mm2048")
    p2k = DeviceProblem(mm2k, kb, torch, device)
    tune = {}
    for name, pr in (("mm_2048^3", p2k), ("c3_4096^3_Bcol", p3), ("c4_8192^3", prob_c4)):
        c = pr.case
        time.sleep(1.0)     # let the power state settle: a sweep that starts hot times its first candidates low
        with kb.Gemm(device.index, b_col_major=c.b_col_major, c_bf16=c.c_bf16) as tg:
            n_cand = len(tg.plan_candidates(pr.A, pr.B, pr.C, c.M, c.N, c.K, c.lda, c.ldb, c.ldc))
            plan, best_us, heur_us = tg.autotune(pr.A, pr.B, pr.C, c.M, c.N, c.K, c.lda, c.ldb, c.ldc, iters=10)
        tune[name] = {"candidates": n_cand, "pinned_plan": plan.as_dict(),
                      "us_pinned": best_us, "us_heuristic": heur_us,
                      "tflops_pinned": c.flops / (best_us * 1e-6) / 1e12,
                      "tflops_heuristic": c.flops / (heur_us * 1e-6) / 1e12}
    tune["note"] = "microseconds per launch in back-to-back loops of 10 launches, minimum of two passes"
    out["autotune"] = tune
    del p2k

    out["gemm_family"] = family_table(kb, gen, torch, device, peaks, flush)

    c5 = gen.make_config("c5", 1)
    p5 = DeviceProblem(c5, kb, torch, device)
    rot = [p5.B] + [p5.B.clone() for _ in range(3)]          # 4 x 128 MiB of weights: no warm-L2 replay
    rows = {}
    for v in LINEAGE_ORDER:
        loops, per_loop = (3, 4) if v != 4 else (9, 40)
        best = []
        for _ in range(loops):
            for i in range(4):
                p5.run(v, rot[i])
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(per_loop):
                p5.run(v, rot[i % 4])
            e1.record()
            e1.synchronize()
            best.append(e0.elapsed_time(e1) / per_loop)
        med, mn = statistics.median(best), min(best)
        gbs = c5.algorithmic_bytes / (med * 1e-3) / 1e9
        rows[VARIANT_NAMES[v]] = {"us_median": med * 1e3, "us_min": mn * 1e3, "gbs": gbs,
                                  "frac_hbm": gbs / peaks["hbm_gbs"], "tflops": c5.flops / (med * 1e-3) / 1e12,
                                  "kernel_id": p5.gemm.last_kernel_id()}
    out["c5_16x8192x8192"] = rows
    # the same shape through a handle created with KLINEAGE_FLAG_STATIC_B (the weights are never written by
    # in-flight GPU work): the first B loads of a launch go out before the wait on the previous kernel
    with kb.Gemm(device.index, static_b=True) as gs:
        best = []
        for _ in range(9):
            for i in range(4):
                gs.run(p5.A, rot[i], p5.C, c5.M, c5.N, c5.K, c5.lda, c5.ldb, c5.ldc, 4)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(40):
                gs.run(p5.A, rot[i % 4], p5.C, c5.M, c5.N, c5.K, c5.lda, c5.ldb, c5.ldc, 4)
            e1.record()
            e1.synchronize()
            best.append(e0.elapsed_time(e1) / 40)
        med = statistics.median(best)
        gbs = c5.algorithmic_bytes / (med * 1e-3) / 1e9
        out["c5_16x8192x8192_static_b"] = {"us_median": med * 1e3, "gbs": gbs, "frac_hbm": gbs / peaks["hbm_gbs"],
                                           "kernel_id": gs.last_kernel_id()}
    # Context only (not a target, not a code path of this library): the vendor GEMM on the same buffers, timed
    # the same way as the rows above.
    ctx_rows = {}
    bf = torch.bfloat16
    A5, C5 = p5.A.view(bf), torch.empty((c5.M, c5.N), dtype=torch.float32, device=device)
    best = []
    for _ in range(9):
        for i in range(4):
            torch.matmul(A5, rot[i].view(bf)).float()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(40):
            torch.matmul(A5, rot[i % 4].view(bf))
        e1.record()
        e1.synchronize()
        best.append(e0.elapsed_time(e1) / 40)
    med = statistics.median(best)
    ctx_rows["c5_16x8192x8192"] = {"us_median": med * 1e3, "gbs": c5.algorithmic_bytes / (med * 1e-3) / 1e9,
                                   "note": "bf16 output (the library's default), back-to-back over 4 weight buffers"}
    A4, B4 = prob_c4.A.view(bf), prob_c4.B.view(bf)
    C4 = torch.empty((c4.M, c4.N), dtype=bf, device=device)
    times = []
    for i in range(13):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        torch.matmul(A4, B4, out=C4)
        e1.record()
        e1.synchronize()
        times.append(e0.elapsed_time(e1))
    med = statistics.median(times[3:])
    ctx_rows["c4_8192^3"] = {"ms_median": med, "tflops": c4.flops / (med * 1e-3) / 1e12}
    A3, B3 = p3.A.view(bf).view(c3.M, c3.lda), p3.B.view(bf).view(c3.N, c3.ldb)        # B stored N x K: pass its transpose
    C3 = torch.empty((c3.M, c3.N), dtype=bf, device=device)
    times = []
    for i in range(23):
        flush.fill_(i)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        torch.matmul(A3, B3.t(), out=C3)
        e1.record()
        e1.synchronize()
        times.append(e0.elapsed_time(e1))
    med = statistics.median(times[3:])
    ctx_rows["c3_4096^3_Bcol"] = {"ms_median": med, "tflops": c3.flops / (med * 1e-3) / 1e12}
    out["context_vendor_gemm"] = ctx_rows
    del A5, C5, C4, A3, B3, C3, p3
    # c1 and c2 are launch- and occupancy-bound (report only): back-to-back launches, operands L2-resident.
    for name in ("c1", "c2"):
        cs = gen.make_config(name, 1)
        ps = DeviceProblem(cs, kb, torch, device)
        rows = {}
        for v in LINEAGE_ORDER:
            per_loop = 200 if v else 20
            for _ in range(3):
                ps.run(v)
            torch.cuda.synchronize()
            best = []
            for _ in range(5):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(per_loop):
                    ps.run(v)
                e1.record()
                e1.synchronize()
                best.append(e0.elapsed_time(e1) / per_loop)
            med = statistics.median(best)
            rows[VARIANT_NAMES[v]] = {"us_median": med * 1e3, "us_min": min(best) * 1e3,
                                      "tflops": cs.flops / (med * 1e-3) / 1e12, "kernel_id": ps.gemm.last_kernel_id()}
        out[f"{name}_{cs.M}x{cs.N}x{cs.K}"] = rows
        del ps
        # context: the vendor library on a product of the same shape and pitches (fp32 / bf16 result as it gives it)
        ta = torch.randn(cs.M, cs.K, device=device).to(torch.bfloat16)
        tb = torch.randn(cs.K, cs.N, device=device).to(torch.bfloat16)
        tc = torch.empty(cs.M, cs.N, device=device, dtype=torch.bfloat16)
        for _ in range(3):
            torch.matmul(ta, tb, out=tc)
        torch.cuda.synchronize()
        best = []
        for _ in range(5):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(200):
                torch.matmul(ta, tb, out=tc)
            e1.record()
            e1.synchronize()
            best.append(e0.elapsed_time(e1) / 200)
        ctx_rows[f"{name}_{cs.M}x{cs.N}x{cs.K}"] = {"us_median": statistics.median(best) * 1e3,
                                                   "note": "bf16 output, back-to-back, L2-resident"}
        del ta, tb, tc
    out["note"] = ("c4, c3: single launches timed with CUDA events (c3 after a 256 MiB L2 flush; c4 operands exceed "
                   "L2); c5: back-to-back launches rotating over 4 distinct weight buffers (512 MiB > L2), time per "
                   "launch; c1, c2: back-to-back launches, operands L2-resident (launch/occupancy bound, report only)")
    return out


def family_table(kb, gen, torch, device, peaks, flush):
    """BMM and GroupedGEMM on the tcgen05 rung: one launch over all problems vs one launch per problem.

    Shapes: the paper's held-out BMM instances (batch 16 x 2048^3, batch 32 x 1024^3, bf16).  The paper gives no
    sizes for GroupedGEMM at G = 4 and 8; here 8192 rows are split unevenly over the groups (an expert-routing
    shape) with N = K = 4096, every group with its own weight matrix.
    """
    import numpy as np
    out = {}

    def timed(fn, reps=12):
        times = []
        for i in range(reps + 3):
            flush.fill_(i)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            e1.synchronize()
            times.append(e0.elapsed_time(e1))
        return statistics.median(times[3:])

    def rand_bf16(shape, seed, scale):
        gcpu = torch.Generator().manual_seed(seed)
        return (torch.randn(shape, generator=gcpu) * scale).to(torch.bfloat16).to(device)

    with kb.Gemm(device.index, b_col_major=False, c_bf16=True) as g:
        for batch, n in ((16, 2048), (32, 1024)):
            A = rand_bf16((batch, n, n), 11, 1.0)
            B = rand_bf16((batch, n, n), 12, n ** -0.5)
            C = torch.empty((batch, n, n), dtype=torch.bfloat16, device=device)
            one = timed(lambda: g.run_batched(batch, A, B, C, n, n, n, n, n, n, n * n, n * n, n * n, 4))
            kid, launches = g.last_kernel_id(), g.last_launch_count()
            ref = torch.bmm(A[:2].float(), B[:2].float())
            ok = bool(torch.allclose(C[:2].float(), ref, rtol=2e-2, atol=2e-2))

            def loop():
                for b in range(batch):
                    g.run(A[b], B[b], C[b], n, n, n, n, n, n, 4)
            per = timed(loop)
            lib = timed(lambda: torch.bmm(A, B, out=C))       # context only: the vendor library on the same buffers
            flops = 2.0 * batch * n ** 3
            out[f"bmm_bs{batch}_{n}^3"] = {"context_torch_bmm_ms": lib, "launches_one_call": launches,"ms_one_launch": one, "tflops_one_launch": flops / (one * 1e-3) / 1e12,
                                           "frac_bf16_peak": flops / (one * 1e-3) / 1e12 / peaks["bf16_tflops"],
                                           "ms_launch_per_problem": per,
                                           "tflops_launch_per_problem": flops / (per * 1e-3) / 1e12,
                                           "kernel_id": kid, "sane_vs_torch_bmm_on_2_batches": ok}
            del A, B, C
        for G in (4, 8):
            rng = np.random.default_rng(G)
            cuts = np.sort(rng.choice(np.arange(1, 8192 // 64), G - 1, replace=False)) * 64
            Ms = np.diff(np.concatenate(([0], cuts, [8192]))).tolist()
            n = k = 4096
            A = rand_bf16((8192, k), 21, 1.0)
            B = rand_bf16((G, k, n), 22, k ** -0.5)
            C = torch.empty((8192, n), dtype=torch.bfloat16, device=device)
            offs = np.concatenate(([0], np.cumsum(Ms)))[:-1].tolist()
            Ap = [A[o:].data_ptr() for o in offs]
            Cp = [C[o:].data_ptr() for o in offs]
            Bp = [B[i].data_ptr() for i in range(G)]
            one = timed(lambda: g.run_grouped(Ap, Bp, Cp, Ms, [n] * G, [k] * G, [k] * G, [n] * G, [n] * G, 4))
            kid, launches = g.last_kernel_id(), g.last_launch_count()
            o = offs[1]
            ref = A[o:o + 64].float() @ B[1].float()
            ok = bool(torch.allclose(C[o:o + 64].float(), ref, rtol=2e-2, atol=2e-2))

            def loop():
                for i in range(G):
                    g.run(Ap[i], Bp[i], Cp[i], Ms[i], n, k, k, n, n, 4)
            per = timed(loop)
            flops = 2.0 * 8192 * n * k
            out[f"grouped_G{G}_8192rows_4096x4096"] = {
                "rows_per_group": Ms, "launches_one_call": launches, "ms_one_launch": one, "tflops_one_launch": flops / (one * 1e-3) / 1e12,
                "frac_bf16_peak": flops / (one * 1e-3) / 1e12 / peaks["bf16_tflops"], "ms_launch_per_problem": per,
                "tflops_launch_per_problem": flops / (per * 1e-3) / 1e12, "kernel_id": kid,
                "sane_vs_torch_on_64_rows": ok}
            del A, B, C
        # Column-partitioned multi-GPU GEMM, one rank's share of 8192^3 at world 8 (1024 columns of B), its epilogue
        # storing the slice into 8 full-width C matrices.  All 8 "ranks'" buffers live on this GPU here: the stores'
        # cost is HBM's, not NVLink's; the row shows what the fused all-gather adds to the kernel.
        from paper_2605_28213_b200 import npart
        n, world = 8192, 8
        A = rand_bf16((n, n), 31, 1.0)
        Bs = rand_bf16((n, n // world), 32, n ** -0.5)
        Cs = [torch.empty((n, n), dtype=torch.bfloat16, device=device) for _ in range(world)]
        part = npart.NPartitionedGemm(g, world, 3, n, [c.data_ptr() for c in Cs], n)
        fused = timed(lambda: part.run(A, Bs, n, n, n, n // world))
        kid, launches = g.last_kernel_id(), g.last_launch_count()
        alone = timed(lambda: g.run(A, Bs, part.dst[3], n, n // world, n, n, n // world, n, 4))
        ok = all(bool(torch.equal(Cs[0][:, part.n0:part.n1], c[:, part.n0:part.n1])) for c in Cs[1:])
        flops = 2.0 * n * (n // world) * n
        out["npart_world8_rank_share_of_8192^3"] = {
            "ms_fused_store_to_8_destinations": fused, "tflops_fused": flops / (fused * 1e-3) / 1e12,
            "ms_one_destination": alone, "tflops_one_destination": flops / (alone * 1e-3) / 1e12,
            "extra_bytes_stored": 7 * n * (n // world) * 2, "launches_one_call": launches, "kernel_id": kid,
            "all_destinations_equal": ok}
        del A, Bs, Cs
    # Conv2d of the paper's workload table (N=8, C=64, 56x56, F=128, 3x3, fp16; channels-last, padding 1, stride 1)
    cc = gen.conv_benchmark_case(1)
    x = torch.from_numpy(cc.x.view("int16")).to(device)
    w = torch.from_numpy(cc.w.view("int16")).to(device)
    y = torch.empty((cc.N, cc.P, cc.Q, cc.F), dtype=torch.float16, device=device)
    with kb.Conv2d(device.index, y_f16=True) as conv:
        row = {}
        for v, name in ((0, "naive"), (4, "tcgen05")):
            t = timed(lambda: conv.run(x, w, y, cc.N, cc.H, cc.W, cc.C, cc.F, cc.R, cc.S, cc.pad, cc.stride, v))
            for _ in range(3):
                conv.run(x, w, y, cc.N, cc.H, cc.W, cc.C, cc.F, cc.R, cc.S, cc.pad, cc.stride, v)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(50):
                conv.run(x, w, y, cc.N, cc.H, cc.W, cc.C, cc.F, cc.R, cc.S, cc.pad, cc.stride, v)
            e1.record()
            e1.synchronize()
            loop_ms = e0.elapsed_time(e1) / 50
            row[name] = {"us_single_after_flush": t * 1e3, "us_back_to_back": loop_ms * 1e3,
                         "tflops_back_to_back": cc.flops / (loop_ms * 1e-3) / 1e12, "kernel_id": conv.last_kernel_id()}
        xt = x.view(torch.float16).permute(0, 3, 1, 2)          # NCHW views of channels-last storage
        wt = w.view(torch.float16).permute(0, 3, 1, 2)
        lib = timed(lambda: torch.nn.functional.conv2d(xt, wt, padding=cc.pad, stride=cc.stride))
        ref = torch.nn.functional.conv2d(xt.float(), wt.float(), padding=cc.pad, stride=cc.stride).permute(0, 2, 3, 1)
        conv.run(x, w, y, cc.N, cc.H, cc.W, cc.C, cc.F, cc.R, cc.S, cc.pad, cc.stride, 4)
        row["sane_vs_torch_conv2d"] = bool(torch.allclose(y.float(), ref, rtol=2e-2, atol=2e-2))

        # device-bound: 20 launches captured into a CUDA graph and replayed (in a plain loop both libraries are
        # bound by their host path at this size), also at a larger batch of the same layer
        def in_graph(fn):
            side = torch.cuda.Stream()
            with torch.cuda.stream(side):
                for _ in range(3):
                    fn()
            torch.cuda.synchronize()
            gr = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gr, stream=side):
                for _ in range(20):
                    fn()
            gr.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(10):
                gr.replay()
            e1.record()
            e1.synchronize()
            return e0.elapsed_time(e1) / 200 * 1e3

        row["tcgen05"]["us_in_graph"] = in_graph(
            lambda: conv.run(x, w, y, cc.N, cc.H, cc.W, cc.C, cc.F, cc.R, cc.S, cc.pad, cc.stride, 4))
        row["tcgen05"]["tflops_in_graph"] = cc.flops / (row["tcgen05"]["us_in_graph"] * 1e-6) / 1e12
        row["context_torch_conv2d_us_in_graph"] = in_graph(
            lambda: torch.nn.functional.conv2d(xt, wt, padding=cc.pad, stride=cc.stride))
        c64 = gen.make_conv_case(64, cc.H, cc.W, cc.C, cc.F, cc.R, cc.S, seed=1)
        x64 = torch.from_numpy(c64.x.view("int16")).to(device)
        y64 = torch.empty((c64.N, c64.P, c64.Q, c64.F), dtype=torch.float16, device=device)
        x64t = x64.view(torch.float16).permute(0, 3, 1, 2)
        us64 = in_graph(lambda: conv.run(x64, w, y64, c64.N, c64.H, c64.W, c64.C, c64.F, c64.R, c64.S, c64.pad, c64.stride, 4))
        row["batch64_same_layer"] = {
            "us_in_graph": us64, "tflops_in_graph": c64.flops / (us64 * 1e-6) / 1e12, "kernel_id": conv.last_kernel_id(),
            "context_torch_conv2d_us_in_graph": in_graph(
                lambda: torch.nn.functional.conv2d(x64t, wt, padding=cc.pad, stride=cc.stride))}
        del x64, y64
        row["context_torch_conv2d_us_single"] = lib * 1e3
        row["algorithmic_bytes"] = int(x.numel() * 2 + w.numel() * 2 + y.numel() * 2)
        out["conv2d_n8_c64_56x56_f128_3x3_f16"] = row
    out["note"] = ("median of 12 timed calls, each after a 256 MiB L2 flush; 'launch_per_problem' issues the "
                   "single-problem call once per batch / group on the same stream; the torch comparison is a "
                   "sanity check of the timed buffers, parity is established by the tests against the oracle")
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="klineage", choices=["klineage", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the per-rung table and the CPU baseline")
    ap.add_argument("--workload", default="c4", choices=sorted(WORKLOADS),
                    help="configuration to time (default: the headline 8192^3; others are for profiling)")
    ap.add_argument("--variant", type=int, default=4, choices=range(6),
                    help="lineage rung to time (default 4 = tcgen05; 5 = the mma.sync rung 3.5)")
    ap.add_argument("--partition", default="replicas", choices=["replicas", "n"],
                    help="N > 1: 'replicas' = independent GEMMs (default, weak scaling); 'n' = ONE GEMM partitioned by "
                         "columns over the ranks with the all-gather fused into the epilogue (strong scaling)")
    ap.add_argument("--shape", default=None, help="MxNxK: time one ad-hoc product (profiling aid) and print a short JSON line")
    ap.add_argument("--family", action="store_true",
                    help="time only the BMM / GroupedGEMM rows (for profiling) and print them as one JSON line")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.family:
        import torch
        from paper_2605_28213_b200 import binding as kb
        from paper_2605_28213_b200 import inputs as gen
        device = torch.device("cuda", 0)
        torch.cuda.set_device(device)
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
        print(json.dumps({"gemm_family": family_table(kb, gen, torch, device, load_peaks()[0], flush)}), flush=True)
        return 0
    if args.shape:
        return run_shape(args)
    if args.partition == "n":
        return run_partitioned(args)
    return run_gpu(args)


if __name__ == "__main__":
    sys.exit(main())
