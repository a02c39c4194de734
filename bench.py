#!/usr/bin/env python3
"""Benchmark of the asymmetric-tile-buffered BFP16 x BF16 GEMM hot path on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One *step* is one pass of the whole hot path over one batch of seeded synthetic input that is
already resident in HBM: quantise A (fp32 -> BFP16 planes), pick the tiling with the host model,
run the GEMM.  ``value`` is 2*M*N*K per step time, summed over ranks (weak scaling: every rank
runs the full workload on its own A; no data-path collective).  ``roofline`` is about the GEMM
kernel alone: its algorithmic FLOPs over its own CUDA-event time inside the same timed region,
against the measured dense-BF16 cuBLAS peak.  ``e2e`` repeats the step with host buffers: pinned
host A and B are copied to the device and C is copied back inside the timed region.
``cpu_baseline`` times the FP64 oracle on the host cores on a bounded row sample (a reported
baseline, not a target).  ``--impl reference`` times that oracle alone.

After the timed region, on one GPU, the line also gets ``ablation`` - the GEMM alone under every T_MA
of the single-CTA 256 x 256 family and of the CTA-pair 256 x 512 family, the symmetric form first, with
the best asymmetric rate over the symmetric one - and ``roofline.sustained``: the headline GEMM
launched back to back for more than 2 s (the GPU settles under its power cap) against the sustained
cuBLAS figure, with the SM clock sampled meanwhile.

``--gpus N`` without a launcher around it (no WORLD_SIZE in the environment) starts N ranks itself.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "ATB GEMM TFLOPS (1xB200) at 8192^3 BFP16xBF16"
DEFAULT_WORKLOAD = "cfg3_8192"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL_BF16_TFLOPS = 2250.0        # NVIDIA's dense BF16 figure for B200 (context beside the measured peak)
# The asymmetric-buffering ablation: for fixed (T_MC, T_K, T_N) only T_MA moves, the first entry of
# each family is its symmetric form.  On the CTA pair each SM holds 128 rows of the 256-row tile (or its
# own 128 x 256 tile of a stacked pair of tiles), so T_MA = 128 is symmetric there.
ABLATION_FAMILIES = {
    "single_cta_256x256": [(256, 256, 64, 256), (128, 256, 64, 256), (64, 256, 64, 256), (32, 256, 64, 256)],
    "cta_pair_256x512": [(128, 256, 64, 512), (64, 256, 64, 512), (32, 256, 64, 512)],
    "cta_pair_stacked_128x256": [(128, 128, 128, 256), (64, 128, 128, 256), (32, 128, 128, 256)],
}
SUSTAINED_SECONDS = 2.2


def load_ncu_traffic():
    """dram__bytes_read.sum + dram__bytes_write.sum per GEMM launch, from the 1-pass ncu captures of the
    full launch that are summarised beside this table (None where no capture exists)."""
    try:
        with open(os.path.join(ROOT, "profiles", "ncu_dram_traffic.json")) as f:
            rows = json.load(f)["launches"]
        return {(r["workload"], r["kernel"]): float(r["dram_read_bytes"]) + float(r["dram_write_bytes"]) for r in rows}
    except Exception:
        return {}


def rho_per_core(t):
    """rho = T_MC / T_MA as one SM sees it: the CTA-pair tiling keeps 128 of its 256 rows per SM."""
    T_MA, T_MC, T_K, T_N = t
    rows = 128 if (T_MC, T_K, T_N) == (256, 64, 512) else T_MC
    return rows // min(T_MA, rows)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Polls SM clock and throttle reasons through NVML (read only) while the timed region runs."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self._h) if hasattr(
                    nv, "nvmlDeviceGetCurrentClocksEventReasons") else nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def rank_seed(base_seed: int, rank: int) -> int:
    """Each rank multiplies its own rows of a taller A: a different seed per rank, same B."""
    return base_seed + rank


def max_over_ranks(values, device, world: int):
    """Element-wise maximum of per-rank timings over all ranks (identity for one rank)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def aggregate_tflops(flops_per_rank: float, world: int, ms_per_step: float) -> float:
    """Whole-job throughput: every rank does `flops_per_rank` per step in the slowest rank's time."""
    return world * flops_per_rank / (ms_per_step * 1e-3) / 1e12


def cpu_oracle_sample(name: str, target_seconds: float):
    """Times the FP64 oracle GEMM (as it stands) on a bounded row sample of workload `name`."""
    import oracle
    from paper_2511_16041_b200 import inputs
    c = inputs.CONFIGS[name]
    N, K = c["N"], c["K"]
    Bb = inputs.make_B_bits(K, N, c["b_scale"])
    probe = min(c["M"], 64)
    A = inputs.make_A(c["A"], probe, K)
    mant, exp = oracle.quantize_bfp16(A)
    t0 = time.perf_counter()
    oracle.gemm(mant, exp, Bb)
    t_probe = time.perf_counter() - t0
    # the probe pays the fixed B conversion; size the sample from a second, larger probe
    rows2 = min(c["M"], 256)
    A = inputs.make_A(c["A"], rows2, K)
    mant, exp = oracle.quantize_bfp16(A)
    t0 = time.perf_counter()
    oracle.gemm(mant, exp, Bb)
    t2 = time.perf_counter() - t0
    per_row = max((t2 - t_probe) / max(rows2 - probe, 1), 1e-6)
    rows = int(min(c["M"], max(rows2, (target_seconds - t_probe) / per_row)))
    rows -= rows % 8
    A = inputs.make_A(c["A"], rows, K)
    t0 = time.perf_counter()
    mant, exp = oracle.quantize_bfp16(A)
    oracle.gemm(mant, exp, Bb)
    dt = time.perf_counter() - t0
    return {"value": 2.0 * rows * N * K / dt / 1e12, "unit": "TFLOPS", "cores": oracle.num_threads(),
            "kind": "oracle", "seconds": round(dt, 3),
            "sample": f"first {rows} of {c['M']} rows of {name} (all {N} columns, K={K}): oracle quantise + FP64 GEMM and |a||b| sum"}


def run_reference(args):
    """--impl reference: the oracle, as it stands, on the host cores; one bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    from paper_2511_16041_b200 import inputs
    name = args.workload
    c = inputs.CONFIGS[name]
    M, N, K = c["M"], c["N"], c["K"]
    rows = min(M, 256)
    A = inputs.make_A(c["A"], rows, K)
    Bb = inputs.make_B_bits(K, N, c["b_scale"])
    times = []
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        mant, exp = oracle.quantize_bfp16(A)
        oracle.gemm(mant, exp, Bb)
        dt = time.perf_counter() - t0
        if i >= args.warmup:
            times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    value = 2.0 * rows * N * K / (ms * 1e-3) / 1e12
    sample = f"{rows} of {M} rows of {name} per step (all {N} columns, K={K})"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOPS", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": name, "M": M, "N": N, "K": K, "sampled_rows_per_step": rows},
            "cpu_baseline": {"value": value, "unit": "TFLOPS", "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": "TFLOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


def spawn_ranks(args) -> int:
    """``python bench.py --gpus N`` outside a launcher: start N ranks of this script, one per GPU, under
    torch.distributed.run on 127.0.0.1 (the same command line a launcher would use)."""
    import socket
    import subprocess
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def run_stub(args) -> int:
    """--stub-step: the rank plumbing of run_ours (rendezvous, barrier, max over ranks, whole-job figure,
    one line from rank 0) with a pretend step time instead of GPU work; gloo on CPU."""
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    ms = max_over_ranks([1.0 + rank], torch.device("cpu"), world)[0]
    if rank == 0:
        print(json.dumps({"stub": True, "n_gpus": world, "ms_per_step": ms, "value": aggregate_tflops(1e9, world, ms)}))
    if world > 1:
        dist.destroy_process_group()
    return 0


def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2511_16041_b200 as atb
    from paper_2511_16041_b200 import inputs

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback of the hot path")
    if local_rank >= torch.cuda.device_count():
        raise RuntimeError(f"rank {rank} wants GPU {local_rank} but only {torch.cuda.device_count()} are visible")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    atb.load_library()

    name = args.workload
    c = inputs.CONFIGS[name]
    M, N, K = c["M"], c["N"], c["K"]
    seed = rank_seed(inputs.BASE_SEED, rank)
    A_host = torch.from_numpy(inputs.make_A(c["A"], M, K, seed)).pin_memory()
    B_host = torch.from_numpy(inputs.make_B_bits(K, N, c["b_scale"]).view(np.int16)).pin_memory()
    C_host = torch.empty((M, N), dtype=torch.int16).pin_memory()

    stream = torch.cuda.Stream(dev)
    A_dev = A_host.to(dev)
    B_dev = B_host.to(dev).view(torch.bfloat16)
    mant = torch.empty((M, K), dtype=torch.int8, device=dev)
    plane = torch.empty(atb.atb_bfp16_exp_bytes(M, K), dtype=torch.uint8, device=dev)
    C_dev = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
    torch.cuda.synchronize()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    tiling_used = []

    def step(ev=None, A_d=None, B_d=None, C_d=None, on=None):
        """Whole hot path on device-resident input: quantise -> select tiling -> GEMM."""
        A_d = A_dev if A_d is None else A_d
        B_d = B_dev if B_d is None else B_d
        C_d = C_dev if C_d is None else C_d
        on = stream if on is None else on
        atb.atb_quantize_bfp16(A_d, mant, plane, stream=on)
        if args.tiling:
            t = tuple(args.tiling)
        else:
            t, _ = atb.atb_select_tiling(M, N, K, max_scores=1)
        if ev is not None:
            ev[0].record(on)
        atb.atb_gemm(M, N, K, *t, mant, plane, B_d, C_d, stream=on)
        if ev is not None:
            ev[1].record(on)
        if not tiling_used:
            tiling_used.append(tuple(t))

    # End-to-end leg: every step copies its A and B from pinned host memory and its C back.  Two sets
    # of device buffers and three streams let step i+1's upload and step i-1's download overlap step
    # i's kernels (PCIe is full duplex); every step still pays all three transfers.
    e2e_sets = []

    def e2e_setup():
        for _ in range(2):
            e2e_sets.append(dict(
                A=torch.empty_like(A_dev), B=torch.empty_like(B_dev), C=torch.empty_like(C_dev),
                C_host=torch.empty((M, N), dtype=torch.int16).pin_memory(),
                up=torch.cuda.Event(), done=torch.cuda.Event(), down=torch.cuda.Event()))
        return torch.cuda.Stream(dev), torch.cuda.Stream(dev)

    def run_e2e(n_steps, s_up, s_down):
        for i in range(n_steps):
            b = e2e_sets[i % 2]
            s_up.wait_event(b["done"])                 # the kernels that read this set two steps ago
            with torch.cuda.stream(s_up):
                b["A"].copy_(A_host, non_blocking=True)
                b["B"].view(torch.int16).copy_(B_host, non_blocking=True)
                b["up"].record(s_up)
            stream.wait_event(b["up"])
            stream.wait_event(b["down"])               # C of this set has been read back
            step(A_d=b["A"], B_d=b["B"], C_d=b["C"])
            b["done"].record(stream)
            s_down.wait_event(b["done"])
            with torch.cuda.stream(s_down):
                b["C_host"].copy_(b["C"].view(torch.int16), non_blocking=True)
                b["down"].record(s_down)
        s_up.synchronize(); stream.synchronize(); s_down.synchronize()

    # ---------------- device-resident timing ----------------
    for _ in range(max(args.warmup, 3)):
        step()
    atb.atb_device_status(stream)
    sampler = ClockSampler(physical_gpu_index(local_rank))
    gemm_events = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                   for _ in range(args.steps)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.start()
    t_begin.record(stream)
    for i in range(args.steps):
        step(gemm_events[i])
    t_end.record(stream)
    stream.synchronize()
    barrier()
    clocks = sampler.stop()
    atb.atb_device_status(stream)
    total_ms = t_begin.elapsed_time(t_end)
    gemm_ms = sum(a.elapsed_time(b) for a, b in gemm_events) / args.steps

    # ---------------- end-to-end timing (host buffers) ----------------
    e2e_steps = max(4, min(args.steps, 10))
    s_up, s_down = e2e_setup()
    run_e2e(2, s_up, s_down)
    barrier()
    t0 = time.perf_counter()
    run_e2e(e2e_steps, s_up, s_down)
    torch.cuda.synchronize()
    e2e_wall_ms = 1e3 * (time.perf_counter() - t0)
    barrier()
    e2e_ms = e2e_wall_ms / e2e_steps
    e2e_check = e2e_sets[(e2e_steps - 1) % 2]["C_host"]
    assert bool((e2e_check == C_dev.view(torch.int16).cpu()).all()), "end-to-end result differs from the resident run"

    # ---------------- quantiser alone (HBM roofline) ----------------
    q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    q0.record(stream)
    for _ in range(10):
        atb.atb_quantize_bfp16(A_dev, mant, plane, stream=stream)
    q1.record(stream)
    stream.synchronize()
    quant_ms = q0.elapsed_time(q1) / 10

    # ---------------- the T_MA ablation and a sustained leg (one GPU only) ----------------
    ablation = sustained = library = None
    if world == 1 and not args.no_ablation:
        def time_gemm(t, reps):
            for _ in range(2):
                atb.atb_gemm(M, N, K, *t, mant, plane, B_dev, C_dev, stream=stream)
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
            for a, b in evs:
                a.record(stream)
                atb.atb_gemm(M, N, K, *t, mant, plane, B_dev, C_dev, stream=stream)
                b.record(stream)
            stream.synchronize()
            return min(a.elapsed_time(b) for a, b in evs)

        # the library's bf16 GEMM (torch.matmul -> cuBLAS) on operands of the same shape, timed the same way in
        # the same walk: context for the fraction of the measured peak, which moves from GPU to GPU
        A_lib = torch.randn((M, K), device=dev, dtype=torch.float32).to(torch.bfloat16)
        C_lib = torch.empty((M, N), device=dev, dtype=torch.bfloat16)

        def time_library(reps):
            with torch.cuda.stream(stream):
                for _ in range(2):
                    torch.matmul(A_lib, B_dev, out=C_lib)
                evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
                for a, b in evs:
                    a.record(stream)
                    torch.matmul(A_lib, B_dev, out=C_lib)
                    b.record(stream)
            stream.synchronize()
            return min(a.elapsed_time(b) for a, b in evs)

        # every tiling of the families in one process, walked in two opposite orders (what ran just
        # before moves a rate by a few per cent); a tiling keeps its better time
        t_head = tuple(tiling_used[0])
        walk = [t for fam in ABLATION_FAMILIES.values() for t in fam]
        walk += [t_head] if t_head not in walk else []
        best_ms, lib_ms = {}, []
        for order in (walk, walk[::-1]):
            for t in order:
                ms = time_gemm(t, 5)
                best_ms[t] = min(ms, best_ms.get(t, ms))
                if t == t_head:
                    lib_ms.append(time_library(5))
        atb.atb_device_status(stream)
        tf = lambda t: 2.0 * M * N * K / (best_ms[t] * 1e-3) / 1e12
        ablation = {"how": "atb_gemm alone on the resident planes; both families interleaved in one process, "
                           "two opposite orders, best of 2 x 5 launches per tiling (CUDA events)",
                    "families": {}, "atb_over_symmetric": {}}
        for fam, tilings in ABLATION_FAMILIES.items():
            ablation["families"][fam] = [{"tiling": list(t), "rho_per_core": rho_per_core(t), "tflops": tf(t)} for t in tilings]
            ablation["atb_over_symmetric"][fam] = max(tf(t) for t in tilings[1:]) / tf(tilings[0])

        library = {"tflops": 2.0 * M * N * K / (min(lib_ms) * 1e-3) / 1e12, "headline_tiling_tflops": tf(t_head),
                   "how": "torch.matmul (cuBLAS) on bf16 A, B of the same shape, no conversion, timed next to the headline "
                          "tiling in the ablation walk (best of 2 x 5 launches each)"}
        library["headline_over_library"] = library["headline_tiling_tflops"] / library["tflops"]

        # sustained: the headline GEMM back to back for >= 2 s, so that the GPU settles under its power cap
        n_launch = max(200, int(SUSTAINED_SECONDS * 1e3 / gemm_ms))
        s_sampler = ClockSampler(physical_gpu_index(local_rank))
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        stream.synchronize()
        s_sampler.start()
        s0.record(stream)
        for _ in range(n_launch):
            atb.atb_gemm(M, N, K, *t_head, mant, plane, B_dev, C_dev, stream=stream)
        s1.record(stream)
        stream.synchronize()
        s_clocks = s_sampler.stop()
        atb.atb_device_status(stream)
        s_ms = s0.elapsed_time(s1)
        # and the library GEMM the same way, for as many launches
        l0, l1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            l0.record(stream)
            for _ in range(n_launch):
                torch.matmul(A_lib, B_dev, out=C_lib)
            l1.record(stream)
        stream.synchronize()
        library["sustained_tflops"] = 2.0 * M * N * K * n_launch / (l0.elapsed_time(l1) * 1e-3) / 1e12
        sustained = {"launches": n_launch, "seconds": s_ms * 1e-3,
                     "achieved": 2.0 * M * N * K * n_launch / (s_ms * 1e-3) / 1e12, "clocks": s_clocks}

    total_ms, gemm_ms, e2e_ms, quant_ms = max_over_ranks([total_ms, gemm_ms, e2e_ms, quant_ms], dev, world)

    if rank == 0:
        peaks, peak_src = load_peaks()
        flops = 2.0 * M * N * K
        ms_per_step = total_ms / args.steps
        value = aggregate_tflops(flops, world, ms_per_step)
        achieved = flops / (gemm_ms * 1e-3) / 1e12
        T_MA, T_MC, T_K, T_N = tiling_used[0]
        # T_MC = 256, T_K = 64, T_N = 512 runs on a CTA pair, a kernel of its own, and so does T_MC = 128, T_K = 128,
        # T_N = 256 on more than one tile row (two stacked tiles per pair)
        stacked = (T_MC, T_K, T_N) == (128, 128, 256) and M > 128
        gemm_kernel = "atb_gemm_pair_kernel" if (T_MC, T_K, T_N) == (256, 64, 512) or stacked else "atb_gemm_kernel"
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOPS", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": name, "M": M, "N": N, "K": K,
                       "A": f"BFP16 quantised on device from seeded {c['A']} fp32", "B": "bf16, seeded normal",
                       "tiling": {"T_MA": T_MA, "T_MC": T_MC, "T_K": T_K, "T_N": T_N,
                                  "chosen_by": "flag" if args.tiling else "atb_select_tiling",
                                  "rho_per_core": rho_per_core((T_MA, T_MC, T_K, T_N)),
                                  "note": ("CTA-pair tiling: two 128 x 256 tiles, one above the other, on the two SMs of a "
                                           "pair that share their B tiles (Eq. 2); T_MA = 128 buffers symmetrically") if stacked
                                  else ("CTA-pair tiling: each SM holds 128 of the 256 rows, so T_MA = 128 buffers "
                                        "symmetrically per SM and the B tile is shared by two SMs (Eq. 2)")
                                  if gemm_kernel == "atb_gemm_pair_kernel" else "single-CTA tiling"},
                       "step": "atb_quantize_bfp16 + atb_select_tiling + atb_gemm",
                       "l2": "inputs larger than L2 (A fp32 %d MB, B %d MB, C %d MB per step)" % (
                           M * K * 4 >> 20, K * N * 2 >> 20, M * N * 2 >> 20),
                       "parallelism": "replicas, one full GEMM per GPU" if world > 1 else "single GPU"},
            "clocks": clocks,
            "e2e": {"value": aggregate_tflops(flops, world, e2e_ms), "unit": "TFLOPS",
                    "h2d_bytes_per_step": A_host.numel() * 4 + B_host.numel() * 2,
                    "d2h_bytes_per_step": C_host.numel() * 2, "ms_per_step": e2e_ms, "steps": e2e_steps,
                    "how": "wall clock over pipelined steps: upload, kernels and download of neighbouring steps overlap on three streams"},
            "gpu_launches": 2 * args.steps,
            "roofline": {"bound": "tensor", "kernel": gemm_kernel, "achieved": achieved,
                         "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"],
                         "peak_source": f"{peak_src} cuBLAS bf16 burst (a kernel timed alone, launch by launch)",
                         "frac_of_nominal": achieved / NOMINAL_BF16_TFLOPS, "nominal_peak": NOMINAL_BF16_TFLOPS,
                         "kernel_ms": gemm_ms, "traffic": load_ncu_traffic().get((name, gemm_kernel)),
                         "compulsory_bytes": 1.125 * M * K + 2.0 * K * N + 2.0 * M * N},
            "quantize": {"bound": "hbm", "achieved": M * K * 5.125 / (quant_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                         "unit": "GB/s", "frac": M * K * 5.125 / (quant_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                         "kernel_ms": quant_ms},
        }
        if sustained is not None:
            mhz = sustained["clocks"].get("sm_mhz")
            sustained.update({"peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                              "frac": sustained["achieved"] / peaks["bf16_tflops_sustained"],
                              "peak_source": f"{peak_src} cuBLAS bf16 back to back under the power cap",
                              "frac_of_nominal": sustained["achieved"] / NOMINAL_BF16_TFLOPS,
                              "flop_per_cycle_per_sm": (sustained["achieved"] * 1e12 / (148 * mhz * 1e6)) if mhz else None})
            line["roofline"]["sustained"] = sustained
        if ablation is not None:
            line["ablation"] = ablation
            line["roofline"]["library_bf16_gemm_same_run"] = library
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_oracle_sample(name, args.cpu_seconds)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def run_entry(args):
    """--entry bfp16_out | config1 | config2: the further GEMM entry points on the same workload, one GPU,
    device-resident input.  A step is what the entry needs per batch of A: quantise A where the entry
    takes BFP16 A, then the GEMM.  B (and the planes of B transposed) are prepared once, like weights.
    The line has the fields of the main line that apply (no end-to-end leg, no CPU baseline)."""
    import torch
    import paper_2511_16041_b200 as atb
    from paper_2511_16041_b200 import inputs

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback of the hot path")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    atb.load_library()
    name = args.workload
    c = inputs.CONFIGS[name]
    M, N, K = c["M"], c["N"], c["K"]
    A_dev = torch.from_numpy(inputs.make_A(c["A"], M, K, inputs.BASE_SEED)).to(dev)
    B_dev = torch.from_numpy(inputs.make_B_bits(K, N, c["b_scale"]).view(np.int16)).to(dev).view(torch.bfloat16)
    stream = torch.cuda.Stream(dev)
    mant = torch.empty((M, K), dtype=torch.int8, device=dev)
    plane = torch.empty(atb.atb_bfp16_exp_bytes(M, K), dtype=torch.uint8, device=dev)
    tiling = tuple(args.tiling) if args.tiling else (128, 256, 64, 256)
    if args.entry == "bfp16_out":
        if not args.tiling:         # the selection's pick where this entry has that tiling
            best, _ = atb.atb_select_tiling(M, N, K)
            pick = (best.T_MA, best.T_MC, best.T_K, best.T_N)
            if pick[0] in (64, 128) and (pick[1:] == (128, 128, 256) or (pick[2] == 64 and (pick[1], pick[3]) in (
                    (128, 128), (128, 256), (256, 128), (256, 256), (256, 512)))):
                tiling = pick
        Cm = torch.empty((M, N), dtype=torch.int8, device=dev)
        Ce = torch.empty(atb.atb_bfp16_exp_bytes(M, N), dtype=torch.uint8, device=dev)
        on_pair = tiling[1:] == (256, 64, 512) or (tiling[1:] == (128, 128, 256) and M > 128)
        kname = "atb_gemm_pair_kernel" if on_pair else "atb_gemm_kernel"
        kernel, what = kname + " (quantising epilogue)", "atb_quantize_bfp16 + atb_gemm_bfp16_out"
        quantises = True
        call = lambda: atb.atb_gemm_bfp16_out(M, N, K, *tiling, mant, plane, B_dev, Cm, Ce, stream=stream)
    else:
        Bt_m, Bt_e = atb.atb_quantize_bfp16(B_dev.float().t().contiguous())      # planes of B transposed, once
        # T_MA is free; T_MC = 512 is the CTA pair that shares the converted B tile, 256 one SM
        tiling = tuple(args.tiling) if args.tiling else (128, 512, 64, 256)
        if args.entry == "config1":
            A16 = A_dev.to(torch.bfloat16)
            C = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
            form = "CTA pair" if tiling[1] == 512 else "single CTA"
            kernel, what, quantises = f"atb_gemm_cfg_kernel<A bf16, C bf16, {form}>", "atb_gemm_config_tiled(1)", False
            call = lambda: atb.atb_gemm_config_tiled(1, M, N, K, *tiling, A16, None, Bt_m, Bt_e, C, stream=stream)
        else:
            Cm = torch.empty((M, N), dtype=torch.int8, device=dev)
            Ce = torch.empty(atb.atb_bfp16_exp_bytes(M, N), dtype=torch.uint8, device=dev)
            form = "CTA pair" if tiling[1] == 512 else "single CTA"
            kernel, what, quantises = f"atb_gemm_cfg_kernel<A BFP16, C BFP16, {form}>", "atb_quantize_bfp16 + atb_gemm_config_tiled(2)", True
            call = lambda: atb.atb_gemm_config_tiled(2, M, N, K, *tiling, mant, plane, Bt_m, Bt_e, Cm, Ce, stream=stream)
    torch.cuda.synchronize()

    def step(ev=None):
        if quantises:
            atb.atb_quantize_bfp16(A_dev, mant, plane, stream=stream)
        if ev is not None:
            ev[0].record(stream)
        call()
        if ev is not None:
            ev[1].record(stream)

    for _ in range(max(args.warmup, 3)):
        step()
    atb.atb_device_status(stream)
    sampler = ClockSampler(physical_gpu_index(0))
    events = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    sampler.start()
    t_begin.record(stream)
    for i in range(args.steps):
        step(events[i])
    t_end.record(stream)
    stream.synchronize()
    clocks = sampler.stop()
    atb.atb_device_status(stream)
    ms_per_step = t_begin.elapsed_time(t_end) / args.steps
    gemm_ms = sum(a.elapsed_time(b) for a, b in events) / args.steps
    peaks, peak_src = load_peaks()
    flops = 2.0 * M * N * K
    achieved = flops / (gemm_ms * 1e-3) / 1e12
    line = {"metric": METRIC + " [entry " + args.entry + "]", "value": flops / (ms_per_step * 1e-3) / 1e12, "unit": "TFLOPS",
            "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": name, "M": M, "N": N, "K": K, "entry": args.entry, "step": what,
                       "tiling": dict(zip(("T_MA", "T_MC", "T_K", "T_N"), tiling)),
                       "l2": "inputs larger than L2", "parallelism": "single GPU"},
            "clocks": clocks, "e2e": None, "gpu_launches": (2 if quantises else 1) * args.steps,
            "roofline": {"bound": "tensor", "kernel": kernel, "achieved": achieved, "peak": peaks["bf16_tflops"],
                         "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"],
                         "peak_source": f"{peak_src} cuBLAS bf16 burst", "kernel_ms": gemm_ms, "traffic": None}}
    print(json.dumps(line))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--tiling", type=int, nargs=4, metavar=("T_MA", "T_MC", "T_K", "T_N"), default=None)
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-ablation", action="store_true", help="skip the T_MA ablation and the sustained leg")
    ap.add_argument("--stub-step", action="store_true",
                    help="host-only rehearsal of the multi-rank plumbing (gloo, no GPU work); the line is marked as a stub")
    ap.add_argument("--entry", default="gemm", choices=["gemm", "bfp16_out", "config1", "config2"],
                    help="gemm: the headline hot path (default); the others time the further entry points")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return spawn_ranks(args)
    if args.stub_step:
        return run_stub(args)
    if args.entry != "gemm":
        return run_entry(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
