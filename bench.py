#!/usr/bin/env python
"""Benchmark of the block-scaled FP4 quantize + scale-search + MSE hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl mxq|reference]

Workload (N = 1): the weight-shaped sweep -- 4096x4096 bf16, 0.02 * Student-t(nu=5), UE4M3 block
scales, no tensor scale, block sizes {2,4,8,16,32,64}.  One STEP is one pass of the whole hot path
over that batch: for every block size, quantize with abs-max, abs-max + prevent-zero, 4-over-6 and
brute force, each followed by the tensor MSE reduction; plus the hierarchical leg (tensor abs-max ->
device-resident global scale -> abs-max quantize at block 16 -> MSE) and one de-quantization.
Successive passes read different tensors out of a rotating set larger than L2, so inputs come from
HBM.  `value` = elements quantized per second over the whole job (all passes, all ranks).

With N > 1 (torchrun, one rank per GPU) every rank runs the same sweep on its own tensors: weak
scaling, no data-path collective; the timed region is bracketed by barrier + synchronize and the
time is the maximum over ranks.

`--impl reference` times the CPU oracle (oracle/mxq_oracle.c) on the host cores on a bounded sample
of the same workload and prints the same JSON line with "impl": "reference".
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "GElem/s quantize+MSE per recipe (abs-max, 4/6, brute force); % HBM/ALU roofline"
UNIT = "GElem/s"
ROWS, COLS = 4096, 4096
N_ELEM = ROWS * COLS
BLOCKS = (2, 4, 8, 16, 32, 64)
N_ROTATE = 8                      # 8 x 32 MiB inputs = 256 MiB > 126 MB L2
UE4M3 = 1
ABSMAX, ABSMAX_PZ, R4O6, BRUTE = 0, 1, 2, 4
RECIPE_NAME = {ABSMAX: "absmax", ABSMAX_PZ: "absmax_pz", R4O6: "4o6", BRUTE: "brute"}
N_CODES_UE4M3 = 127
ALU_LANES_PER_SM = 128            # 4 schedulers x 32 lanes, one instruction per scheduler per clock
CPU_SAMPLE_ELEMS = 1 << 20
REFERENCE_BUDGET_S = 35.0        # wall-clock target of a whole --impl reference run
STREAM_ELEMS = 1 << 27            # tensor size of the streaming (HBM-bound) kernel measurements
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under
# profiles/ (same kernel build, same launch configuration); set an entry to None when its kernel changes.
# smsp__issue_active.avg.pct_of_peak_sustained_active of the brute-force kernel in the same capture
NCU_BRUTE_ISSUE_ACTIVE_PCT = 70.8
NCU_TRAFFIC_BYTES = {
    "k_brute<bf16,B=16,UE4M3>@16Mi": 33.620224e6 + 0.016128e6,
    "k_quantize<bf16,B=16,UE4M3,absmax>@128Mi": 268.471552e6 + 82.490624e6,
    "k_quantize<bf16,B=16,UE4M3,4o6>@128Mi": 268.489216e6 + 83.071488e6,
    "k_quantize<f32,B=16,UE4M3,absmax>@128Mi": 536.895488e6 + 95.571200e6,
}


def pass_list():
    return [(B, r) for B in BLOCKS for r in (ABSMAX, ABSMAX_PZ, R4O6, BRUTE)]


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "sm_max_mhz": float(p.get("sm_max_mhz", 1965.0)), "source": "measured"}
    return {"hbm_gbs": 6650.0, "sm_max_mhz": 1965.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons every 200 ms while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: str):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "200",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------------
# CPU oracle legs (cpu_baseline of the normal run; the whole of --impl reference)
# ------------------------------------------------------------------------------------------------
def oracle_sample_run(sample_bits, threads: int) -> tuple[float, float]:
    """One pass of the step's recipe mix over the sample with the oracle; returns (elements, seconds)."""
    from oracle import mxq_oracle as orc
    n = sample_bits.size
    t0 = time.perf_counter()
    elems = 0
    for B, r in pass_list():
        _, _, sse = orc.quantize(sample_bits, B, orc.UE4M3, r, 1.0, threads=threads)
        orc.tensor_mse(sse, n)
        elems += n
    amax = orc.tensor_amax(sample_bits)
    g = float(orc.global_scale_from_amax(amax))
    codes, scales, sse = orc.quantize(sample_bits, 16, orc.UE4M3, orc.ABSMAX, g, threads=threads)
    orc.tensor_mse(sse, n)
    orc.dequantize(codes, scales, n, 16, orc.UE4M3, g, orc.BF16)
    elems += n
    return float(elems), time.perf_counter() - t0


def host_threads() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return os.cpu_count() or 1


def host_sample(seed: int, n: int):
    import torch
    from paper_2605_08565_b200 import inputs
    return inputs.to_numpy_bits(inputs.student_t(n, 5, 0.02, seed, torch.bfloat16, "cpu"))


def run_reference(args) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import mxq_oracle as orc
    orc.build()
    threads = host_threads()
    # Size the per-step sample so that the whole run (warm-up + steps) stays near REFERENCE_BUDGET_S:
    # probe the oracle's rate on 4096 elements, then give every step the same prefix of tensor 0.
    full = host_sample(2, CPU_SAMPLE_ELEMS // 8)
    pe, ps = oracle_sample_run(full[: 1 << 12], 1)
    rate1 = pe / max(ps, 1e-6)                                  # elements of the recipe mix per second, one thread
    passes = len(pass_list()) + 1
    trips = max(1, args.steps + args.warmup)
    n_sample, use = 256, 1
    for t in sorted({1, 2, 4, 8, threads}):                     # most threads that still get >= 2048 elements each
        if t > threads:
            continue
        n_t = int(min(full.size, REFERENCE_BUDGET_S * rate1 * t / trips / passes)) // 64 * 64
        if t == 1 or n_t >= 2048 * t:
            n_sample, use = max(256, n_t), t
    threads = use
    sample = full[:n_sample]
    for _ in range(args.warmup):
        oracle_sample_run(sample, threads)
    elems, secs = 0.0, 0.0
    for _ in range(args.steps):
        e, s = oracle_sample_run(sample, threads)
        elems += e
        secs += s
    value = elems / secs / 1e9
    sample_desc = (f"first {sample.size} elements of the 4096x4096 bf16 Student-t tensor, every pass of the step "
                   f"(6 block sizes x abs-max, abs-max+pz, 4-over-6, brute force, + hierarchical leg)")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": secs / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": "weight sweep 4096x4096 bf16 Student-t(5)*0.02, UE4M3, B in {2..64} (bounded sample)",
                   "sample_elems": int(sample.size)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample_desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------
class Workload:
    def __init__(self, rank: int, device):
        import torch
        from paper_2605_08565_b200 import binding as mxq
        from paper_2605_08565_b200 import dist, inputs
        self.torch, self.mxq = torch, mxq
        self.device = device
        self.x = [inputs.student_t(N_ELEM, 5, 0.02, dist.rank_seed(2, rank, i), torch.bfloat16, device)
                  for i in range(N_ROTATE)]
        self.codes = torch.empty(N_ELEM // 2, dtype=torch.uint8, device=device)
        self.scales = torch.empty(N_ELEM // 2, dtype=torch.uint8, device=device)
        self.sse = torch.empty(N_ELEM // 2, dtype=torch.float32, device=device)
        self.passes = pass_list()
        self.mse = torch.zeros(len(self.passes) + 1, dtype=torch.float64, device=device)
        self.ws = torch.empty(mxq.mxq_tensor_mse_workspace_bytes(N_ELEM // 2) // 8, dtype=torch.float64, device=device)
        self.amax = torch.empty(1, dtype=torch.float32, device=device)
        self.g = torch.empty(1, dtype=torch.float32, device=device)
        self.xhat = torch.empty(N_ELEM, dtype=torch.bfloat16, device=device)
        self.rot = 0
        self.timers = {}          # (B, recipe) -> list of (start, stop) event pairs
        self.elems_per_step = float(N_ELEM * (len(self.passes) + 1))

    def _next_input(self):
        x = self.x[self.rot % len(self.x)]
        self.rot += 1
        return x

    def one_pass(self, x, B, recipe, slot, timed_keys=()):
        mxq, torch = self.mxq, self.torch
        key = (B, recipe)
        ev = None
        if key in timed_keys:
            ev = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
            ev[0].record()
        mxq.mxq_quantize_ex(x, N_ELEM, B, UE4M3, recipe, 1.0, None, self.codes, self.scales, self.sse)
        if ev is not None:
            ev[1].record()
            self.timers.setdefault(key, []).append(ev)
        mxq.mxq_tensor_mse(self.sse, N_ELEM // B, N_ELEM, self.mse[slot:slot + 1], self.ws)

    def step(self, x_override=None, timed_keys=()):
        mxq = self.mxq
        for slot, (B, r) in enumerate(self.passes):
            x = x_override if x_override is not None else self._next_input()
            self.one_pass(x, B, r, slot, timed_keys)
        # hierarchical leg + de-quantization
        x = x_override if x_override is not None else self._next_input()
        mxq.mxq_tensor_amax(x, N_ELEM, self.amax, self.g)
        mxq.mxq_quantize_ex(x, N_ELEM, 16, UE4M3, ABSMAX, 1.0, self.g, self.codes, self.scales, self.sse)
        slot = len(self.passes)
        mxq.mxq_tensor_mse(self.sse, N_ELEM // 16, N_ELEM, self.mse[slot:slot + 1], self.ws)
        mxq.mxq_dequantize(self.codes, self.scales, N_ELEM, 16, UE4M3, 1.0, self.xhat)

    def kernel_ms(self, key):
        evs = self.timers.get(key, [])
        return (sum(a.elapsed_time(b) for a, b in evs) / len(evs)) if evs else None


def algorithmic_bytes(n: int, elem_bytes: int, B: int) -> float:
    """Input + packed codes + scale bytes + block SSE of one fused quantize launch."""
    return n * (elem_bytes + 0.5 + 5.0 / B)


def streaming_rooflines(torch, mxq, device, peaks):
    """HBM-bound kernels on a tensor far larger than L2 (134M elements), ten launches back to back
    per CUDA-event pair, outside the timed region of the step: the 16.8M-element launches of the
    step itself last 8-20 us and are dominated by launch ramp."""
    from paper_2605_08565_b200 import inputs
    out = {}
    n = STREAM_ELEMS

    def entry(name, fn, nbytes, traffic):
        for _ in range(3):
            fn()
        times = []
        for _ in range(5):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(10):
                fn()
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1) / 10)
        ms = statistics.median(times)
        ach = nbytes / (ms * 1e-3) / 1e9
        out[name] = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": ach / peaks["hbm_gbs"], "frac_of_nominal_8TBs": ach / 8000.0, "traffic": traffic,
                     "ms_per_launch": ms, "gelem_s": n / (ms * 1e-3) / 1e9, "elems": n,
                     "peak_source": peaks["source"], "l2": "input larger than L2"}

    for name, dt, recipe, B, key in (
            ("absmax_bf16_B16", torch.bfloat16, ABSMAX, 16, "k_quantize<bf16,B=16,UE4M3,absmax>@128Mi"),
            ("4o6_bf16_B16", torch.bfloat16, R4O6, 16, "k_quantize<bf16,B=16,UE4M3,4o6>@128Mi"),
            ("absmax_f32_B16", torch.float32, ABSMAX, 16, "k_quantize<f32,B=16,UE4M3,absmax>@128Mi"),
            ("4o6_f32_B16", torch.float32, R4O6, 16, None),
            ("absmax_bf16_B64", torch.bfloat16, ABSMAX, 64, None),
            ("absmax_f32_B64", torch.float32, ABSMAX, 64, None)):
        codes, scales, sse = mxq.alloc_outputs(n, B, device)
        x = inputs.student_t(n, 5, 0.02, 2, dt, device)
        fn = lambda: mxq.mxq_quantize_ex(x, n, B, UE4M3, recipe, 1.0, None, codes, scales, sse)
        entry(name, fn, algorithmic_bytes(n, x.element_size(), B), NCU_TRAFFIC_BYTES[key] if key else None)
        del x
    # the other two kernels of the path: tensor abs-max (reads n elements) and de-quantization
    x = inputs.student_t(n, 5, 0.02, 2, torch.bfloat16, device)
    amax = torch.empty(1, dtype=torch.float32, device=device)
    entry("tensor_amax_bf16", lambda: mxq.mxq_tensor_amax(x, n, amax), n * 2.0, None)
    codes, scales, sse = mxq.alloc_outputs(n, 16, device)
    mxq.mxq_quantize_ex(x, n, 16, UE4M3, ABSMAX, 1.0, None, codes, scales, sse)
    xh = torch.empty(n, dtype=torch.float32, device=device)
    entry("dequantize_B16_to_f32", lambda: mxq.mxq_dequantize(codes, scales, n, 16, UE4M3, 1.0, xh), n * (0.5 + 1.0 / 16 + 4.0), None)
    return out


def pruned_sweep_report(torch, mxq, wl):
    """The brute-force passes of the step once more with the pruned sweep switched on (outside the
    timed region; `value` and `roofline` are always the full sweep): per block size the time of both
    sweeps over the rotating tensors, launches back to back, and whether the outputs are identical."""
    out = {}
    x0 = wl.x[0]
    n = x0.numel()
    try:
        for B in BLOCKS:
            bufs = {}
            ms = {}
            for mode in (0, 1):
                mxq.mxq_set_option(mxq.MXQ_OPT_BRUTE_PRUNE, mode)
                codes, scales, sse = mxq.alloc_outputs(n, B, x0.device)
                fn = lambda x: mxq.mxq_quantize_ex(x, n, B, UE4M3, BRUTE, 1.0, None, codes, scales, sse)
                fn(x0)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for x in wl.x:
                    fn(x)
                e1.record()
                fn(x0)
                torch.cuda.synchronize()
                ms[mode] = e0.elapsed_time(e1) / len(wl.x)
                bufs[mode] = (codes, scales, sse)
            same = all(torch.equal(a.view(torch.uint8), b.view(torch.uint8)) for a, b in zip(bufs[0], bufs[1]))
            out[f"B{B}"] = {"full_ms": ms[0], "pruned_ms": ms[1], "speedup": ms[0] / ms[1], "outputs_identical": bool(same)}
    finally:
        mxq.mxq_set_option(mxq.MXQ_OPT_BRUTE_PRUNE, 0)
    return out


def run_gpu(args) -> None:
    import torch
    from paper_2605_08565_b200 import binding as mxq
    from paper_2605_08565_b200 import dist

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: libmxq has no CPU fallback")
    rank, local_rank, world = dist.init("nccl")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    mxq.load_library()
    peaks = measured_peaks()

    wl = Workload(rank, device)
    hot = {(16, BRUTE), (16, ABSMAX), (16, R4O6)}   # kernels timed live for the roofline entries

    for _ in range(args.warmup):
        wl.step()
    torch.cuda.synchronize()
    wl.timers.clear()

    # ---- device-resident timing ---------------------------------------------------------------
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(device).uuid)
    except Exception:
        gpu_id = str(local_rank)
    sampler = ClockSampler(gpu_id)
    if rank == 0:
        sampler.start()
    dist.barrier()
    torch.cuda.synchronize()
    launches0 = mxq.mxq_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        wl.step(timed_keys=hot)
    e1.record()
    torch.cuda.synchronize()
    dist.barrier()
    launches = mxq.mxq_launch_count() - launches0
    local_s = e0.elapsed_time(e1) / 1e3
    clocks = sampler.stop() if rank == 0 else None
    value, t_max = dist.whole_job_throughput(wl.elems_per_step * args.steps, local_s)
    mse_host = wl.mse.cpu().numpy().copy()

    # ---- end to end: host buffers, H2D of the step's input and D2H of its results every step ----
    # The input of step i + 1 is copied on a second stream into the other of two device buffers while
    # step i computes; every copy is awaited by the compute stream, so all of them lie inside the
    # timed region.
    host_in = wl.x[0].cpu().pin_memory()
    host_out = torch.empty(wl.mse.numel(), dtype=torch.float64).pin_memory()
    dev_in = [torch.empty_like(wl.x[0]), torch.empty_like(wl.x[0])]
    copy_stream = torch.cuda.Stream(device=device)
    main_stream = torch.cuda.current_stream(device)

    def e2e_loop(n_steps):
        ready = [torch.cuda.Event(), torch.cuda.Event()]
        free = [torch.cuda.Event(), torch.cuda.Event()]
        for ev in free:
            ev.record(main_stream)

        def enqueue_copy(i):
            with torch.cuda.stream(copy_stream):
                copy_stream.wait_event(free[i % 2])
                dev_in[i % 2].copy_(host_in, non_blocking=True)
                ready[i % 2].record(copy_stream)

        enqueue_copy(0)
        for i in range(n_steps):
            if i + 1 < n_steps:
                enqueue_copy(i + 1)
            main_stream.wait_event(ready[i % 2])
            wl.step(x_override=dev_in[i % 2])
            free[i % 2].record(main_stream)
            host_out.copy_(wl.mse, non_blocking=True)

    e2e_loop(2)
    torch.cuda.synchronize()
    dist.barrier()
    e0.record()
    e2e_loop(args.steps)
    e1.record()
    torch.cuda.synchronize()
    dist.barrier()
    e2e_value, _ = dist.whole_job_throughput(wl.elems_per_step * args.steps, e0.elapsed_time(e1) / 1e3)

    if rank != 0:
        dist.shutdown()
        return

    # ---- rooflines of the kernels timed live --------------------------------------------------
    sm_mhz = (clocks or {}).get("sm_mhz") or peaks["sm_max_mhz"]
    n_sm = torch.cuda.get_device_properties(device).multi_processor_count
    alu_peak_max = n_sm * ALU_LANES_PER_SM * peaks["sm_max_mhz"] * 1e6 / 1e12          # Tlaneop/s at max clock
    brute_ms = wl.kernel_ms((16, BRUTE))
    brute_ops = N_ELEM * N_CODES_UE4M3 * 4.0                                            # 4 lane-ops per element-code
    brute_ach = brute_ops / (brute_ms * 1e-3) / 1e12
    roofline = {"kernel": "k_brute<bf16,B=16,UE4M3>", "bound": "alu", "achieved": brute_ach, "peak": alu_peak_max,
                "unit": "Tlaneop/s", "frac": brute_ach / alu_peak_max,
                "traffic": NCU_TRAFFIC_BYTES["k_brute<bf16,B=16,UE4M3>@16Mi"],
                "peak_source": f"{n_sm} SMs x 128 lanes x {peaks['sm_max_mhz']:.0f} MHz (max SM clock, {peaks['source']})",
                "frac_at_observed_clock": brute_ach / (n_sm * ALU_LANES_PER_SM * sm_mhz * 1e6 / 1e12),
                "ms_per_launch": brute_ms, "ncu_issue_active_pct": NCU_BRUTE_ISSUE_ACTIVE_PCT}
    hbm = {}
    for name, key in (("absmax_B16", (16, ABSMAX)), ("4o6_B16", (16, R4O6))):
        ms = wl.kernel_ms(key)
        ach = algorithmic_bytes(N_ELEM, 2, 16) / (ms * 1e-3) / 1e9
        hbm[name] = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": ach / peaks["hbm_gbs"], "frac_of_nominal_8TBs": ach / 8000.0, "traffic": None,
                     "ms_per_launch": ms, "gelem_s": N_ELEM / (ms * 1e-3) / 1e9, "peak_source": peaks["source"]}
    streaming = None if args.skip_streaming else streaming_rooflines(torch, mxq, device, peaks)
    pruned = None if args.skip_streaming else pruned_sweep_report(torch, mxq, wl)
    per_recipe = {"brute_B16": N_ELEM / (brute_ms * 1e-3) / 1e9, "absmax_B16": hbm["absmax_B16"]["gelem_s"],
                  "4o6_B16": hbm["4o6_B16"]["gelem_s"]}

    # ---- CPU oracle on a bounded sample of the same workload ------------------------------------
    from oracle import mxq_oracle as orc
    orc.build()
    threads = host_threads()
    sample = host_sample(dist.rank_seed(2, 0, 0), CPU_SAMPLE_ELEMS)
    oracle_sample_run(sample[: 1 << 12], threads)
    c_elems, c_secs = oracle_sample_run(sample, threads)
    cpu_baseline = {"value": c_elems / c_secs / 1e9, "unit": UNIT, "cores": threads, "kind": "oracle",
                    "seconds": c_secs,
                    "sample": f"first {CPU_SAMPLE_ELEMS} elements of tensor 0, every pass of one step"}

    print(json.dumps({
        "metric": METRIC, "value": value / 1e9, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": t_max / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": "weight sweep: 4096x4096 bf16 0.02*Student-t(5), UE4M3 block scales, g=1, "
                               "B in {2,4,8,16,32,64} x {abs-max, abs-max+pz, 4-over-6, brute force} + MSE each; "
                               "+ hierarchical leg (amax, g, abs-max B=16, MSE) + dequantize",
                   "elements_per_step": wl.elems_per_step, "passes_per_step": len(wl.passes) + 1,
                   "l2": f"inputs rotate over {N_ROTATE} tensors (256 MiB) > 126 MB L2"},
        "roofline": roofline, "roofline_hbm": hbm, "roofline_hbm_streaming": streaming,
        "per_recipe_gelem_s": per_recipe, "brute_pruned_sweep": pruned,
        "cpu_baseline": cpu_baseline,
        "e2e": {"value": e2e_value / 1e9, "unit": UNIT, "h2d_bytes_per_step": int(host_in.numel() * 2),
                "d2h_bytes_per_step": int(host_out.numel() * 8)},
        "gpu_launches": int(launches), "clocks": clocks,
        "mse_by_block_size": {RECIPE_NAME[r] + f"_B{B}": float(mse_host[i]) for i, (B, r) in enumerate(wl.passes)},
    }))
    dist.shutdown()


def run_single_kernel(args) -> None:
    """Time one kernel alone (`--kernel`): used for sweeps and as the small case for ncu captures."""
    import torch
    from paper_2605_08565_b200 import binding as mxq
    from paper_2605_08565_b200 import inputs
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    n = args.elems - args.elems % 64
    dtype = torch.bfloat16 if args.dtype == "bf16" else torch.float32
    fmt = {"ue8m0": 0, "ue4m3": 1, "ue5m3": 2}[args.fmt]
    x = inputs.student_t(n, 5, 0.02, 2, dtype, dev) if args.dtype == "bf16" else inputs.laplace(n, 5, dtype, dev)
    B = args.block
    codes, scales, sse = mxq.alloc_outputs(n, B, dev)
    g = args.global_scale
    recipe = {"absmax": 0, "absmax_pz": 1, "4o6": 2, "4o6_pz": 3, "brute": 4, "brute_pz": 5}.get(args.kernel)
    if args.prune:
        mxq.mxq_set_option(mxq.MXQ_OPT_BRUTE_PRUNE, 1)
    out = torch.empty(n, dtype=dtype, device=dev)
    amax = torch.empty(1, dtype=torch.float32, device=dev)
    mse = torch.empty(1, dtype=torch.float64, device=dev)
    ws = torch.empty(mxq.mxq_tensor_mse_workspace_bytes(n // B) // 8, dtype=torch.float64, device=dev)
    eb = x.element_size()
    if recipe is not None:
        fn = lambda: mxq.mxq_quantize_ex(x, n, B, fmt, recipe, g, None, codes, scales, sse)
        nbytes = algorithmic_bytes(n, eb, B)
    elif args.kernel == "amax":
        fn = lambda: mxq.mxq_tensor_amax(x, n, amax)
        nbytes = n * eb
    elif args.kernel == "mse":
        fn = lambda: mxq.mxq_tensor_mse(sse, n // B, n, mse, ws)
        nbytes = 4.0 * n / B
    elif args.kernel == "dequant":
        mxq.mxq_quantize_ex(x, n, B, fmt, 0, g, None, codes, scales, sse)
        fn = lambda: mxq.mxq_dequantize(codes, scales, n, B, fmt, g, out)
        nbytes = n * (eb + 0.5 + 1.0 / B)
    else:
        raise SystemExit(f"unknown --kernel {args.kernel}")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if n * eb < (256 << 20) else None
    for _ in range(3):
        fn()
    times = []
    for _ in range(args.iters):
        if flush is not None:
            flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); fn(); e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    ms = statistics.median(times)
    res = {"kernel": args.kernel + ("+prune" if args.prune else ""), "block": B, "dtype": args.dtype, "fmt": args.fmt, "elems": n, "ms": ms,
           "gelem_s": n / ms / 1e6, "algorithmic_gb_s": nbytes / ms / 1e6,
           "l2": "flushed between iterations" if flush is not None else "input larger than L2"}
    if recipe in (4, 5):
        ncodes = 127 if fmt == 1 else 255
        res["tlaneop_s"] = n * ncodes * 4.0 / (ms * 1e-3) / 1e12
    print(json.dumps(res))


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--kernel", default=None, help="time one kernel alone: absmax|absmax_pz|4o6|4o6_pz|brute|brute_pz|amax|mse|dequant")
    ap.add_argument("--block", type=int, default=16)
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "f32"])
    ap.add_argument("--fmt", default="ue4m3", choices=["ue8m0", "ue4m3", "ue5m3"])
    ap.add_argument("--elems", type=int, default=1 << 27)
    ap.add_argument("--iters", type=int, default=5)
    ap.add_argument("--global-scale", type=float, default=1.0)
    ap.add_argument("--prune", action="store_true", help="with --kernel brute|brute_pz: the pruned sweep")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--skip-streaming", action="store_true",
                    help="leave out the measurements taken outside the timed step: the 134M-element streaming "
                         "launches and the pruned brute-force sweep (roofline_hbm_streaming, brute_pruned_sweep = null)")
    ap.add_argument("--impl", default="mxq", choices=["mxq", "reference"])
    args = ap.parse_args()
    if args.kernel:
        run_single_kernel(args)
        return
    if args.warmup < 3 and args.impl == "mxq":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
