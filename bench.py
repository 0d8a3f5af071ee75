#!/usr/bin/env python
"""Benchmark of the block-scaled FP4 quantize + scale-search + MSE hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl mxq|reference]
    python bench.py --config 1|2|3|4|5|all      one benchmark configuration, one recipe at a time
    python bench.py --kernel absmax|4o6|brute|...   one kernel alone (sweeps, ncu captures)

Workload of the default run (N = 1), one STEP = one pass of the whole hot path over one batch:

* bulk scale search: 16384 x 16384 fp32 Laplace(0,1), tensor abs-max -> device-resident tensor scale
  g = amax / 2688, then the full brute-force sweep for every block size in {2,4,8,16,32} and every
  scale format in {UE8M0, UE4M3, UE5M3}, each scored by the tensor MSE (15 sweeps; quantization and MSE
  are one call, ``mxq_quantize_mse``);
* weight leg: one matrix of each shape of an 8B-parameter Llama-style layer (4096x4096, 1024x4096,
  14336x4096, 4096x14336; bf16, Student-t(4)/sqrt(fan_in)), block sizes {8,16} x {UE4M3, UE5M3} x
  {abs-max, abs-max + prevent-zero, 4-over-6, 4-over-6 + prevent-zero}, tensor MSE after each;
* activation leg: 8192 x 4096 bf16 with 1 % outlier columns, block 16: hierarchical scaling (tensor
  abs-max -> g -> UE4M3 blocks) against UE5M3 blocks without a tensor scale, abs-max and 4-over-6,
  tensor MSE after each, and one de-quantization.

Inputs larger than L2 (the 1 GiB tensor), or visited so that no tensor is read twice within 126 MB of
other traffic (the legs walk their matrices round-robin).  `value` = elements quantized per second
over the whole job (all passes, all ranks).

With N > 1 (one rank per GPU; `--gpus N` starts the ranks itself when it was not started by torchrun)
every rank runs the same step on its own tensors: weak scaling, no data-path collective; the timed
region is bracketed by barrier + synchronize and the time is the maximum over ranks.

`--impl reference` times the CPU oracle (oracle/mxq_oracle.c) on the host cores on a bounded sample
of the same workload and prints the same JSON line with "impl": "reference".
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import re
import socket
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
UE8M0, UE4M3, UE5M3 = 0, 1, 2
ABSMAX, ABSMAX_PZ, R4O6, R4O6_PZ, BRUTE, BRUTE_PZ = 0, 1, 2, 3, 4, 5
RECIPE_NAME = {ABSMAX: "absmax", ABSMAX_PZ: "absmax_pz", R4O6: "4o6", R4O6_PZ: "4o6_pz", BRUTE: "brute",
               BRUTE_PZ: "brute_pz"}
FMT_NAME = {UE8M0: "ue8m0", UE4M3: "ue4m3", UE5M3: "ue5m3"}
N_CODES = {UE8M0: 255, UE4M3: 127, UE5M3: 255}
ALU_LANES_PER_SM = 128            # 4 schedulers x 32 lanes, one instruction per scheduler per clock
NOMINAL_HBM_GBS = 8000.0          # the bandwidth the targets are quoted against; the measured copy peak is lower

# ---- the step's workload -------------------------------------------------------------------------
SEARCH_ROWS = SEARCH_COLS = 16384
SEARCH_N = SEARCH_ROWS * SEARCH_COLS
SEARCH_BLOCKS = (2, 4, 8, 16, 32)
SEARCH_FMTS = (UE8M0, UE4M3, UE5M3)
WEIGHT_SHAPES = (("q", 4096, 4096, 0), ("k", 1024, 4096, 1), ("gate", 14336, 4096, 4), ("down", 4096, 14336, 6))
WEIGHT_BLOCKS = (8, 16)
WEIGHT_FMTS = (UE4M3, UE5M3)
WEIGHT_RECIPES = (ABSMAX, ABSMAX_PZ, R4O6, R4O6_PZ)
ACT_ROWS, ACT_COLS, ACT_ROTATE = 8192, 4096, 3
ACT_N = ACT_ROWS * ACT_COLS
ACT_PASSES = ((UE4M3, True, ABSMAX), (UE5M3, False, ABSMAX), (UE4M3, True, R4O6), (UE5M3, False, R4O6))

CPU_SAMPLE_ELEMS = 1 << 22        # per tensor, cpu_baseline leg (about 15 s on 16 host cores)
REFERENCE_BUDGET_S = 40.0         # wall-clock target of a whole --impl reference run
REF_SAMPLE_ELEMS = 1 << 18        # longest prefix per tensor the reference arm may take per step
STREAM_ELEMS = 1 << 27            # tensor size of the streaming (HBM-bound) kernel measurements


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "sm_max_mhz": float(p.get("sm_max_mhz", 1965.0)), "source": "measured"}
    return {"hbm_gbs": 6650.0, "sm_max_mhz": 1965.0, "source": "fallback"}


def kernel_source_digest(*names) -> str:
    """SHA-256 over the kernel sources a profile summary depends on (ties recorded ncu figures to the code)."""
    h = hashlib.sha256()
    for n in names:
        with open(os.path.join(ROOT, "paper_2605_08565_b200", "csrc", n), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def recorded_profile(fname: str, sources) -> dict:
    """Figures of a committed ncu summary (profiles/<fname>): returned only while the kernel sources still
    hash to the digest written in that file; otherwise the figures are stale and reported as such."""
    path = os.path.join(ROOT, "profiles", fname)
    out = {"file": "profiles/" + fname, "stale": True, "dram_bytes": None, "issue_active_pct": None, "elems": None}
    if not os.path.exists(path):
        return out
    txt = open(path).read()
    m = re.search(r"kernel_source_digest:\s*([0-9a-f]+)", txt)
    if not m or m.group(1) != kernel_source_digest(*sources):
        return out

    def num(key):
        mm = re.search(re.escape(key) + r"\s+([0-9.eE+-]+)\s*(\S*)", txt)
        if not mm:
            return None
        v = float(mm.group(1))
        unit = mm.group(2).lower()
        return v * {"kbyte": 1e3, "mbyte": 1e6, "gbyte": 1e9}.get(unit, 1.0)

    rd, wr = num("dram__bytes_read.sum"), num("dram__bytes_write.sum")
    me = re.search(r"elements_per_launch:\s*(\d+)", txt)
    out.update(stale=False, dram_bytes=(rd + wr) if rd is not None and wr is not None else None,
               issue_active_pct=num("smsp__issue_active.avg.pct_of_peak_sustained_active"),
               elems=int(me.group(1)) if me else None)
    return out


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


def host_threads() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return os.cpu_count() or 1


def algorithmic_bytes(n: int, elem_bytes: int, B: int) -> float:
    """Input + packed codes + scale bytes + block SSE of one fused quantize launch."""
    return n * (elem_bytes + 0.5 + 5.0 / B)


def pass_table():
    """Every quantize pass of one step: (leg, tensor key, elements, block, format, recipe, tensor scale?)."""
    rows = []
    for B in SEARCH_BLOCKS:
        for fmt in SEARCH_FMTS:
            rows.append(("search", "search", SEARCH_N, B, fmt, BRUTE, True))
    for B in WEIGHT_BLOCKS:
        for fmt in WEIGHT_FMTS:
            for r in WEIGHT_RECIPES:
                for name, rr, cc, _ in WEIGHT_SHAPES:
                    rows.append(("weight", "w_" + name, rr * cc, B, fmt, r, False))
    for i, (fmt, hier, r) in enumerate(ACT_PASSES):
        rows.append(("act", f"a_{i % ACT_ROTATE}", ACT_N, 16, fmt, r, hier))
    return rows


WORKLOAD_NAME = ("bulk scale search 16384x16384 fp32 Laplace, g=amax/2688, brute force full sweep, B in {2,4,8,16,32} x "
                 "{UE8M0,UE4M3,UE5M3} + MSE each; + weight leg (Llama-8B layer shapes 4096x4096, 1024x4096, 14336x4096, "
                 "4096x14336 bf16 t4/sqrt(fan_in), B in {8,16} x {UE4M3,UE5M3} x {abs-max, +pz, 4-over-6, +pz} + MSE each); "
                 "+ activation leg (8192x4096 bf16 outlier columns, B=16, hierarchical UE4M3 vs UE5M3, abs-max and "
                 "4-over-6 + MSE each, dequantize)")


# ------------------------------------------------------------------------------------------------
# Host-side inputs (the oracle legs and the end-to-end arm read these)
# ------------------------------------------------------------------------------------------------
def make_inputs(rank: int, device, n_limit: int | None = None):
    """The step's tensors, keyed as in pass_table(); n_limit keeps only a prefix of each (oracle legs)."""
    import torch
    from paper_2605_08565_b200 import dist, inputs

    def cut(n):
        return n if n_limit is None else min(n, n_limit)

    t = {"search": inputs.laplace(cut(SEARCH_N), dist.rank_seed(5, rank), torch.float32, device)}
    for name, rr, cc, idx in WEIGHT_SHAPES:
        t["w_" + name] = inputs.student_t(cut(rr * cc), 4, 1.0 / math.sqrt(cc), dist.rank_seed(4, rank, idx),
                                          torch.bfloat16, device)
    for i in range(ACT_ROTATE):
        if n_limit is None:
            t[f"a_{i}"] = inputs.outlier_columns(ACT_ROWS, ACT_COLS, dist.rank_seed(3, rank, i), dtype=torch.bfloat16,
                                                 device=device)
        else:
            rows = max(1, n_limit // ACT_COLS)
            t[f"a_{i}"] = inputs.outlier_columns(rows, ACT_COLS, dist.rank_seed(3, rank, i), dtype=torch.bfloat16,
                                                 device=device)
    return t


# ------------------------------------------------------------------------------------------------
# CPU oracle legs (cpu_baseline of the normal run; the whole of --impl reference)
# ------------------------------------------------------------------------------------------------
def oracle_step(samples: dict, threads: int, frac: float = 1.0) -> tuple[float, float]:
    """One step's pass list over host samples with the oracle; returns (elements, seconds).
    samples: key -> numpy bits (prefixes of the step's tensors); frac < 1 shortens every prefix."""
    from oracle import mxq_oracle as orc
    t0 = time.perf_counter()
    elems = 0
    g_of = {}
    for leg, key, _, B, fmt, recipe, hier in pass_table():
        x = samples[key]
        n = max(64, int(x.size * frac) // 64 * 64)
        x = x[:n]
        g = 1.0
        if hier:
            if (key, n) not in g_of:
                g_of[(key, n)] = float(orc.global_scale_from_amax(orc.tensor_amax(x)))
            g = g_of[(key, n)]
        codes, scales, sse = orc.quantize(x, B, fmt, recipe, g, threads=threads)
        orc.tensor_mse(sse, n)
        elems += n
    orc.dequantize(codes, scales, n, 16, fmt, g, orc.BF16)
    return float(elems), time.perf_counter() - t0


def run_reference(args) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    from oracle import mxq_oracle as orc
    from paper_2605_08565_b200 import inputs
    orc.build()
    threads = host_threads()
    full = {k: inputs.to_numpy_bits(v) for k, v in make_inputs(0, "cpu", REF_SAMPLE_ELEMS).items()}
    # Size the per-step sample so that the whole run (warm-up + steps) stays near REFERENCE_BUDGET_S:
    # probe the oracle's rate on a short prefix, then give every step the same prefix of every tensor.
    probe_frac = 4096.0 / REF_SAMPLE_ELEMS
    pe, ps = oracle_step(full, threads, probe_frac)
    rate = pe / max(ps, 1e-6)                                    # elements of the pass mix per second
    trips = max(1, args.steps + args.warmup)
    per_step_elems = REFERENCE_BUDGET_S * rate / trips
    frac = min(1.0, max(probe_frac / 8, per_step_elems / (len(pass_table()) * REF_SAMPLE_ELEMS)))
    for _ in range(args.warmup):
        oracle_step(full, threads, frac)
    elems, secs = 0.0, 0.0
    for _ in range(args.steps):
        e, s = oracle_step(full, threads, frac)
        elems += e
        secs += s
    value = elems / secs / 1e9
    n_prefix = max(64, int(REF_SAMPLE_ELEMS * frac) // 64 * 64)
    sample_desc = (f"first {n_prefix} elements of every tensor of the step, every pass of the step "
                   f"({len(pass_table())} quantize passes + MSE each, dequantize)")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": secs / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD_NAME + " (bounded sample)", "sample_elems_per_tensor": n_prefix},
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
        self.torch, self.mxq, self.device = torch, mxq, device
        self.x = make_inputs(rank, device)
        self.passes = pass_table()
        nmax = SEARCH_N
        self.codes = torch.empty(nmax // 2, dtype=torch.uint8, device=device)
        self.scales = torch.empty(nmax // 2, dtype=torch.uint8, device=device)
        self.sse = torch.empty(nmax // 2, dtype=torch.float32, device=device)
        self.mse = torch.zeros(len(self.passes), dtype=torch.float64, device=device)
        self.ws = torch.empty(mxq.mxq_tensor_mse_workspace_bytes(nmax // 2) // 8, dtype=torch.float64, device=device)
        self.amax = torch.empty(4, dtype=torch.float32, device=device)
        self.g = torch.empty(4, dtype=torch.float32, device=device)
        self.xhat = torch.empty(ACT_N, dtype=torch.bfloat16, device=device)
        self.search_events = {}   # (B, fmt) -> list of (start, stop)
        self.leg_events = {}      # leg -> list of (start, stop)
        self.elems_per_step = float(sum(p[2] for p in self.passes))

    def _ev(self):
        return self.torch.cuda.Event(enable_timing=True)

    def step(self, x=None, timed=False):
        """One pass of the whole hot path.  x: the tensors to read (default: the resident set)."""
        mxq = self.mxq
        x = x or self.x
        slot = 0
        leg_start = {}
        prev_leg = None
        g_for = {}
        for leg, key, n, B, fmt, recipe, hier in self.passes:
            if timed and leg != prev_leg:
                if prev_leg is not None:
                    e = self._ev(); e.record()
                    self.leg_events.setdefault(prev_leg, []).append((leg_start[prev_leg], e))
                leg_start[leg] = self._ev(); leg_start[leg].record()
            prev_leg = leg
            t = x[key]
            dg = None
            if hier:
                if key not in g_for:             # hierarchical scaling: tensor abs-max -> g, on the device
                    i = len(g_for)
                    mxq.mxq_tensor_amax(t, n, self.amax[i:i + 1], self.g[i:i + 1])
                    g_for[key] = self.g[i:i + 1]
                dg = g_for[key]
            ev = None
            if timed and leg == "search":
                ev = (self._ev(), self._ev())
                ev[0].record()
            # quantize + tensor MSE in one call: the kernel sums its own block SSEs, a one-CTA kernel finishes
            mxq.mxq_quantize_mse(t, n, B, fmt, recipe, 1.0, dg, self.codes, self.scales, self.sse,
                                 self.mse[slot:slot + 1], self.ws)
            if ev is not None:
                ev[1].record()
                self.search_events.setdefault((B, fmt), []).append(ev)
            slot += 1
        # the last pass left UE5M3 / 4-over-6 codes of an activation tensor: de-quantize them
        mxq.mxq_dequantize(self.codes, self.scales, ACT_N, 16, UE5M3, 1.0, self.xhat)
        if timed:
            e = self._ev(); e.record()
            self.leg_events.setdefault(prev_leg, []).append((leg_start[prev_leg], e))

    def mean_ms(self, evs):
        return sum(a.elapsed_time(b) for a, b in evs) / len(evs)


def graph_timed(torch, body, launches: int, reps: int = 5):
    """Average duration (ms) of one launch of `body`'s launch sequence when it is replayed from a CUDA
    graph (host launch overhead excluded), median over reps; also the plain Python-loop figure."""
    body()
    torch.cuda.synchronize()
    loop = []
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); body(); e1.record()
        torch.cuda.synchronize()
        loop.append(e0.elapsed_time(e1) / launches)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        body()
    torch.cuda.current_stream().wait_stream(s)
    gr = torch.cuda.CUDAGraph()
    with torch.cuda.graph(gr):
        body()
    gr.replay()
    torch.cuda.synchronize()
    rep = []
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); gr.replay(); e1.record()
        torch.cuda.synchronize()
        rep.append(e0.elapsed_time(e1) / launches)
    del gr
    return statistics.median(rep), statistics.median(loop)


def hbm_entry(n, elem_bytes, B, ms, ms_loop, peaks, extra=None):
    ach = algorithmic_bytes(n, elem_bytes, B) / (ms * 1e-3) / 1e9
    d = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
         "frac_of_nominal_8TBs": ach / NOMINAL_HBM_GBS, "ms_per_launch": ms, "ms_per_launch_python_loop": ms_loop,
         "gelem_s": n / (ms * 1e-3) / 1e9, "elems": n, "peak_source": peaks["source"]}
    if extra:
        d.update(extra)
    return d


def config_size_rooflines(torch, mxq, wl, peaks):
    """The one-pass kernels at the sizes of the step's own tensors: launches back to back over copies
    of the tensor that together exceed L2, replayed from a CUDA graph (and as a plain Python loop)."""
    out = {}
    cases = [("w_q", 4096 * 4096), ("w_k", 1024 * 4096), ("w_gate", 14336 * 4096), ("act", ACT_N)]
    for key, n in cases:
        src = wl.x["a_0"] if key == "act" else wl.x[key]
        ncopies = max(3, min(48, (512 << 20) // (n * 2)))
        xs = [src] + [src.clone() for _ in range(ncopies - 1)]
        for recipe in (ABSMAX, R4O6):
            for B in (16, 8):
                if B == 8 and key not in ("w_q", "w_gate"):
                    continue
                codes, scales, sse = mxq.alloc_outputs(n, B, src.device)

                def body():
                    for x in xs:
                        mxq.mxq_quantize_ex(x, n, B, UE4M3, recipe, 1.0, None, codes, scales, sse)
                ms, ms_loop = graph_timed(torch, body, len(xs))
                out[f"{RECIPE_NAME[recipe]}_bf16_B{B}_{key}"] = hbm_entry(
                    n, 2, B, ms, ms_loop, peaks, {"l2": f"{len(xs)} copies of the tensor, {len(xs) * n * 2 >> 20} MiB, round-robin"})
        del xs
    return out


def streaming_rooflines(torch, mxq, device, peaks):
    """HBM-bound kernels on a tensor far larger than L2 (134M elements), launches back to back."""
    from paper_2605_08565_b200 import inputs
    out = {}
    n = STREAM_ELEMS
    prof = {("bf16", ABSMAX): "k_quantize_absmax_bf16_B16_128Mi.txt", ("bf16", R4O6): "k_quantize_4o6_bf16_B16_128Mi.txt",
            ("f32", ABSMAX): "k_quantize_absmax_f32_B16_128Mi.txt", ("f32", R4O6): "k_quantize_4o6_f32_B16_128Mi.txt"}
    for name, dt, recipe, B in (
            ("absmax_bf16_B16", torch.bfloat16, ABSMAX, 16), ("4o6_bf16_B16", torch.bfloat16, R4O6, 16),
            ("absmax_f32_B16", torch.float32, ABSMAX, 16), ("4o6_f32_B16", torch.float32, R4O6, 16),
            ("absmax_bf16_B64", torch.bfloat16, ABSMAX, 64), ("4o6_bf16_B8", torch.bfloat16, R4O6, 8)):
        codes, scales, sse = mxq.alloc_outputs(n, B, device)
        xs = [inputs.student_t(n, 5, 0.02, 2 + i, dt, device) for i in range(2)]

        def body():
            for _ in range(3):
                for x in xs:
                    mxq.mxq_quantize_ex(x, n, B, UE4M3, recipe, 1.0, None, codes, scales, sse)
        ms, ms_loop = graph_timed(torch, body, 6)
        rec = recorded_profile(prof.get(("bf16" if dt == torch.bfloat16 else "f32", recipe), "-"),
                               ("mxq_quantize.cuh", "mxq_device.cuh")) if B == 16 else None
        extra = {"l2": "input larger than L2"}
        if rec is not None:
            extra.update(traffic=rec["dram_bytes"], traffic_source=rec["file"], traffic_stale=rec["stale"])
        out[name] = hbm_entry(n, xs[0].element_size(), B, ms, ms_loop, peaks, extra)
        del xs
    x = inputs.student_t(n, 5, 0.02, 2, torch.bfloat16, device)
    amax = torch.empty(1, dtype=torch.float32, device=device)

    def body_amax():
        for _ in range(6):
            mxq.mxq_tensor_amax(x, n, amax)
    ms, ms_loop = graph_timed(torch, body_amax, 6)
    ach = n * 2.0 / (ms * 1e-3) / 1e9
    out["tensor_amax_bf16"] = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                               "frac": ach / peaks["hbm_gbs"], "frac_of_nominal_8TBs": ach / NOMINAL_HBM_GBS,
                               "ms_per_launch": ms, "ms_per_launch_python_loop": ms_loop, "elems": n}
    codes, scales, sse = mxq.alloc_outputs(n, 16, device)
    mxq.mxq_quantize_ex(x, n, 16, UE4M3, ABSMAX, 1.0, None, codes, scales, sse)
    xh = torch.empty(n, dtype=torch.float32, device=device)

    def body_deq():
        for _ in range(6):
            mxq.mxq_dequantize(codes, scales, n, 16, UE4M3, 1.0, xh)
    ms, ms_loop = graph_timed(torch, body_deq, 6)
    ach = n * (0.5 + 1.0 / 16 + 4.0) / (ms * 1e-3) / 1e9
    out["dequantize_B16_to_f32"] = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                    "frac": ach / peaks["hbm_gbs"], "frac_of_nominal_8TBs": ach / NOMINAL_HBM_GBS,
                                    "ms_per_launch": ms, "ms_per_launch_python_loop": ms_loop, "elems": n}
    return out


def weight_set_report(torch, mxq, device, peaks, layers: int = 8):
    """A quarter of the Llama-3-8B-shaped weight set (8 layers x 7 matrices, 1.74 G bf16 elements) quantized
    three ways: one launch per matrix from a Python loop, the same launches replayed from a CUDA graph, and
    ONE multi-tensor launch (mxq_quantize_batch); abs-max and 4-over-6, B = 16, UE4M3."""
    from paper_2605_08565_b200 import inputs
    xs = []
    for layer in range(layers):
        for idx, (name, rows_, cols) in enumerate(inputs.LLAMA8B_LAYER_SHAPES):
            xs.append(inputs.student_t(rows_ * cols, 4, 1.0 / math.sqrt(cols), 4 + layer * 7 + idx, torch.bfloat16, device))
    outs = [mxq.alloc_outputs(x.numel(), 16, device) for x in xs]
    h, d = mxq.make_tensor_descs([(x, c, s_, e) for x, (c, s_, e) in zip(xs, outs)])
    n_total = sum(x.numel() for x in xs)
    res = {"matrices": len(xs), "elements": n_total}
    for recipe in (ABSMAX, R4O6):
        def per_matrix():
            for x, (c, s_, e) in zip(xs, outs):
                mxq.mxq_quantize_ex(x, x.numel(), 16, UE4M3, recipe, 1.0, None, c, s_, e)

        def batched():
            mxq.mxq_quantize_batch(h, d, len(xs), mxq.MXQ_BF16, 16, UE4M3, recipe, 1.0)
        ms_graph, ms_loop = graph_timed(torch, per_matrix, 1, reps=3)
        ms_batch_graph, ms_batch = graph_timed(torch, batched, 1, reps=3)
        nbytes = algorithmic_bytes(n_total, 2, 16)
        res[RECIPE_NAME[recipe]] = {
            "per_matrix_python_loop_ms": ms_loop, "per_matrix_graph_ms": ms_graph, "one_batch_launch_ms": ms_batch,
            "gelem_s": {"per_matrix_python_loop": n_total / ms_loop / 1e6, "per_matrix_graph": n_total / ms_graph / 1e6,
                        "one_batch_launch": n_total / ms_batch / 1e6},
            "frac_of_measured_hbm": {"per_matrix_python_loop": nbytes / ms_loop / 1e6 / peaks["hbm_gbs"],
                                     "per_matrix_graph": nbytes / ms_graph / 1e6 / peaks["hbm_gbs"],
                                     "one_batch_launch": nbytes / ms_batch / 1e6 / peaks["hbm_gbs"]}}
    return res


def pruned_sweep_report(torch, mxq, wl):
    """The 15 brute-force sweeps of the step once more with the pruned sweep switched on (outside the timed
    region; `value` and `roofline` are always the full sweep): per sweep the time of both modes on the same
    tensor and whether every output byte is identical."""
    out = {}
    x = wl.x["search"]
    n = x.numel()
    dg = wl.g[0:1]
    mxq.mxq_tensor_amax(x, n, wl.amax[0:1], dg)
    try:
        for B in SEARCH_BLOCKS:
            for fmt in SEARCH_FMTS:
                res = {}
                ms = {}
                for mode in (0, 1):
                    mxq.mxq_set_option(mxq.MXQ_OPT_BRUTE_PRUNE, mode)
                    codes, scales, sse = mxq.alloc_outputs(n, B, x.device)
                    mxq.mxq_quantize_ex(x, n, B, fmt, BRUTE, 1.0, dg, codes, scales, sse)
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    mxq.mxq_quantize_ex(x, n, B, fmt, BRUTE, 1.0, dg, codes, scales, sse)
                    e1.record()
                    torch.cuda.synchronize()
                    ms[mode] = e0.elapsed_time(e1)
                    res[mode] = (codes, scales, sse)
                same = all(torch.equal(a.view(torch.uint8), b.view(torch.uint8)) for a, b in zip(res[0], res[1]))
                out[f"B{B}_{FMT_NAME[fmt]}"] = {"full_ms": ms[0], "pruned_ms": ms[1], "speedup": ms[0] / ms[1],
                                               "outputs_identical": bool(same)}
                del res
    finally:
        mxq.mxq_set_option(mxq.MXQ_OPT_BRUTE_PRUNE, 0)
    return out


def spawn_ranks(n_ranks: int, script: str | None = None, argv=None) -> int:
    """`--gpus N` without a torchrun environment: start the N ranks on this node (one process per GPU,
    rendezvous on 127.0.0.1) with the same command line; their output goes to this process's stdout."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_ranks}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), script or os.path.abspath(__file__)]
    return subprocess.call(cmd + list(sys.argv[1:] if argv is None else argv))


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
    for _ in range(args.warmup):
        wl.step()
    torch.cuda.synchronize()

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
        wl.step(timed=True)
    e1.record()
    torch.cuda.synchronize()
    dist.barrier()
    launches = mxq.mxq_launch_count() - launches0
    local_s = e0.elapsed_time(e1) / 1e3
    clocks = sampler.stop() if rank == 0 else None
    value, t_max = dist.whole_job_throughput(wl.elems_per_step * args.steps, local_s)
    mse_host = wl.mse.cpu().numpy().copy()

    # ---- end to end: host buffers, H2D of the step's inputs and D2H of its results every step ----
    # The inputs of step i + 1 are copied on a second stream into the other of two device sets while
    # step i computes; every copy is awaited by the compute stream, so all of them lie inside the
    # timed region.
    host_in = {k: v.cpu().pin_memory() for k, v in wl.x.items()}
    h2d_bytes = sum(v.numel() * v.element_size() for v in host_in.values())
    host_out = torch.empty(wl.mse.numel(), dtype=torch.float64).pin_memory()
    dev_in = [{k: torch.empty_like(v) for k, v in wl.x.items()} for _ in range(2)]
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
                for k, v in host_in.items():
                    dev_in[i % 2][k].copy_(v, non_blocking=True)
                ready[i % 2].record(copy_stream)

        enqueue_copy(0)
        for i in range(n_steps):
            if i + 1 < n_steps:
                enqueue_copy(i + 1)
            main_stream.wait_event(ready[i % 2])
            wl.step(x=dev_in[i % 2])
            free[i % 2].record(main_stream)
            host_out.copy_(wl.mse, non_blocking=True)

    e2e_steps = max(2, min(args.steps, 10))
    e2e_loop(2)
    torch.cuda.synchronize()
    dist.barrier()
    e0.record()
    e2e_loop(e2e_steps)
    e1.record()
    torch.cuda.synchronize()
    dist.barrier()
    e2e_value, _ = dist.whole_job_throughput(wl.elems_per_step * e2e_steps, e0.elapsed_time(e1) / 1e3)
    del dev_in

    # ---- end to end, second form: one abs-max pass whose codes and scale bytes go back to the host ----
    nq = 14336 * 4096
    hq_in = host_in["w_gate"]
    dq_in = torch.empty_like(wl.x["w_gate"])
    cq, sq, _ = mxq.alloc_outputs(nq, 16, device, with_sse=False)
    hq_codes = torch.empty(nq // 2, dtype=torch.uint8).pin_memory()
    hq_scales = torch.empty(nq // 16, dtype=torch.uint8).pin_memory()

    def to_host_loop(k):
        for _ in range(k):
            dq_in.copy_(hq_in, non_blocking=True)
            mxq.mxq_quantize_ex(dq_in, nq, 16, UE4M3, ABSMAX, 1.0, None, cq, sq, None)
            hq_codes.copy_(cq, non_blocking=True)
            hq_scales.copy_(sq, non_blocking=True)
    to_host_loop(2)
    torch.cuda.synchronize()
    dist.barrier()
    e0.record()
    to_host_loop(10)
    e1.record()
    torch.cuda.synchronize()
    dist.barrier()
    q2h_value, _ = dist.whole_job_throughput(float(nq) * 10, e0.elapsed_time(e1) / 1e3)

    if rank != 0:
        dist.shutdown()
        return

    # ---- roofline of the dominant kernel: every brute-force launch of the step, time-weighted ----
    sm_mhz = (clocks or {}).get("sm_mhz") or peaks["sm_max_mhz"]
    n_sm = torch.cuda.get_device_properties(device).multi_processor_count
    alu_peak = n_sm * ALU_LANES_PER_SM * peaks["sm_max_mhz"] * 1e6 / 1e12          # Tlaneop/s at the maximum SM clock
    per_inst, tot_ops, tot_ms = {}, 0.0, 0.0
    for (B, fmt), evs in wl.search_events.items():
        ms = wl.mean_ms(evs)
        ops = SEARCH_N * N_CODES[fmt] * 4.0                                        # 4 lane-ops per (element, code)
        per_inst[f"B{B}_{FMT_NAME[fmt]}"] = {"ms_per_launch": ms, "achieved": ops / (ms * 1e-3) / 1e12,
                                             "frac": ops / (ms * 1e-3) / 1e12 / alu_peak,
                                             "gelem_s": SEARCH_N / (ms * 1e-3) / 1e9}
        tot_ops += ops
        tot_ms += ms
    step_ms = t_max / args.steps * 1e3
    largest = max(per_inst, key=lambda k: per_inst[k]["ms_per_launch"])
    rec = recorded_profile("k_brute_f32_B16_ue4m3_tensor_scale_16Mi.txt", ("mxq_brute.cuh", "mxq_device.cuh"))
    traffic = None
    if rec["dram_bytes"] is not None and rec["elems"]:
        traffic = rec["dram_bytes"] * SEARCH_N / rec["elems"]      # input and outputs grow in proportion to the elements
    roofline = {"kernel": "k_brute<f32, B, fmt> full sweep, tensor scale: the 15 launches of a step, time-weighted",
                "bound": "alu", "achieved": tot_ops / (tot_ms * 1e-3) / 1e12, "peak": alu_peak, "unit": "Tlaneop/s",
                "frac": tot_ops / (tot_ms * 1e-3) / 1e12 / alu_peak,
                "frac_at_observed_clock": tot_ops / (tot_ms * 1e-3) / 1e12 / (n_sm * ALU_LANES_PER_SM * sm_mhz * 1e6 / 1e12),
                "traffic": traffic, "traffic_source": rec["file"] + " (16.8M-element capture scaled to 268M elements)",
                "traffic_stale": rec["stale"], "ncu_issue_active_pct_recorded": rec["issue_active_pct"],
                "peak_source": f"{n_sm} SMs x 128 lanes x {peaks['sm_max_mhz']:.0f} MHz (max SM clock, {peaks['source']})",
                "launches_per_step": len(per_inst), "ms_per_launch": tot_ms / len(per_inst),
                "ms_all_launches_per_step": tot_ms, "share_of_step_time": tot_ms / step_ms,
                "largest_share": largest, "per_instantiation": per_inst}
    legs = {leg: {"ms_per_step": wl.mean_ms(evs),
                  "gelem_s": sum(p[2] for p in wl.passes if p[0] == leg) / (wl.mean_ms(evs) * 1e-3) / 1e9}
            for leg, evs in wl.leg_events.items()}

    hbm = None if args.skip_extras else config_size_rooflines(torch, mxq, wl, peaks)
    streaming = None if args.skip_extras else streaming_rooflines(torch, mxq, device, peaks)
    pruned = None if args.skip_extras else pruned_sweep_report(torch, mxq, wl)
    weight_set = None if args.skip_extras else weight_set_report(torch, mxq, device, peaks)

    # ---- CPU oracle on a bounded sample of the same workload ------------------------------------
    from oracle import mxq_oracle as orc
    from paper_2605_08565_b200 import inputs
    orc.build()
    threads = host_threads()
    samples = {k: inputs.to_numpy_bits(v[:CPU_SAMPLE_ELEMS]) for k, v in wl.x.items()}
    oracle_step(samples, threads, 4096.0 / CPU_SAMPLE_ELEMS)
    c_elems, c_secs = oracle_step(samples, threads)
    cpu_baseline = {"value": c_elems / c_secs / 1e9, "unit": UNIT, "cores": threads, "kind": "oracle", "seconds": c_secs,
                    "sample": f"first {CPU_SAMPLE_ELEMS} elements of every tensor of the step, every pass of one step"}

    names = [f"{leg}:{key}:B{B}:{FMT_NAME[fmt]}:{RECIPE_NAME[r]}" + (":g" if hier else "")
             for leg, key, _, B, fmt, r, hier in wl.passes]
    print(json.dumps({
        "metric": METRIC, "value": value / 1e9, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD_NAME, "elements_per_step": wl.elems_per_step, "passes_per_step": len(wl.passes),
                   "l2": "search tensor 1 GiB > 126 MB L2; the legs walk their tensors round-robin (277 MB and 201 MB sets)"},
        "roofline": roofline, "legs": legs, "roofline_hbm": hbm, "roofline_hbm_streaming": streaming,
        "brute_pruned_sweep": pruned, "weight_set_8_layers": weight_set, "cpu_baseline": cpu_baseline,
        "e2e": {"value": e2e_value / 1e9, "unit": UNIT, "h2d_bytes_per_step": int(h2d_bytes),
                "d2h_bytes_per_step": int(host_out.numel() * 8), "steps": e2e_steps,
                "what": "the same step with all inputs copied from pinned host memory every step (overlapped with the "
                        "previous step) and the per-pass MSE values copied back"},
        "e2e_quantize_to_host": {"value": q2h_value / 1e9, "unit": UNIT, "h2d_bytes_per_step": int(nq * 2),
                                 "d2h_bytes_per_step": int(nq // 2 + nq // 16),
                                 "what": "one abs-max pass (14336x4096 bf16, B=16, UE4M3): input from pinned host memory, "
                                         "codes and scale bytes back to pinned host memory, one stream, no overlap"},
        "gpu_launches": int(launches), "clocks": clocks,
        "mse": {nm: float(mse_host[i]) for i, nm in enumerate(names)},
    }))
    dist.shutdown()


# ------------------------------------------------------------------------------------------------
# --config: the five benchmark configurations, one recipe at a time
# ------------------------------------------------------------------------------------------------
class _Acc:
    """CUDA-event time and elements per (B, fmt, recipe, tensor-scale) key.  A key's tensors are quantized
    back to back inside one event pair (after one untimed launch), `rounds` times over; sequences of four
    or more one-pass launches are replayed from a CUDA graph (the Python-loop time is kept beside it); the
    tensor MSE is taken afterwards, untimed."""

    def __init__(self, torch, mxq):
        self.torch, self.mxq = torch, mxq
        self.ms, self.ms_loop, self.elems, self.mse = {}, {}, {}, {}

    def run(self, key, xs, B, fmt, recipe, g, dgs, bufs, rounds=1):
        self._run(key, xs, B, fmt, recipe, g, dgs, bufs, rounds)
        if recipe in (BRUTE, BRUTE_PZ):   # the same pass with the pruned sweep, as a row of its own
            self.mxq.mxq_set_option(self.mxq.MXQ_OPT_BRUTE_PRUNE, 1)
            try:
                self._run(key + ("pruned",), xs, B, fmt, recipe, g, dgs, bufs, rounds)
            finally:
                self.mxq.mxq_set_option(self.mxq.MXQ_OPT_BRUTE_PRUNE, 0)

    def _run(self, key, xs, B, fmt, recipe, g, dgs, bufs, rounds):
        torch, mxq = self.torch, self.mxq
        codes, scales, sse, mse_out, ws = bufs
        dgs = dgs if dgs is not None else [None] * len(xs)

        def body():
            for _ in range(rounds):
                for x, dg in zip(xs, dgs):
                    mxq.mxq_quantize_ex(x, x.numel(), B, fmt, recipe, g, dg, codes, scales, sse)

        launches = rounds * len(xs)
        if recipe not in (BRUTE, BRUTE_PZ) and launches >= 4:
            # microsecond kernels: replayed from a CUDA graph, so that the host's launch rate is not what is timed
            ms_graph, ms_loop = graph_timed(torch, body, 1, reps=3)
            self.ms_loop[key] = self.ms_loop.get(key, 0.0) + ms_loop
        else:
            mxq.mxq_quantize_ex(xs[0], xs[0].numel(), B, fmt, recipe, g, dgs[0], codes, scales, sse)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            body()
            e1.record()
            torch.cuda.synchronize()
            ms_graph = e0.elapsed_time(e1)
        tot, cnt = 0.0, 0
        for x, dg in zip(xs, dgs):
            mxq.mxq_quantize_ex(x, x.numel(), B, fmt, recipe, g, dg, codes, scales, sse)
            mxq.mxq_tensor_mse(sse, x.numel() // B, x.numel(), mse_out, ws)
            tot += float(mse_out.cpu()[0]) * x.numel()
            cnt += x.numel()
        torch.cuda.synchronize()
        self.ms[key] = self.ms.get(key, 0.0) + ms_graph
        self.elems[key] = self.elems.get(key, 0) + cnt * rounds
        m = self.mse.setdefault(key, [0.0, 0])
        m[0] += tot
        m[1] += cnt

    def rows(self, cfg, elem_bytes, hbm_gbs, alu_peak):
        out = []
        for key, ms in self.ms.items():
            B, fmt, recipe, gk = key[:4]
            pruned = len(key) > 4
            n = self.elems[key]
            ge = n / ms / 1e6
            row = {"config": cfg, "block": B, "scale_fmt": FMT_NAME[fmt],
                   "recipe": RECIPE_NAME[recipe] + ("+prune" if pruned else ""), "tensor_scale": gk,
                   "elements": n, "ms": ms, "gelem_s": ge, "mse": self.mse[key][0] / self.mse[key][1]}
            if pruned:
                # codes left out are not work done: no roofline fraction, only the speed-up over the full sweep
                full = self.elems[key[:4]] / self.ms[key[:4]] / 1e6
                row.update(bound="alu", speedup_over_full_sweep=ge / full, frac=None)
            elif recipe in (BRUTE, BRUTE_PZ):
                ach = ge * 1e9 * N_CODES[fmt] * 4 / 1e12
                row.update(bound="alu", achieved_tlaneop_s=ach, frac=ach / alu_peak)
            else:
                ach = ge * (elem_bytes + 0.5 + 5.0 / B)
                row.update(bound="hbm", achieved_gb_s=ach, frac=ach / hbm_gbs, frac_of_8tbs=ach / NOMINAL_HBM_GBS)
                if key in self.ms_loop:
                    row.update(timed="cuda graph replay", ms_python_loop=self.ms_loop[key])
            out.append(row)
        return out


class _InputDigest:
    """SHA-256 over the bytes of a configuration's input tensors, in generation order (so that a run
    can be tied to the exact inputs it quantized); computed on the host, only when asked for."""

    def __init__(self, enabled):
        self.h = hashlib.sha256() if enabled else None
        self.tensors, self.elements = 0, 0

    def add(self, x):
        import torch
        self.tensors += 1
        self.elements += x.numel()
        if self.h is not None:
            self.h.update(x.view(torch.uint8).cpu().numpy().tobytes())

    def result(self):
        return {"tensors": self.tensors, "elements": self.elements,
                "sha256": self.h.hexdigest() if self.h is not None else None}


def run_configs(configs, hash_inputs=False):
    """Times every (configuration, block size, scale format, recipe) of the five benchmark configurations
    at full size with CUDA events: the quantize launches of a row back to back (tensors larger than L2 or
    rotated so that inputs come from HBM), replayed from a CUDA graph where a launch lasts microseconds
    (the one-pass recipes) and called from Python where it lasts milliseconds (brute force); the tensor MSE
    afterwards, untimed."""
    import torch
    from paper_2605_08565_b200 import binding as mxq
    from paper_2605_08565_b200 import inputs
    if not torch.cuda.is_available():
        raise mxq.MxqError("needs a CUDA device (no CPU fallback)")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    peaks = measured_peaks()
    hbm, mhz = peaks["hbm_gbs"], peaks["sm_max_mhz"]
    n_sm = torch.cuda.get_device_properties(dev).multi_processor_count
    alu_peak = n_sm * ALU_LANES_PER_SM * mhz * 1e6 / 1e12
    A, P, R4, R4P, BR, BRP = ABSMAX, ABSMAX_PZ, R4O6, R4O6_PZ, BRUTE, BRUTE_PZ
    rows, digests = [], {}

    def bufs(n, B):
        codes, scales, sse = mxq.alloc_outputs(n, B, dev)
        return (codes, scales, sse, torch.empty(1, dtype=torch.float64, device=dev),
                torch.empty(mxq.mxq_tensor_mse_workspace_bytes(n // B) // 8, dtype=torch.float64, device=dev))

    def tensor_scale(x):
        amax = torch.empty(1, dtype=torch.float32, device=dev)
        dg = torch.empty(1, dtype=torch.float32, device=dev)
        mxq.mxq_tensor_amax(x, x.numel(), amax, dg)
        return dg

    warm = inputs.normal(1 << 20, 0, 1.0, torch.float32, dev)          # first-launch costs out of the way
    for r in (A, R4, BR):
        mxq.quantize(warm, 16, UE4M3, r)

    if 1 in configs:   # 1024 x 1024 fp32 N(0,1), B=16, UE4M3 + tensor scale; 4 MB: L2-resident, launch-bound
        x = inputs.normal(1024 * 1024, 1, 1.0, torch.float32, dev)
        digests["C1"] = _InputDigest(hash_inputs)
        digests["C1"].add(x)
        dg = tensor_scale(x)
        acc, b = _Acc(torch, mxq), bufs(x.numel(), 16)
        for r in (A, R4, BR):
            acc.run((16, UE4M3, r, "amax/2688"), [x], 16, UE4M3, r, 1.0, [dg], b, rounds=50)
        rows += acc.rows("C1 1024x1024 fp32 N(0,1)", 4, hbm, alu_peak)

    if 2 in configs:   # 4096 x 4096 bf16 0.02 * t5, all block sizes, UE4M3, no tensor scale; 8 rotating tensors
        xs = [inputs.student_t(4096 * 4096, 5, 0.02, 2 * 1_000_003 + i, torch.bfloat16, dev) for i in range(8)]
        digests["C2"] = _InputDigest(hash_inputs)
        for x in xs:
            digests["C2"].add(x)
        acc = _Acc(torch, mxq)
        for B in (2, 4, 8, 16, 32, 64):
            b = bufs(xs[0].numel(), B)
            for r in (A, P, R4, BR):
                acc.run((B, UE4M3, r, "none"), xs, B, UE4M3, r, 1.0, None, b, rounds=4 if r != BR else 1)
        rows += acc.rows("C2 4096x4096 bf16 0.02*t5", 2, hbm, alu_peak)
        del xs

    if 3 in configs:   # 8192 x 4096 bf16 N(0,1) with 1 % outlier columns x50, B=16; 4 rotating tensors
        xs = [inputs.outlier_columns(8192, 4096, 3 + i, dtype=torch.bfloat16, device=dev) for i in range(4)]
        digests["C3"] = _InputDigest(hash_inputs)
        for x in xs:
            digests["C3"].add(x)
        dgs = [tensor_scale(x) for x in xs]
        acc, b = _Acc(torch, mxq), bufs(xs[0].numel(), 16)
        for r in (A, R4):
            acc.run((16, UE4M3, r, "amax/2688"), xs, 16, UE4M3, r, 1.0, dgs, b, rounds=4)
            acc.run((16, UE5M3, r, "none"), xs, 16, UE5M3, r, 1.0, None, b, rounds=4)
        rows += acc.rows("C3 8192x4096 bf16 outlier columns", 2, hbm, alu_peak)
        del xs

    if 4 in configs:   # Llama-3-8B-shaped weight set, 224 matrices: one launch per matrix, then one launch for all
        acc = _Acc(torch, mxq)
        digests["C4"] = _InputDigest(hash_inputs)
        xs = []
        for layer in range(inputs.LLAMA8B_LAYERS):
            for idx, (name, rows_, cols) in enumerate(inputs.LLAMA8B_LAYER_SHAPES):
                x = inputs.student_t(rows_ * cols, 4, 1.0 / math.sqrt(cols), 4 + layer * 7 + idx, torch.bfloat16, dev)
                digests["C4"].add(x)
                xs.append(x)
        # one matrix at a time: the 224 launches of a (block size, format, recipe) back to back, outputs into
        # one buffer set sized for the largest matrix
        n_max = max(x.numel() for x in xs)
        for B in (8, 16):
            b = bufs(n_max, B)
            for fmt in (UE4M3, UE5M3):
                for r in (A, P, R4, R4P, BR, BRP):
                    acc.run((B, fmt, r, "none"), xs, B, fmt, r, 1.0, None, b)
            del b
        name = "C4 Llama-3-8B-shaped set (224 matrices, 6.98 G elements)"
        rows += acc.rows(name, 2, hbm, alu_peak)
        # the same set through the multi-tensor entry point: ONE launch per (block size, format, recipe)
        n_total = sum(x.numel() for x in xs)
        for B in (8, 16):
            outs = [mxq.alloc_outputs(x.numel(), B, dev) for x in xs]
            h, d = mxq.make_tensor_descs([(x, c, s_, e) for x, (c, s_, e) in zip(xs, outs)])
            mse_out = torch.empty(1, dtype=torch.float64, device=dev)
            ws = torch.empty(1024, dtype=torch.float64, device=dev)
            for fmt in (UE4M3, UE5M3):
                for r in (A, P, R4, R4P):
                    mxq.mxq_quantize_batch(h, d, len(xs), mxq.MXQ_BF16, B, fmt, r, 1.0)
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    mxq.mxq_quantize_batch(h, d, len(xs), mxq.MXQ_BF16, B, fmt, r, 1.0)
                    e1.record()
                    tot = 0.0
                    for x, (c, s_, e) in zip(xs, outs):
                        mxq.mxq_tensor_mse(e, x.numel() // B, x.numel(), mse_out, ws)
                        tot += float(mse_out.cpu()[0]) * x.numel()
                    ms = e0.elapsed_time(e1)
                    ach = n_total * (2 + 0.5 + 5.0 / B) / ms / 1e6
                    rows.append({"config": name, "block": B, "scale_fmt": FMT_NAME[fmt], "recipe": RECIPE_NAME[r] + " (one batch launch)",
                                 "tensor_scale": "none", "elements": n_total, "ms": ms, "gelem_s": n_total / ms / 1e6,
                                 "mse": tot / n_total, "bound": "hbm", "achieved_gb_s": ach, "frac": ach / hbm,
                                 "frac_of_8tbs": ach / NOMINAL_HBM_GBS})
            del outs
        del xs

    if 5 in configs:   # 16384 x 16384 fp32 Laplace, brute force, tensor scale
        x = inputs.laplace(16384 * 16384, 5, torch.float32, dev)
        digests["C5"] = _InputDigest(hash_inputs)
        digests["C5"].add(x)
        dg = tensor_scale(x)
        acc = _Acc(torch, mxq)
        for B in (2, 4, 8, 16, 32):
            b = bufs(x.numel(), B)
            for fmt in (UE8M0, UE4M3, UE5M3):
                acc.run((B, fmt, BR, "amax/2688"), [x], B, fmt, BR, 1.0, [dg], b)
        rows += acc.rows("C5 16384x16384 fp32 Laplace", 4, hbm, alu_peak)
    return {"hbm_gbs": hbm, "alu_peak_tlaneop_s": alu_peak, "peak_source": peaks["source"], "rows": rows,
            "inputs": {k: d.result() for k, d in digests.items()}}


def run_config_mode(args) -> None:
    configs = (1, 2, 3, 4, 5) if args.config == "all" else tuple(int(c) for c in args.config.split(","))
    res = run_configs(configs, hash_inputs=args.hash_inputs)
    for r in res["rows"]:
        head = (f'{r["config"][:28]:28s} B={r["block"]:<2d} {r["scale_fmt"]:5s} {r["recipe"]:28s} g={r["tensor_scale"]:9s} '
                f'{r["gelem_s"]:9.1f} GElem/s  ')
        if r["frac"] is None:
            print(head + f'{r["speedup_over_full_sweep"]:8.2f} x the full sweep{"":14s}  mse={r["mse"]:.4e}', file=sys.stderr)
            continue
        ach = r.get("achieved_gb_s", r.get("achieved_tlaneop_s"))
        unit = "GB/s" if r["bound"] == "hbm" else "Tlop/s"
        print(head + f'{ach:8.1f} {unit:6s} {100 * r["frac"]:5.1f}% of {r["bound"]}  mse={r["mse"]:.4e}', file=sys.stderr)
    print(json.dumps(res))


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
    elif args.kernel == "hist":
        mxq.mxq_quantize_ex(x, n, B, fmt, 0, g, None, codes, scales, sse)
        ch = torch.zeros(16, dtype=torch.int64, device=dev)
        sh = torch.zeros(256, dtype=torch.int64, device=dev)
        fn = lambda: mxq.mxq_histograms(codes, scales, n, B, ch, sh)
        nbytes = n * (0.5 + 1.0 / B)
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
        res["tlaneop_s"] = n * N_CODES[fmt] * 4.0 / (ms * 1e-3) / 1e12
    print(json.dumps(res))


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--kernel", default=None, help="time one kernel alone: absmax|absmax_pz|4o6|4o6_pz|brute|brute_pz|amax|mse|dequant|hist")
    ap.add_argument("--config", default=None, help="time one benchmark configuration (1..5, comma list, or all), one recipe at a time")
    ap.add_argument("--hash-inputs", action="store_true", help="with --config: record the SHA-256 of every configuration's input bytes")
    ap.add_argument("--block", type=int, default=16)
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "f32"])
    ap.add_argument("--fmt", default="ue4m3", choices=["ue8m0", "ue4m3", "ue5m3"])
    ap.add_argument("--elems", type=int, default=1 << 27)
    ap.add_argument("--iters", type=int, default=5)
    ap.add_argument("--global-scale", type=float, default=1.0)
    ap.add_argument("--prune", action="store_true", help="with --kernel brute|brute_pz: the pruned sweep")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--skip-extras", action="store_true",
                    help="leave out the measurements taken outside the timed step (roofline_hbm, roofline_hbm_streaming, "
                         "brute_pruned_sweep = null)")
    ap.add_argument("--impl", default="mxq", choices=["mxq", "reference"])
    args = ap.parse_args()
    if args.kernel:
        run_single_kernel(args)
        return
    if args.config:
        run_config_mode(args)
        return
    if args.warmup < 3 and args.impl == "mxq":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args.gpus))
    run_gpu(args)


if __name__ == "__main__":
    main()
